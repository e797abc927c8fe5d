// Launchers of the verification kernels for one logits dtype (compiled once with
// -DAASD_DT=0 for fp32 and once with -DAASD_DT=1 for bf16).
#include "aasd_host.h"

#ifndef AASD_DT
#error "compile with -DAASD_DT=0 (fp32) or -DAASD_DT=1 (bf16)"
#endif

namespace aasd {
namespace {

constexpr int DT = AASD_DT;

template <int ND, bool TK, bool FIN = false, int K = 1>
int launch_verify_stream(const LaunchEnv& env, const StreamJob& sj, const VerifyArgs& a, unsigned int grid) {
    return launch_stream<DT, K, ND, TK, FIN, VerifyEpilogue<DT>>(env, sj, a, grid, row_bytes_of(sj) < kShortVerifyRow);
}

// K: the best tokens kept per row (1; the table's width when the step extends the table)
template <int K>
int dispatch_mode(const LaunchEnv& env, const StreamJob& sj, const VerifyArgs& a, unsigned int grid) {
    const bool finite = (a.hints & AASD_HINT_FINITE) != 0;
    if (a.mode == AASD_VERIFY_STRICT_SAMPLED)
        return finite ? launch_verify_stream<1, false, true, K>(env, sj, a, grid)
                      : launch_verify_stream<1, false, false, K>(env, sj, a, grid);
    if (a.mode == AASD_VERIFY_TOP_K) return launch_verify_stream<0, true, false, K>(env, sj, a, grid);
    return finite ? launch_verify_stream<0, false, true, K>(env, sj, a, grid)
                  : launch_verify_stream<0, false, false, K>(env, sj, a, grid);
}

int dispatch_verify_stream(const LaunchEnv& env, const StreamJob& sj, const VerifyArgs& a, unsigned int grid) {
    if (!a.row_extra) return dispatch_mode<1>(env, sj, a, grid);
    // the table extension wants the best tokens of every row
    return a.seq.table_k > 2 ? dispatch_mode<4>(env, sj, a, grid) : dispatch_mode<2>(env, sj, a, grid);
}

}  // namespace

#if AASD_DT == 0
int launch_verify_f32(const LaunchEnv& env, const StreamJob* sj, const VerifyArgs& a, unsigned int grid) {
#else
int launch_verify_bf16(const LaunchEnv& env, const StreamJob* sj, const VerifyArgs& a, unsigned int grid) {
#endif
    if (sj) return dispatch_verify_stream(env, *sj, a, grid);
    if (!a.row_extra) launch(verify_kernel<DT, 1>, grid, kThreads, 0, env.stream, a);
    else if (a.seq.table_k > 2) launch(verify_kernel<DT, 4>, grid, kThreads, 0, env.stream, a);
    else launch(verify_kernel<DT, 2>, grid, kThreads, 0, env.stream, a);
    return AASD_OK;
}

}  // namespace aasd
