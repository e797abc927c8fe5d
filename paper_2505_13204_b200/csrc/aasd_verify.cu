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

int dispatch_verify_stream(const LaunchEnv& env, const StreamJob& sj, const VerifyArgs& a, unsigned int grid) {
    const bool finite = (a.hints & AASD_HINT_FINITE) != 0;
    if (a.row_extra) {
        // the table extension wants the best tokens of every row
        if (a.seq.table_k > 2)
            return finite ? launch_verify_stream<0, false, true, 4>(env, sj, a, grid)
                          : launch_verify_stream<0, false, false, 4>(env, sj, a, grid);
        return finite ? launch_verify_stream<0, false, true, 2>(env, sj, a, grid)
                      : launch_verify_stream<0, false, false, 2>(env, sj, a, grid);
    }
    if (a.mode == AASD_VERIFY_STRICT_SAMPLED)
        return finite ? launch_verify_stream<1, false, true>(env, sj, a, grid)
                      : launch_verify_stream<1, false>(env, sj, a, grid);
    if (a.mode == AASD_VERIFY_TOP_K) return launch_verify_stream<0, true>(env, sj, a, grid);
    return finite ? launch_verify_stream<0, false, true>(env, sj, a, grid)
                  : launch_verify_stream<0, false>(env, sj, a, grid);
}

}  // namespace

#if AASD_DT == 0
int launch_verify_f32(const LaunchEnv& env, const StreamJob* sj, const VerifyArgs& a, unsigned int grid) {
#else
int launch_verify_bf16(const LaunchEnv& env, const StreamJob* sj, const VerifyArgs& a, unsigned int grid) {
#endif
    if (sj) return dispatch_verify_stream(env, *sj, a, grid);
    launch(verify_kernel<DT>, grid, kThreads, 0, env.stream, a);
    return AASD_OK;
}

}  // namespace aasd
