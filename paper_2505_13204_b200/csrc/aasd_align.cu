// Launchers of the alignment-sampling kernels for one logits dtype (compiled once with
// -DAASD_DT=0 for fp32 and once with -DAASD_DT=1 for bf16): the extras that rank above the
// prompt token (TOPK) on the streaming path, and the plain-load kernels of both modes.
#include "aasd_host.h"

#ifndef AASD_DT
#error "compile with -DAASD_DT=0 (fp32) or -DAASD_DT=1 (bf16)"
#endif

namespace aasd {
namespace {

constexpr int DT = AASD_DT;

template <int K, bool FIN = false>
int launch_align_stream(const LaunchEnv& env, const StreamJob& sj, const AlignArgs& a, unsigned int grid) {
    return launch_stream<DT, K, 0, false, FIN, AlignEpilogue<DT>>(env, sj, a, grid, row_bytes_of(sj) < kShortAlignRow);
}

}  // namespace

#if AASD_DT == 0
int launch_align_topk_f32(const LaunchEnv& env, const StreamJob* sj, const AlignArgs& a, unsigned int grid) {
#else
int launch_align_topk_bf16(const LaunchEnv& env, const StreamJob* sj, const AlignArgs& a, unsigned int grid) {
#endif
    if (sj) {
        const int k = a.k_extra <= 1 ? 1 : (a.k_extra == 2 ? 2 : 4);
        if (a.hints & AASD_HINT_FINITE) {
            if (k == 1) return launch_align_stream<1, true>(env, *sj, a, grid);
            if (k == 2) return launch_align_stream<2, true>(env, *sj, a, grid);
            return launch_align_stream<4, true>(env, *sj, a, grid);
        }
        if (k == 1) return launch_align_stream<1>(env, *sj, a, grid);
        if (k == 2) return launch_align_stream<2>(env, *sj, a, grid);
        return launch_align_stream<4>(env, *sj, a, grid);
    }
    // plain kernels: the K best tokens in TOPK mode, the best token alone in GUMBEL mode
    const int K = (a.k_extra <= 1 || a.mode == AASD_ALIGN_GUMBEL) ? 1 : (a.k_extra == 2 ? 2 : 4);
    if (K == 1) launch(align_kernel<DT, 1>, grid, kThreads, 0, env.stream, a);
    else if (K == 2) launch(align_kernel<DT, 2>, grid, kThreads, 0, env.stream, a);
    else launch(align_kernel<DT, 4>, grid, kThreads, 0, env.stream, a);
    return AASD_OK;
}

}  // namespace aasd
