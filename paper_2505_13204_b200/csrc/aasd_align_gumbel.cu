// Launchers of alignment sampling with keyed draws (GUMBEL mode) on the streaming path for
// one logits dtype (compiled once with -DAASD_DT=0 for fp32 and once with -DAASD_DT=1 for
// bf16): the best token for the alignment test, and ND >= k_extra draws per row.
#include "aasd_host.h"

#ifndef AASD_DT
#error "compile with -DAASD_DT=0 (fp32) or -DAASD_DT=1 (bf16)"
#endif

namespace aasd {
namespace {

constexpr int DT = AASD_DT;

template <int ND, bool FIN = false>
int launch_draws(const LaunchEnv& env, const StreamJob& sj, const AlignArgs& a, unsigned int grid) {
    return launch_stream<DT, 1, ND, false, FIN, AlignEpilogue<DT>>(env, sj, a, grid, false);
}

}  // namespace

#if AASD_DT == 0
int launch_align_gumbel_f32(const LaunchEnv& env, const StreamJob& sj, const AlignArgs& a, unsigned int grid) {
#else
int launch_align_gumbel_bf16(const LaunchEnv& env, const StreamJob& sj, const AlignArgs& a, unsigned int grid) {
#endif
    const int k = a.k_extra <= 1 ? 1 : (a.k_extra == 2 ? 2 : 4);
    if (a.hints & AASD_HINT_FINITE) {
        if (k == 1) return launch_draws<1, true>(env, sj, a, grid);
        if (k == 2) return launch_draws<2, true>(env, sj, a, grid);
        return launch_draws<4, true>(env, sj, a, grid);
    }
    if (k == 1) return launch_draws<1>(env, sj, a, grid);
    if (k == 2) return launch_draws<2>(env, sj, a, grid);
    return launch_draws<4>(env, sj, a, grid);
}

}  // namespace aasd
