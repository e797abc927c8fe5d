// Launchers of tree verification for one logits dtype (compiled once with -DAASD_DT=0 for
// fp32 and once with -DAASD_DT=1 for bf16).
#include "aasd_host.h"

#ifndef AASD_DT
#error "compile with -DAASD_DT=0 (fp32) or -DAASD_DT=1 (bf16)"
#endif

namespace aasd {

#if AASD_DT == 0
int launch_tree_f32(const LaunchEnv& env, const StreamJob* sj, const TreeArgs& a, unsigned int grid) {
#else
int launch_tree_bf16(const LaunchEnv& env, const StreamJob* sj, const TreeArgs& a, unsigned int grid) {
#endif
    constexpr int DT = AASD_DT;
    if (sj) {
        if (a.mode == AASD_VERIFY_STRICT_SAMPLED)
            return launch_stream<DT, 1, 1, false, false, TreeEpilogue<DT>>(env, *sj, a, grid, false);
        if (a.mode == AASD_VERIFY_TOP_K)   // the consumers also count the tokens ahead of each row's first child
            return launch_stream<DT, 1, 0, true, false, TreeEpilogue<DT>>(env, *sj, a, grid, false);
        return launch_stream<DT, 1, 0, false, false, TreeEpilogue<DT>>(env, *sj, a, grid, false);
    }
    launch(tree_kernel<DT>, grid, (unsigned int)kThreads, 0, env.stream, a);
    return AASD_OK;
}

}  // namespace aasd
