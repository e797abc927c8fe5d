// Host-side internals shared by the translation units of the library: the context, the
// workspace layout, the launch helpers, and the launchers of the streaming kernels, which are
// compiled once per logits dtype in files of their own (aasd_verify.cu, aasd_align.cu,
// aasd_tree.cu) so that the library builds in parallel.
#pragma once

#include <cuda_runtime.h>

#include <atomic>
#include <map>

#include "../../include/aasd.h"
#include "aasd_rows.cuh"
#include "aasd_stream.cuh"
#include "aasd_tree.cuh"

namespace aasd {

struct WorkspaceLayout {
    size_t bytes;
    int64_t max_rows, max_cands;
    size_t off_partials, off_row_tickets, off_cand_tickets, off_seq_tickets, off_sched, off_row_accept, off_row_own, off_next, off_race,
        off_tree_stats, off_row_extra;
    bool full;
};

constexpr size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// with_tree: room for the per-row statistics of tree verification and for the per-row extras
// of the table extension (the fixed block of aasd_verify_static does without both).
constexpr WorkspaceLayout make_layout(int64_t max_rows, int64_t max_cands, bool with_tree = true) {
    WorkspaceLayout L{};
    L.max_rows = max_rows;
    L.max_cands = max_cands;
    size_t o = 0;
    L.off_partials = o;
    o = align_up(o + sizeof(RowPartial) * (size_t)kPartialSlots, 256);
    L.off_row_tickets = o;
    o = align_up(o + 4 * (size_t)max_rows, 256);
    L.off_cand_tickets = o;
    o = align_up(o + 4 * (size_t)max_cands, 256);
    L.off_seq_tickets = o;
    o = align_up(o + 4 * (size_t)max_cands, 256);
    L.off_sched = o;
    o = align_up(o + 2 * sizeof(unsigned int), 256);
    L.off_row_accept = o;
    o = align_up(o + (size_t)max_rows, 256);
    L.off_row_own = o;
    o = align_up(o + 8 * (size_t)max_rows, 256);
    L.off_next = o;
    o = align_up(o + 4 * (size_t)max_rows, 256);
    L.off_race = o;
    o = align_up(o + sizeof(RaceSummary) * (size_t)kRaceSlots * kMaxK, 256);
    L.off_tree_stats = o;
    if (with_tree) o = align_up(o + sizeof(TreeRowStat) * (size_t)max_rows, 256);
    L.off_row_extra = o;
    if (with_tree) o = align_up(o + sizeof(int32_t) * kRowExtraInts * (size_t)max_rows, 256);
    L.full = with_tree;
    L.bytes = o;
    return L;
}

#define AASD_CUDA(call)                                   \
    do {                                                  \
        cudaError_t e__ = (call);                         \
        if (e__ != cudaSuccess) return AASD_ERR_CUDA;     \
    } while (0)

// Every kernel of the library is launched with programmatic stream serialization: it may be
// scheduled while its predecessor in the stream drains, and waits (griddepcontrol.wait,
// first thing in each kernel) for that predecessor to complete before it touches memory.
// cluster > 1: the grid is made of thread-block clusters of that many CTAs.
template <class... Params, class... Args>
void launch_clustered(void (*kernel)(Params...), unsigned int grid, unsigned int block, size_t smem,
                      cudaStream_t stream, unsigned int cluster, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (cluster > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    cudaLaunchKernelEx(&cfg, kernel, Params(args)...);   // errors surface in cudaGetLastError
}
template <class... Params, class... Args>
void launch(void (*kernel)(Params...), unsigned int grid, unsigned int block, size_t smem, cudaStream_t stream,
            Args&&... args) {
    launch_clustered(kernel, grid, block, smem, stream, 1u, static_cast<Args&&>(args)...);
}

// Where a launch goes.
struct LaunchEnv {
    cudaStream_t stream;
    int device;
};

constexpr int kMaxDevices = 64;

// The streaming kernel needs more dynamic shared memory than a kernel gets by default; the
// attribute is set once per kernel and device, not on every call.
template <auto Kernel>
int enable_stream_smem(int device) {
    static std::atomic<unsigned long long> done{0ull};
    const unsigned long long bit = 1ull << (device & (kMaxDevices - 1));
    if (done.load(std::memory_order_acquire) & bit) return AASD_OK;
    if (cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemBytes) != cudaSuccess)
        return AASD_ERR_CUDA;
    done.fetch_or(bit, std::memory_order_release);
    return AASD_OK;
}

// One launch of the streaming kernel.  Rows that stream faster than a finisher gets through
// one (short_rows) take the variant with three finisher warps; sampling kernels, whose
// consumers are the slower side, always run with one.
template <int DT, int K, int ND, bool TK, bool FIN, class E>
int launch_stream(const LaunchEnv& env, const StreamJob& sj, const typename E::Args& a, unsigned int grid,
                  bool short_rows) {
    const unsigned int cluster = sj.cluster_pieces ? (unsigned int)sj.tail_chunks : 1u;
    if (ND == 0 && short_rows) {
        constexpr auto kernel = stream_kernel<DT, K, ND, TK, FIN, E, (ND == 0 ? kShortRowFinishers : 1)>;
        if (enable_stream_smem<kernel>(env.device) != AASD_OK) return AASD_ERR_CUDA;
        launch_clustered(kernel, grid, stream_threads(kShortRowFinishers), kStreamSmemBytes, env.stream, cluster, sj, a);
        return AASD_OK;
    }
    constexpr auto kernel = stream_kernel<DT, K, ND, TK, FIN, E, 1>;
    if (enable_stream_smem<kernel>(env.device) != AASD_OK) return AASD_ERR_CUDA;
    launch_clustered(kernel, grid, stream_threads(1), kStreamSmemBytes, env.stream, cluster, sj, a);
    return AASD_OK;
}

// bytes of a row below which the finisher, not the copy, paces a CTA (measured: a verification
// row costs a finisher about 7 us under load, an alignment row 5 us; a CTA streams 25 GB/s)
constexpr int64_t kShortVerifyRow = 200 * 1024;
constexpr int64_t kShortAlignRow = 96 * 1024;
inline int64_t row_bytes_of(const StreamJob& sj) { return (int64_t)sj.row.stream_nvec * 16; }

// Launchers, one set per logits dtype, each in a translation unit of its own.  sj == nullptr:
// the plain-load kernels (one CTA, or job.chunks CTAs, per row: `grid` CTAs in all).
int launch_verify_f32(const LaunchEnv& env, const StreamJob* sj, const VerifyArgs& a, unsigned int grid);
int launch_verify_bf16(const LaunchEnv& env, const StreamJob* sj, const VerifyArgs& a, unsigned int grid);
int launch_align_topk_f32(const LaunchEnv& env, const StreamJob* sj, const AlignArgs& a, unsigned int grid);
int launch_align_topk_bf16(const LaunchEnv& env, const StreamJob* sj, const AlignArgs& a, unsigned int grid);
int launch_align_gumbel_f32(const LaunchEnv& env, const StreamJob& sj, const AlignArgs& a, unsigned int grid);
int launch_align_gumbel_bf16(const LaunchEnv& env, const StreamJob& sj, const AlignArgs& a, unsigned int grid);
int launch_tree_f32(const LaunchEnv& env, const StreamJob* sj, const TreeArgs& a, unsigned int grid);
int launch_tree_bf16(const LaunchEnv& env, const StreamJob* sj, const TreeArgs& a, unsigned int grid);

}  // namespace aasd
