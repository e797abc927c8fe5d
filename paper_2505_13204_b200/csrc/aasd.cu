// Host side of the C ABI declared in include/aasd.h: argument checks, workspace layout,
// launch geometry.  Every step of the path runs in the kernels of aasd_rows.cuh and
// aasd_tokens.cuh; nothing here computes on the host.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>

// this translation unit holds the kernels that are not templates (see AASD_HOST_TU in the headers)
#define AASD_HOST_TU 1
#include "aasd_host.h"
#include "aasd_tokens.cuh"

using namespace aasd;

namespace {
// Named range around an entry point, visible to tools that collect NVTX (no cost without one).
struct TraceRange {
    explicit TraceRange(const char* name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
};

// Two environment switches for measurements and tests, read once per context:
// AASD_NO_CLUSTER=1 sends the pieces of cut rows through global memory instead of a cluster's
// shared memory, AASD_STREAM_CHUNKS=n sets the piece count of scarce rows.
struct Tuning {
    bool no_cluster;
    long stream_chunks;   // 0: the library's own choice
};
Tuning read_tuning() {
    Tuning t{};
    t.no_cluster = getenv("AASD_NO_CLUSTER") != nullptr;
    if (const char* e = getenv("AASD_STREAM_CHUNKS")) {
        const long v = atol(e);
        if (v >= 1) t.stream_chunks = v;
    }
    return t;
}
}  // namespace

struct aasd_ctx {
    int device;
    cudaStream_t stream;
    int sm_count;
    DeviceState* state;
    uint64_t launches;
    Tuning tuning;
    std::map<void*, WorkspaceLayout> workspaces;
    // testing aid, armed by aasd_debug_withhold_tile and used up by the next streaming launch
    long long withhold_item = -1;
    int withhold_tile = 0;
    unsigned int test_wait_limit = 0;
};

namespace {

int after_launch(aasd_ctx* ctx, int n) {
    ctx->launches += (uint64_t)n;
    return cudaGetLastError() == cudaSuccess ? AASD_OK : AASD_ERR_CUDA;
}

const WorkspaceLayout* find_workspace(aasd_ctx* ctx, void* ws, size_t bytes, int64_t rows, int64_t cands,
                                      int* err) {
    auto it = ctx->workspaces.find(ws);
    if (ws == nullptr || it == ctx->workspaces.end()) {
        *err = AASD_ERR_INVALID_ARG;
        return nullptr;
    }
    const WorkspaceLayout& L = it->second;
    if (bytes < L.bytes || rows > L.max_rows || cands > L.max_cands) {
        *err = AASD_ERR_WORKSPACE_TOO_SMALL;
        return nullptr;
    }
    return &L;
}

// Geometry of a streaming launch: how many CTAs share a row and which path the rows take.
int plan_rows(aasd_ctx* ctx, RowJob& job, const void* logits, int dtype, int vocab, int64_t row_stride,
              int64_t n_rows, float inv_temperature, char* ws, const WorkspaceLayout& L) {
    if (dtype != AASD_F32 && dtype != AASD_BF16) return AASD_ERR_BAD_DTYPE;
    if (vocab <= 0 || row_stride < vocab || n_rows < 0) return AASD_ERR_BAD_SHAPE;
    if (!(inv_temperature > 0.f) || !(inv_temperature <= 3.0e38f)) return AASD_ERR_INVALID_ARG;
    if (n_rows > 0 && logits == nullptr) return AASD_ERR_INVALID_ARG;
    const int esize = dtype == AASD_F32 ? 4 : 2;
    const int vec = 16 / esize;
    if (((uintptr_t)logits % esize) != 0) return AASD_ERR_INVALID_ARG;
    job.logits = logits;
    job.row_stride = row_stride;
    job.n_rows = n_rows;
    job.vocab = vocab;
    job.vector_ok = ((uintptr_t)logits % 16 == 0) && ((row_stride * esize) % 16 == 0);
    job.nvec = job.vector_ok ? vocab / vec : 0;
    // a row that starts anywhere has at most vec - 1 tokens in front of its first 16-byte boundary
    job.stream_nvec = job.vector_ok ? job.nvec : ((int64_t)vocab * esize >= 256 ? (vocab - (vec - 1)) / vec : 0);
    job.vec_elts = vec;
    job.c1 = inv_temperature * kLog2e;
    // Fill the machine: aim at eight CTAs per SM, but keep at least one sweep of the CTA
    // per chunk and stay within the partial-record slots of the workspace.
    int chunks = 1;
    if (n_rows > 0) {
        const int64_t target = (int64_t)ctx->sm_count * 8;
        const int64_t units = job.vector_ok ? job.nvec : vocab;
        int64_t c = target / n_rows;
        c = c < 1 ? 1 : c;
        c = c > kMaxSplit ? kMaxSplit : c;
        int64_t by_size = units / (2 * kThreads);
        c = c > by_size ? (by_size < 1 ? 1 : by_size) : c;
        while (c > 1 && c * n_rows > kPartialSlots) --c;
        chunks = (int)c;
    }
    job.chunks = chunks;
    int per = (job.nvec + chunks - 1) / chunks;
    per = (per + 7) / 8 * 8;
    job.vec_per_chunk = per;
    job.partials = reinterpret_cast<RowPartial*>(ws + L.off_partials);
    job.row_tickets = reinterpret_cast<unsigned int*>(ws + L.off_row_tickets);
    job.state = ctx->state;
    return AASD_OK;
}

// Which rows the persistent streaming kernel takes: 16-byte aligned layouts always; any other
// element-aligned layout too (every row is then streamed from its own first 16-byte boundary)
// unless the launch samples, since the sampler's groups of 32 ids are tied to the vectors.
bool stream_path(const RowJob& job, bool sampling) {
    return job.vector_ok ? job.nvec > 0 : (!sampling && job.stream_nvec > 0);
}

// Geometry of the persistent streaming launch: a grid of two CTAs
// per SM that claim work items from a counter.  An item is a whole row unless there are
// fewer rows than CTA slots; then every row is cut into pieces at tile boundaries.
void plan_stream(aasd_ctx* ctx, StreamJob& sj, const RowJob& job, const int32_t* hint_ids, char* ws,
                 const WorkspaceLayout& L, const SampleJob* smp, unsigned int* grid) {
    sj.row = job;
    sj.hint_ids = hint_ids;
    sj.sched = reinterpret_cast<unsigned int*>(ws + L.off_sched);
    sj.race_partials = reinterpret_cast<RaceSummary*>(ws + L.off_race);
    sj.full_groups = (int)(((int64_t)job.nvec * job.vec_elts) / kGroup);
    if (smp) sj.smp = *smp;
    // (rows that are not aligned may hold one vector more than this: a piece count that suits
    // the smaller figure suits them too)
    const int64_t row_bytes = (int64_t)job.stream_nvec * 16;
    const int tiles = (int)((row_bytes + kTileBytes - 1) / kTileBytes);
    const int64_t slots = (int64_t)ctx->sm_count * 2;
    // Cutting a row costs its pieces a trip through global memory (partial record, fence,
    // ticket) on the finisher's serial path; with many rows that measured slower than the
    // idle time it removes at the end of the launch (dynamic claiming already evens out
    // CTAs of different speed), so rows are cut only when they are scarce.
    int64_t tail_rows = 0, chunks = 1;
    if (job.n_rows < slots) {
        tail_rows = job.n_rows;
        chunks = slots / (2 * job.n_rows);
        if (chunks > 8) chunks = 8;
        if (ctx->tuning.stream_chunks >= 1) chunks = ctx->tuning.stream_chunks;   // tuning override
    }
    if (chunks > tiles) chunks = tiles;
    if (chunks <= 1) {
        chunks = 1;
        tail_rows = 0;
    }
    while (chunks > 1 && tail_rows * chunks > (smp ? kRaceSlots : kPartialSlots)) --chunks;
    if (chunks <= 1) {
        chunks = 1;
        tail_rows = 0;
    }
    sj.wait_limit = kWaitLimit;
    sj.withhold_item = -1;
    sj.withhold_tile = 0;
    if (ctx->withhold_item >= 0) {
        sj.wait_limit = ctx->test_wait_limit;
        sj.withhold_item = ctx->withhold_item;
        sj.withhold_tile = ctx->withhold_tile;
        ctx->withhold_item = -1;
        // one CTA per piece of a row would wait for the withheld piece at a cluster barrier
        // as well; the aid is about the waits of one CTA, so such a launch goes without clusters
    }
    sj.tiles_per_row = tiles;
    sj.whole_rows = (int)(job.n_rows - tail_rows);
    sj.tail_chunks = (int)chunks;
    sj.n_items = (job.n_rows - tail_rows) + tail_rows * chunks;
    *grid = (unsigned int)(sj.n_items < slots ? sj.n_items : slots);
    // Few rows, every row cut, one CTA per piece: the pieces of a row form a thread-block
    // cluster and meet in its first CTA's shared memory.  (The sampler's per-piece records
    // travel through global memory, so sampling launches stay as they are.)
    sj.cluster_pieces = (chunks > 1 && chunks <= kMaxCluster && tail_rows == job.n_rows && smp == nullptr &&
                         (int64_t)*grid == sj.n_items && sj.withhold_item < 0 && !ctx->tuning.no_cluster)
                            ? 1
                            : 0;
}

LaunchEnv env_of(const aasd_ctx* ctx) { return LaunchEnv{ctx->stream, ctx->device}; }

SampleJob make_sample_job(uint64_t seed, uint32_t step, bool align, float inv_temperature) {
    SampleJob s{};
    s.key0 = (unsigned int)(seed & 0xFFFFFFFFull);
    s.key1 = (unsigned int)(seed >> 32);
    s.step = step;
    s.dom_group = align ? kDomAlignGroup : kDomVerifyGroup;
    s.dom_elem = align ? kDomAlignElem : kDomVerifyElem;
    s.inv_t = inv_temperature;
    fill_round_keys(s);
    return s;
}

}  // namespace

extern "C" {

const char* aasd_status_str(int status) {
    switch (status) {
        case AASD_OK: return "ok";
        case AASD_ERR_INVALID_ARG: return "invalid argument";
        case AASD_ERR_BAD_SHAPE: return "bad shape";
        case AASD_ERR_BAD_DTYPE: return "bad dtype";
        case AASD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case AASD_ERR_CUDA: return "CUDA error";
        case AASD_ERR_NOT_SM100: return "device is not compute capability 10.x";
        case AASD_ERR_UNSUPPORTED: return "unsupported mode";
        default: return "unknown status";
    }
}

int aasd_create(aasd_ctx** out, int device, void* stream) {
    if (out == nullptr) return AASD_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return AASD_ERR_CUDA;
    cudaDeviceProp prop;
    AASD_CUDA(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return AASD_ERR_NOT_SM100;
    AASD_CUDA(cudaSetDevice(device));
    aasd_ctx* ctx = new (std::nothrow) aasd_ctx();
    if (ctx == nullptr) return AASD_ERR_CUDA;
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(stream);
    ctx->sm_count = prop.multiProcessorCount;
    ctx->launches = 0;
    ctx->tuning = read_tuning();
    if (cudaMalloc(&ctx->state, sizeof(DeviceState)) != cudaSuccess) {
        delete ctx;
        return AASD_ERR_CUDA;
    }
    if (cudaMemset(ctx->state, 0, sizeof(DeviceState)) != cudaSuccess) {
        cudaFree(ctx->state);
        delete ctx;
        return AASD_ERR_CUDA;
    }
    *out = ctx;
    return AASD_OK;
}

int aasd_destroy(aasd_ctx* ctx) {
    if (ctx == nullptr) return AASD_OK;
    cudaStreamSynchronize(ctx->stream);
    cudaFree(ctx->state);
    delete ctx;
    return AASD_OK;
}

int aasd_set_stream(aasd_ctx* ctx, void* stream) {
    if (ctx == nullptr) return AASD_ERR_INVALID_ARG;
    ctx->stream = static_cast<cudaStream_t>(stream);
    return AASD_OK;
}

int aasd_poll_status(aasd_ctx* ctx, uint32_t* bits) {
    if (ctx == nullptr || bits == nullptr) return AASD_ERR_INVALID_ARG;
    unsigned int v = 0;
    AASD_CUDA(cudaMemcpyAsync(&v, &ctx->state->status, 4, cudaMemcpyDeviceToHost, ctx->stream));
    AASD_CUDA(cudaMemsetAsync(&ctx->state->status, 0, 4, ctx->stream));
    AASD_CUDA(cudaStreamSynchronize(ctx->stream));
    *bits = v;
    return AASD_OK;
}

int aasd_get_counters(aasd_ctx* ctx, aasd_counters* out) {
    if (ctx == nullptr || out == nullptr) return AASD_ERR_INVALID_ARG;
    static_assert(sizeof(aasd_counters) == 64, "counter block layout");
    AASD_CUDA(cudaMemcpyAsync(out, ctx->state->counters, 64, cudaMemcpyDeviceToHost, ctx->stream));
    AASD_CUDA(cudaStreamSynchronize(ctx->stream));
    return AASD_OK;
}

int aasd_reset_counters(aasd_ctx* ctx) {
    if (ctx == nullptr) return AASD_ERR_INVALID_ARG;
    AASD_CUDA(cudaMemsetAsync(ctx->state->counters, 0, 64, ctx->stream));
    return AASD_OK;
}

uint64_t aasd_launch_count(const aasd_ctx* ctx) { return ctx ? ctx->launches : 0; }

int aasd_workspace_bytes(int64_t max_rows, int64_t max_cands, size_t* bytes) {
    if (bytes == nullptr || max_rows < 0 || max_cands < 0) return AASD_ERR_INVALID_ARG;
    *bytes = make_layout(max_rows, max_cands).bytes;
    return AASD_OK;
}

int aasd_workspace_init(aasd_ctx* ctx, void* workspace, size_t bytes, int64_t max_rows, int64_t max_cands) {
    if (ctx == nullptr || workspace == nullptr || max_rows < 0 || max_cands < 0) return AASD_ERR_INVALID_ARG;
    if ((uintptr_t)workspace % 256 != 0) return AASD_ERR_INVALID_ARG;
    WorkspaceLayout L = make_layout(max_rows, max_cands);
    if (bytes < L.bytes) return AASD_ERR_WORKSPACE_TOO_SMALL;
    AASD_CUDA(cudaMemsetAsync(workspace, 0, L.bytes, ctx->stream));
    ctx->workspaces[workspace] = L;
    return AASD_OK;
}

int aasd_workspace_release(aasd_ctx* ctx, void* workspace) {
    if (ctx == nullptr) return AASD_ERR_INVALID_ARG;
    ctx->workspaces.erase(workspace);
    return AASD_OK;
}

int aasd_align_sample(aasd_ctx* ctx, const void* prefill_logits, const int32_t* prompt_ids,
                      const int32_t* seq_offsets, int32_t n_seqs, int64_t n_rows,
                      const aasd_align_params* p, void* workspace, size_t workspace_bytes,
                      const aasd_align_out* out) {
    TraceRange trace("aasd_align_sample");
    if (ctx == nullptr || p == nullptr || out == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_seqs < 0 || n_rows < 0) return AASD_ERR_BAD_SHAPE;
    if (p->k_extra < 0 || p->k_extra > AASD_MAX_EXTRA) return AASD_ERR_INVALID_ARG;
    if (p->mode != AASD_ALIGN_TOPK && p->mode != AASD_ALIGN_GUMBEL) return AASD_ERR_INVALID_ARG;
    if (n_rows > 0 && (prompt_ids == nullptr || seq_offsets == nullptr || n_seqs == 0)) return AASD_ERR_INVALID_ARG;
    int err = AASD_OK;
    const WorkspaceLayout* L = find_workspace(ctx, workspace, workspace_bytes, n_rows, 0, &err);
    if (L == nullptr) return err;
    char* ws = static_cast<char*>(workspace);
    AlignArgs a{};
    err = plan_rows(ctx, a.job, prefill_logits, p->dtype, p->vocab, p->row_stride, n_rows, p->inv_temperature, ws, *L);
    if (err != AASD_OK) return err;
    if (n_rows == 0) return AASD_OK;
    if (n_rows * (int64_t)a.job.chunks > 0x7FFFFFFFLL) return AASD_ERR_BAD_SHAPE;
    a.prompt_ids = prompt_ids;
    a.seq_offsets = seq_offsets;
    a.n_seqs = n_seqs;
    a.k_extra = p->k_extra;
    a.mode = p->mode;
    a.hints = p->hints;
    a.next_ids = reinterpret_cast<int32_t*>(ws + L->off_next);
    a.smp = make_sample_job(p->seed, p->stream_tag, true, p->inv_temperature);
    a.out = *out;
    AASD_CUDA(cudaSetDevice(ctx->device));
    launch(align_next_kernel, (unsigned int)((n_rows + 255) / 256), 256, 0, ctx->stream, a);
    const bool f32 = p->dtype == AASD_F32;
    const bool draws = p->mode == AASD_ALIGN_GUMBEL && p->k_extra > 0;
    const LaunchEnv env = env_of(ctx);
    int rc = AASD_OK;
    if (stream_path(a.job, draws)) {
        // persistent TMA-fed streaming kernel
        StreamJob sj{};
        unsigned int grid = 0;
        plan_stream(ctx, sj, a.job, a.next_ids, ws, *L, draws ? &a.smp : nullptr, &grid);
        if (draws) rc = f32 ? launch_align_gumbel_f32(env, sj, a, grid) : launch_align_gumbel_bf16(env, sj, a, grid);
        else rc = f32 ? launch_align_topk_f32(env, &sj, a, grid) : launch_align_topk_bf16(env, &sj, a, grid);
    } else {
        const unsigned int grid = (unsigned int)(n_rows * a.job.chunks);
        rc = f32 ? launch_align_topk_f32(env, nullptr, a, grid) : launch_align_topk_bf16(env, nullptr, a, grid);
    }
    if (rc != AASD_OK) return rc;
    return after_launch(ctx, 2);
}

int aasd_draft(aasd_ctx* ctx, const aasd_draft_in* in, const aasd_draft_params* p, const aasd_draft_out* out) {
    TraceRange trace("aasd_draft");
    if (ctx == nullptr || in == nullptr || p == nullptr || out == nullptr) return AASD_ERR_INVALID_ARG;
    if (p->n_seqs < 0) return AASD_ERR_BAD_SHAPE;
    if (p->n < 1 || p->n > AASD_MAX_NGRAM || p->draft_len < 1 || p->max_cands < 1 || p->max_cands > kMaxCands)
        return AASD_ERR_INVALID_ARG;
    if (p->k_extra < 0 || p->k_extra > AASD_MAX_EXTRA) return AASD_ERR_INVALID_ARG;
    if (p->n_seqs == 0) return AASD_OK;
    if (!in->hist_ids || !in->hist_offsets || !in->hist_len || !in->prompt_len) return AASD_ERR_INVALID_ARG;
    if (in->recent_ids && !in->recent_len) return AASD_ERR_INVALID_ARG;
    if (in->align_ids && p->k_extra > 0 && (!in->align_n || !in->align_row_offsets)) return AASD_ERR_INVALID_ARG;
    if (in->pool_len < 0 || (in->pool_len > 0 && !in->pool_ids)) return AASD_ERR_INVALID_ARG;
    if (in->pool_align_ids && p->k_extra > 0 && !in->pool_align_n) return AASD_ERR_INVALID_ARG;
    if (!out->draft_ids || !out->draft_flags || !out->cand_len || !out->cand_pos || !out->n_cands || !out->match_len)
        return AASD_ERR_INVALID_ARG;
    DraftArgs a{*in, *p, *out, ctx->state};
    AASD_CUDA(cudaSetDevice(ctx->device));
    if (p->n_seqs > ctx->sm_count)
        launch(draft_kernel<kDraftThreadsBatch>, (unsigned int)p->n_seqs, (unsigned int)kDraftThreadsBatch, 0, ctx->stream, a);
    else
        launch(draft_kernel<kDraftThreads>, (unsigned int)p->n_seqs, (unsigned int)kDraftThreads, 0, ctx->stream, a);
    return after_launch(ctx, 1);
}

}  // extern "C"

namespace {

// aasd_verify, optionally followed inside the same launch by selection and append
// (`seq`, regular candidate layout only).
int verify_impl(aasd_ctx* ctx, const void* target_logits, const int32_t* draft_ids, const uint8_t* draft_flags,
                const int32_t* cand_offsets, int32_t n_cands, int64_t n_rows, const aasd_verify_params* p,
                void* workspace, size_t workspace_bytes, const aasd_verify_out* out, const SeqTail* seq) {
    if (ctx == nullptr || p == nullptr || out == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_cands < 0 || n_rows < 0) return AASD_ERR_BAD_SHAPE;
    if (p->mode < AASD_VERIFY_CONDITIONAL || p->mode > AASD_VERIFY_TOP_K) return AASD_ERR_INVALID_ARG;
    if (p->mode == AASD_VERIFY_TOP_K && p->top_k < 1) return AASD_ERR_INVALID_ARG;
    if (!(p->alpha >= 0.f) || !(p->beta >= 0.f)) return AASD_ERR_INVALID_ARG;
    if (cand_offsets == nullptr) {
        if (p->rows_per_cand < 1 || (int64_t)n_cands * p->rows_per_cand != n_rows) return AASD_ERR_BAD_SHAPE;
    }
    if (n_rows > 0 && (draft_ids == nullptr || n_cands == 0)) return AASD_ERR_INVALID_ARG;
    int err = AASD_OK;
    const WorkspaceLayout* L = find_workspace(ctx, workspace, workspace_bytes, n_rows, n_cands, &err);
    if (L == nullptr) return err;
    char* ws = static_cast<char*>(workspace);
    VerifyArgs a{};
    err = plan_rows(ctx, a.job, target_logits, p->dtype, p->vocab, p->row_stride, n_rows, p->inv_temperature, ws, *L);
    if (err != AASD_OK) return err;
    if (n_rows * (int64_t)a.job.chunks > 0x7FFFFFFFLL) return AASD_ERR_BAD_SHAPE;
    a.draft_ids = draft_ids;
    a.draft_flags = draft_flags;
    a.cand_offsets = cand_offsets;
    a.n_cands = n_cands;
    a.rows_per_cand = p->rows_per_cand;
    a.alpha = p->alpha;
    a.beta = p->beta;
    a.mode = p->mode;
    a.top_k = p->top_k;
    a.hints = p->hints;
    a.cand_tickets = reinterpret_cast<unsigned int*>(ws + L->off_cand_tickets);
    a.row_state = reinterpret_cast<u64*>(ws + L->off_row_own);
    a.smp = make_sample_job(p->seed, p->step, false, p->inv_temperature);
    a.out = *out;
    if (seq) {
        a.seq = *seq;
        a.seq.enabled = 1;
        a.seq.seq_tickets = reinterpret_cast<unsigned int*>(ws + L->off_seq_tickets);
        if (seq->table_ids) {
            if (!L->full) return AASD_ERR_UNSUPPORTED;
            a.row_extra = reinterpret_cast<int32_t*>(ws + L->off_row_extra);
        }
    }
    AASD_CUDA(cudaSetDevice(ctx->device));
    if (n_rows == 0) {
        if (n_cands == 0) return AASD_OK;
        launch(verify_empty_kernel, (unsigned int)((n_cands + 255) / 256), 256, 0, ctx->stream, a);
        return after_launch(ctx, 1);
    }
    const bool f32 = p->dtype == AASD_F32;
    const LaunchEnv env = env_of(ctx);
    int rc = AASD_OK;
    if (stream_path(a.job, p->mode == AASD_VERIFY_STRICT_SAMPLED)) {
        StreamJob sj{};
        unsigned int sgrid = 0;
        plan_stream(ctx, sj, a.job, draft_ids, ws, *L, p->mode == AASD_VERIFY_STRICT_SAMPLED ? &a.smp : nullptr, &sgrid);
        rc = f32 ? launch_verify_f32(env, &sj, a, sgrid) : launch_verify_bf16(env, &sj, a, sgrid);
    } else {
        const unsigned int grid = (unsigned int)(n_rows * a.job.chunks);
        rc = f32 ? launch_verify_f32(env, nullptr, a, grid) : launch_verify_bf16(env, nullptr, a, grid);
    }
    if (rc != AASD_OK) return rc;
    return after_launch(ctx, 1);
}

}  // namespace

extern "C" {

int aasd_verify(aasd_ctx* ctx, const void* target_logits, const int32_t* draft_ids,
                const uint8_t* draft_flags, const int32_t* cand_offsets, int32_t n_cands,
                int64_t n_rows, const aasd_verify_params* p, void* workspace, size_t workspace_bytes,
                const aasd_verify_out* out) {
    TraceRange trace("aasd_verify");
    return verify_impl(ctx, target_logits, draft_ids, draft_flags, cand_offsets, n_cands, n_rows, p, workspace,
                       workspace_bytes, out, nullptr);
}

int aasd_select(aasd_ctx* ctx, const int32_t* accept_len, const int32_t* next_token,
                const int32_t* draft_ids, const int32_t* cand_offsets, int32_t rows_per_cand,
                const int32_t* seq_cand_offsets, int32_t cands_per_seq, int32_t n_seqs,
                int32_t emit_stride, int32_t* best_cand, int32_t* n_emit, int32_t* emit_ids) {
    TraceRange trace("aasd_select");
    if (ctx == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_seqs < 0 || emit_stride < 1) return AASD_ERR_BAD_SHAPE;
    if (n_seqs == 0) return AASD_OK;
    if (!accept_len || !next_token || !draft_ids || !best_cand || !n_emit || !emit_ids) return AASD_ERR_INVALID_ARG;
    if (!cand_offsets && rows_per_cand < 1) return AASD_ERR_BAD_SHAPE;
    if (!seq_cand_offsets && cands_per_seq < 0) return AASD_ERR_BAD_SHAPE;
    SelectArgs a{accept_len, next_token, draft_ids, cand_offsets, rows_per_cand, seq_cand_offsets,
                 cands_per_seq, n_seqs, emit_stride, best_cand, n_emit, emit_ids};
    AASD_CUDA(cudaSetDevice(ctx->device));
    launch(select_kernel, (unsigned int)((n_seqs + 127) / 128), 128, 0, ctx->stream, a);
    return after_launch(ctx, 1);
}

int aasd_append(aasd_ctx* ctx, int32_t* hist_ids, const int32_t* hist_offsets, int32_t* hist_len,
                const int32_t* emit_ids, const int32_t* n_emit, int32_t n_seqs, int32_t emit_stride) {
    TraceRange trace("aasd_append");
    if (ctx == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_seqs < 0 || emit_stride < 1) return AASD_ERR_BAD_SHAPE;
    if (n_seqs == 0) return AASD_OK;
    if (!hist_ids || !hist_offsets || !hist_len || !emit_ids || !n_emit) return AASD_ERR_INVALID_ARG;
    AppendArgs a{hist_ids, hist_offsets, hist_len, emit_ids, n_emit, n_seqs, emit_stride, ctx->state};
    AASD_CUDA(cudaSetDevice(ctx->device));
    launch(append_kernel, (unsigned int)((n_seqs + 127) / 128), 128, 0, ctx->stream, a);
    return after_launch(ctx, 1);
}

int aasd_step(aasd_ctx* ctx, const aasd_step_args* s, void* workspace, size_t workspace_bytes) {
    TraceRange trace("aasd_step");
    if (ctx == nullptr || s == nullptr) return AASD_ERR_INVALID_ARG;
    const aasd_draft_params& dp = s->draft;
    if (!s->hist_ids || !s->hist_len || !s->best_cand || !s->n_emit || !s->emit_ids) return AASD_ERR_INVALID_ARG;
    if (!s->verify_out.accept_len || !s->verify_out.next_token) return AASD_ERR_INVALID_ARG;
    if (s->flags & AASD_STEP_EXTEND_TABLE) {
        if (!s->table_ids || !s->table_n || !s->draft_in.align_row_offsets) return AASD_ERR_INVALID_ARG;
        if (dp.k_extra < 1 || dp.k_extra > AASD_MAX_EXTRA) return AASD_ERR_INVALID_ARG;
    }
    int err = AASD_OK;
    if (!(s->flags & AASD_STEP_REUSE_DRAFT)) {
        err = aasd_draft(ctx, &s->draft_in, &dp, &s->draft_out);
        if (err != AASD_OK) return err;
    } else if (dp.n_seqs < 0 || dp.draft_len < 1 || dp.max_cands < 1 || !s->draft_out.draft_ids) {
        return AASD_ERR_INVALID_ARG;
    }
    aasd_verify_params vp = s->verify;
    vp.rows_per_cand = dp.draft_len;
    const int32_t n_cands = dp.n_seqs * dp.max_cands;
    const int64_t n_rows = (int64_t)n_cands * dp.draft_len;
    if (n_rows == 0) return AASD_OK;
    // selection and append ride on the verification launch: the warp that completes a
    // sequence's last candidate does both
    SeqTail tail{};
    tail.cands_per_seq = dp.max_cands;
    tail.rows_per_seq = dp.max_cands * dp.draft_len;
    tail.emit_stride = dp.draft_len + 1;
    tail.best_cand = s->best_cand;
    tail.n_emit = s->n_emit;
    tail.emit_ids = s->emit_ids;
    tail.hist_ids = s->hist_ids;
    tail.hist_offsets = s->draft_in.hist_offsets;
    tail.hist_len = s->hist_len;
    if (s->flags & AASD_STEP_EXTEND_TABLE) {
        tail.table_ids = s->table_ids;
        tail.table_n = s->table_n;
        tail.table_row_offsets = s->draft_in.align_row_offsets;
        tail.table_k = dp.k_extra;
    }
    return verify_impl(ctx, s->target_logits, s->draft_out.draft_ids, s->draft_out.draft_flags, nullptr, n_cands,
                       n_rows, &vp, workspace, workspace_bytes, &s->verify_out, &tail);
}

}  // extern "C"

extern "C" int aasd_debug_withhold_tile(aasd_ctx* ctx, int64_t item, int32_t tile, uint32_t wait_limit) {
    if (ctx == nullptr || item < 0 || tile < 0 || wait_limit < 1024u) return AASD_ERR_INVALID_ARG;
    ctx->withhold_item = item;
    ctx->withhold_tile = tile;
    ctx->test_wait_limit = wait_limit;
    return AASD_OK;
}

extern "C" int aasd_probe_read(aasd_ctx* ctx, const void* buffer, size_t bytes, uint32_t* sink) {
    if (ctx == nullptr || buffer == nullptr || sink == nullptr) return AASD_ERR_INVALID_ARG;
    if (((uintptr_t)buffer % 16) != 0 || (bytes % 16) != 0) return AASD_ERR_INVALID_ARG;
    if (bytes == 0) return AASD_OK;
    AASD_CUDA(cudaSetDevice(ctx->device));
    launch(probe_read_kernel, (unsigned int)(ctx->sm_count * 32), 256u, 0, ctx->stream,
           static_cast<const uint4*>(buffer), bytes / 16, sink);
    return after_launch(ctx, 1);
}

// ---- draft trees ----------------------------------------------------------------------------

extern "C" int aasd_tree_build(aasd_ctx* ctx, const int32_t* draft_ids, const uint8_t* draft_flags,
                               const int32_t* cand_len, const int32_t* n_cands, int32_t n_seqs, int32_t max_cands,
                               int32_t draft_len, int32_t* node_token, int32_t* node_parent, uint8_t* node_flags,
                               int32_t* node_depth, int32_t* n_nodes) {
    TraceRange trace("aasd_tree_build");
    if (ctx == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_seqs < 0 || max_cands < 1 || draft_len < 1) return AASD_ERR_BAD_SHAPE;
    if (n_seqs == 0) return AASD_OK;
    if (!draft_ids || !draft_flags || !cand_len || !n_cands || !node_token || !node_parent || !node_flags ||
        !node_depth || !n_nodes)
        return AASD_ERR_INVALID_ARG;
    const int64_t cap = 1 + (int64_t)max_cands * draft_len;
    const size_t smem = (size_t)cap * 2 * sizeof(int);
    if (smem > 48 * 1024) return AASD_ERR_UNSUPPORTED;
    TreeBuildArgs a{draft_ids, draft_flags, cand_len, n_cands, max_cands, draft_len, (int)cap,
                    node_token, node_parent, node_flags, node_depth, n_nodes};
    AASD_CUDA(cudaSetDevice(ctx->device));
    launch(tree_build_kernel, (unsigned int)n_seqs, 32u, smem, ctx->stream, a);
    return after_launch(ctx, 1);
}

extern "C" int aasd_verify_tree(aasd_ctx* ctx, const void* target_logits, const int32_t* node_token,
                                const int32_t* node_parent, const uint8_t* node_flags, const int32_t* tree_offsets,
                                int32_t n_trees, int64_t n_rows, const aasd_verify_params* p, int32_t emit_stride,
                                void* workspace, size_t workspace_bytes, const aasd_tree_out* out) {
    TraceRange trace("aasd_verify_tree");
    if (ctx == nullptr || p == nullptr || out == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_trees < 0 || n_rows < 0 || emit_stride < 1) return AASD_ERR_BAD_SHAPE;
    if (p->mode < AASD_VERIFY_CONDITIONAL || p->mode > AASD_VERIFY_TOP_K) return AASD_ERR_INVALID_ARG;
    if (p->mode == AASD_VERIFY_TOP_K && p->top_k < 1) return AASD_ERR_INVALID_ARG;
    if (!(p->alpha >= 0.f) || !(p->beta >= 0.f)) return AASD_ERR_INVALID_ARG;
    if (n_trees > 0 && tree_offsets == nullptr) return AASD_ERR_INVALID_ARG;
    if (n_rows > 0 && (node_token == nullptr || node_parent == nullptr || n_trees == 0)) return AASD_ERR_INVALID_ARG;
    if (!out->best_node || !out->n_accept || !out->n_emit || !out->emit_ids) return AASD_ERR_INVALID_ARG;
    int err = AASD_OK;
    const WorkspaceLayout* L = find_workspace(ctx, workspace, workspace_bytes, n_rows, n_trees, &err);
    if (L == nullptr) return err;
    char* ws = static_cast<char*>(workspace);
    TreeArgs a{};
    err = plan_rows(ctx, a.job, target_logits, p->dtype, p->vocab, p->row_stride, n_rows, p->inv_temperature, ws, *L);
    if (err != AASD_OK) return err;
    if (n_rows * (int64_t)a.job.chunks > 0x7FFFFFFFLL) return AASD_ERR_BAD_SHAPE;
    a.node_token = node_token;
    a.node_parent = node_parent;
    a.node_flags = node_flags;
    a.tree_offsets = tree_offsets;
    a.n_trees = n_trees;
    a.alpha = p->alpha;
    a.beta = p->beta;
    a.mode = p->mode;
    a.top_k = p->top_k;
    a.emit_stride = emit_stride;
    a.smp = make_sample_job(p->seed, p->step, false, p->inv_temperature);
    a.hint = reinterpret_cast<int32_t*>(ws + L->off_next);
    a.stats = reinterpret_cast<TreeRowStat*>(ws + L->off_tree_stats);
    a.tree_tickets = reinterpret_cast<unsigned int*>(ws + L->off_cand_tickets);
    a.node_ok = reinterpret_cast<uint8_t*>(ws + L->off_row_accept);
    a.out = *out;
    AASD_CUDA(cudaSetDevice(ctx->device));
    if (n_rows == 0) {
        if (n_trees == 0) return AASD_OK;
        launch(tree_empty_kernel, (unsigned int)((n_trees + 255) / 256), 256u, 0, ctx->stream, a);
        return after_launch(ctx, 1);
    }
    // rows without children keep the hint NONE (all bits set)
    AASD_CUDA(cudaMemsetAsync(a.hint, 0xFF, 4 * (size_t)n_rows, ctx->stream));
    launch(tree_hint_kernel, (unsigned int)((n_rows + 255) / 256), 256u, 0, ctx->stream, a);
    const bool f32 = p->dtype == AASD_F32;
    const LaunchEnv env = env_of(ctx);
    int rc = AASD_OK;
    if (stream_path(a.job, p->mode == AASD_VERIFY_STRICT_SAMPLED)) {
        StreamJob sj{};
        unsigned int grid = 0;
        plan_stream(ctx, sj, a.job, a.hint, ws, *L, p->mode == AASD_VERIFY_STRICT_SAMPLED ? &a.smp : nullptr, &grid);
        rc = f32 ? launch_tree_f32(env, &sj, a, grid) : launch_tree_bf16(env, &sj, a, grid);
    } else {
        const unsigned int grid = (unsigned int)(n_rows * a.job.chunks);
        rc = f32 ? launch_tree_f32(env, nullptr, a, grid) : launch_tree_bf16(env, nullptr, a, grid);
    }
    if (rc != AASD_OK) return rc;
    return after_launch(ctx, 2);
}

// ---- verification without any allocation ---------------------------------------------------
//
// Scratch of aasd_verify_static: one block per GPU that loads the library, held until the
// process exits.  Layout = the workspace layout for kStaticMaxRows rows and kStaticMaxCands
// candidates, followed by the status word and counters that a context would own.
namespace {

constexpr int64_t kStaticMaxRows = AASD_STATIC_MAX_ROWS;
constexpr int64_t kStaticMaxCands = AASD_STATIC_MAX_CANDS;
// the same function that lays a caller's workspace out sizes the block, at compile time
constexpr size_t kStaticWorkspaceBytes = make_layout(kStaticMaxRows, kStaticMaxCands, false).bytes;
constexpr size_t kStaticBytes = kStaticWorkspaceBytes + 256;

}  // namespace

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

namespace {

constexpr int kStaticMaxDevices = 64;
struct StaticSlot {
    bool ready;
    int sm_count;
    char* scratch;   // device address of g_static_scratch on this device
    Tuning tuning;
};
StaticSlot g_static_slots[kStaticMaxDevices];
std::mutex g_static_mutex;

}  // namespace

extern "C" int aasd_verify_static(int device, void* stream, const void* target_logits,
                                  const int32_t* draft_ids, const uint8_t* draft_flags,
                                  const int32_t* cand_offsets, int32_t n_cands, int64_t n_rows,
                                  const aasd_verify_params* p, const aasd_verify_out* out,
                                  uint32_t* status_bits) {
    if (p == nullptr || out == nullptr) return AASD_ERR_INVALID_ARG;
    if (device < 0 || device >= kStaticMaxDevices) return AASD_ERR_INVALID_ARG;
    if (n_cands < 0 || n_rows < 0) return AASD_ERR_BAD_SHAPE;
    if (n_rows > kStaticMaxRows || n_cands > kStaticMaxCands) return AASD_ERR_WORKSPACE_TOO_SMALL;
    if (p->mode < AASD_VERIFY_CONDITIONAL || p->mode > AASD_VERIFY_TOP_K) return AASD_ERR_INVALID_ARG;
    if (p->mode == AASD_VERIFY_TOP_K && p->top_k < 1) return AASD_ERR_INVALID_ARG;
    if (!(p->alpha >= 0.f) || !(p->beta >= 0.f)) return AASD_ERR_INVALID_ARG;
    if (cand_offsets == nullptr) {
        if (p->rows_per_cand < 1 || (int64_t)n_cands * p->rows_per_cand != n_rows) return AASD_ERR_BAD_SHAPE;
    }
    if (n_rows > 0 && (draft_ids == nullptr || n_cands == 0)) return AASD_ERR_INVALID_ARG;
    constexpr WorkspaceLayout L = make_layout(kStaticMaxRows, kStaticMaxCands, false);
    static_assert(L.bytes == kStaticWorkspaceBytes && L.bytes % 256 == 0, "the block holds exactly this layout");

    std::lock_guard<std::mutex> guard(g_static_mutex);
    AASD_CUDA(cudaSetDevice(device));
    StaticSlot& slot = g_static_slots[device];
    if (!slot.ready) {
        // Set-up, once per device and with that device current.  In host code the array's
        // name is only a handle: the address a kernel can use comes from the runtime.
        int major = 0, sms = 0;
        AASD_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        if (major != 10) return AASD_ERR_NOT_SM100;
        AASD_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return AASD_ERR_CUDA;
        slot.scratch = static_cast<char*>(ptr);
        slot.sm_count = sms;
        slot.tuning = read_tuning();
        slot.ready = true;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = slot.scratch;
    DeviceState* state = reinterpret_cast<DeviceState*>(ws + kStaticWorkspaceBytes);
    // The block keeps what the last call left: the tickets, the work-item counters and the status
    // word must start at zero even if that call was cut short.
    AASD_CUDA(cudaMemsetAsync(ws + L.off_row_tickets, 0, L.off_row_accept - L.off_row_tickets, s));
    AASD_CUDA(cudaMemsetAsync(state, 0, sizeof(DeviceState), s));

    aasd_ctx local{};   // launch geometry only: nothing of it outlives the call
    local.device = device;
    local.stream = s;
    local.sm_count = slot.sm_count;
    local.state = state;
    local.tuning = slot.tuning;
    VerifyArgs a{};
    int err = plan_rows(&local, a.job, target_logits, p->dtype, p->vocab, p->row_stride, n_rows, p->inv_temperature,
                        ws, L);
    if (err != AASD_OK) return err;
    if (n_rows * (int64_t)a.job.chunks > 0x7FFFFFFFLL) return AASD_ERR_BAD_SHAPE;
    a.draft_ids = draft_ids;
    a.draft_flags = draft_flags;
    a.cand_offsets = cand_offsets;
    a.n_cands = n_cands;
    a.rows_per_cand = p->rows_per_cand;
    a.alpha = p->alpha;
    a.beta = p->beta;
    a.mode = p->mode;
    a.top_k = p->top_k;
    a.hints = p->hints;
    a.cand_tickets = reinterpret_cast<unsigned int*>(ws + L.off_cand_tickets);
    a.row_state = reinterpret_cast<u64*>(ws + L.off_row_own);
    a.smp = make_sample_job(p->seed, p->step, false, p->inv_temperature);
    a.out = *out;
    if (n_rows == 0) {
        if (n_cands > 0) launch(verify_empty_kernel, (unsigned int)((n_cands + 255) / 256), 256, 0, s, a);
    } else if (stream_path(a.job, p->mode == AASD_VERIFY_STRICT_SAMPLED)) {
        StreamJob sj{};
        unsigned int sgrid = 0;
        plan_stream(&local, sj, a.job, draft_ids, ws, L, p->mode == AASD_VERIFY_STRICT_SAMPLED ? &a.smp : nullptr, &sgrid);
        const int rc = p->dtype == AASD_F32 ? launch_verify_f32(env_of(&local), &sj, a, sgrid)
                                            : launch_verify_bf16(env_of(&local), &sj, a, sgrid);
        if (rc != AASD_OK) return rc;
    } else {
        const unsigned int grid = (unsigned int)(n_rows * a.job.chunks);
        const int rc = p->dtype == AASD_F32 ? launch_verify_f32(env_of(&local), nullptr, a, grid)
                                            : launch_verify_bf16(env_of(&local), nullptr, a, grid);
        if (rc != AASD_OK) return rc;
    }
    if (cudaGetLastError() != cudaSuccess) return AASD_ERR_CUDA;
    if (status_bits != nullptr)
        AASD_CUDA(cudaMemcpyAsync(status_bits, &state->status, 4, cudaMemcpyDeviceToDevice, s));
    return AASD_OK;
}
