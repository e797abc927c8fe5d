// Persistent, warp-specialised streaming of logits rows (sm_100a).
//
// One CTA per SM slot runs for the whole launch.  A producer warp moves 32 KB tiles of the
// rows from HBM into a ring of shared-memory stages with bulk asynchronous copies (TMA,
// cp.async.bulk, completion signalled on an mbarrier); eight consumer warps turn each tile
// into running sums and best-token candidates; a finisher warp (three of them, taking the
// items in turn, when rows are short) merges what the consumers leave per work item,
// combines the pieces of rows that were split over several CTAs and evaluates the row
// (entropy, probabilities, threshold test, accept scan).  The three roles only meet at
// mbarriers, so the copies of the next rows are in flight while the current row is being
// reduced and finished.
//
// Work is handed out dynamically: the producer claims the next work item from a counter in
// global memory, so a CTA that runs on a slower path to memory simply takes fewer items.
// An item is a whole row, or, when the host finds rows scarce, a piece of a row cut at tile
// boundaries (rows [0, whole_rows) are whole, later rows are cut).  The pieces of a row meet
// in the shared memory of a thread-block cluster's first CTA when the launch is made of one
// cluster per row, else in global memory, where the CTA that delivers the last one finishes
// the row.
//
// Every wait is bounded: a role that gives up raises AASD_STATUS_TIMEOUT, tells the other
// roles through a shared flag and leaves; the producer first waits (bounded again) for the
// copies it still has in flight.
#pragma once

#include "aasd_rows.cuh"

namespace aasd {

constexpr int kTileBytes = 32768;
constexpr int kStages = 3;
constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
// consumers + producer warp + NF finisher warps (item seq goes to finisher seq % NF)
constexpr int stream_threads(int nf) { return kConsumers + 32 + 32 * nf; }
constexpr int kShortRowFinishers = 3;
constexpr int kRing = 16;
constexpr int kSlots = 4;                         // item results in flight between consumers and finisher
constexpr unsigned int kWaitLimit = 1u << 24;     // polls of try_wait before giving up (StreamJob::wait_limit)

// ---- mbarrier / bulk copy primitives ---------------------------------------------------
__device__ __forceinline__ unsigned int smem_u32(const void* p) {
    return (unsigned int)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(u64* bar, unsigned int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(u64* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(u64* bar, unsigned int bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u64* bar, unsigned int parity) {
    unsigned int ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(u64* bar, unsigned int parity, volatile int* abort_flag, unsigned int limit) {
    for (unsigned int it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    return false;
}
// ---- thread-block clusters: the pieces of a row meet in the shared memory of the cluster's
// first CTA instead of global memory ------------------------------------------------------
__device__ __forceinline__ void cluster_sync_all() {
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Taken by every thread of a cluster launch on its way out: no CTA of the cluster leaves
// (and gives its shared memory back) while another one may still write into it, whatever
// path, a timed-out wait included, brought the threads here.
__device__ __forceinline__ void cluster_exit_sync() {
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ unsigned int cluster_map(const void* p, unsigned int rank) {
    unsigned int r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_store_u64(unsigned int addr, u64 v) {
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ void cluster_mbar_arrive(unsigned int addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(u64* bar, unsigned int parity) {
    unsigned int ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(u64* bar, unsigned int parity, volatile int* abort_flag,
                                                  unsigned int limit) {
    for (unsigned int it = 0; it < limit; ++it) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    return false;
}
__device__ __forceinline__ void give_up(volatile int* abort_flag, DeviceState* state) {
    *abort_flag = 1;
    atomicOr(&state->status, AASD_STATUS_TIMEOUT);
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, unsigned int bytes, u64* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ uint4 lds16(const void* p) {
    uint4 q;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w)
                 : "r"(smem_u32(p)));
    return q;
}

// ---- shared state of a streaming CTA -----------------------------------------------------
struct ItemInfo {
    float neg_refc;   // -(reference * c1) of the item's row
    int hint;         // hinted token of the row as given (may lie outside the vocabulary)
    float hint_logit; // its raw logit when it lies inside
    int row;          // logits row of the item; kNoItem: the work list is exhausted
    int chunk;        // which piece of the row
    int head;         // tokens of the row in front of its first 16-byte boundary (0 for aligned rows)
    int nvec;         // whole 16-byte vectors of the row from that boundary on
    int aux;          // a per-row word the epilogue wants fetched ahead of time (E::prefetch)
};
constexpr int kNoItem = -1;
constexpr int kMaxCluster = 8;   // portable cluster size
struct WarpPartial {
    double S, A;
    u64 key[kMaxK];   // vector-level: (ordered vector maximum << 32) | ~vector index
    long long ahead;  // top-k verification: tokens counted ahead of the draft token
};
struct StreamShared {
    u64 full[kStages];
    u64 empty[kStages];
    u64 done[kSlots];
    u64 freeb[kSlots];
    ItemInfo ring[kRing];
    WarpPartial wp[kSlots][kConsumerWarps];
    RaceSummary race[kSlots][kConsumerWarps][kMaxK];   // sampling kernels only
    unsigned short max_tile[kSlots][kConsumerWarps][32];   // tile (within the item) where a lane met its maximum
    int abort_flag;
    // cluster launches: the pieces of the cluster's row, written by the other CTAs of the
    // cluster into the first CTA's copy, and the barrier they arrive on
    RowPartial cluster_piece[kMaxCluster];
    u64 cluster_bar;
};
constexpr size_t kStreamSmemBytes = (size_t)kStages * kTileBytes + sizeof(StreamShared) + 128;

struct StreamJob {
    RowJob row;               // logits, geometry, scratch
    const int32_t* hint_ids;  // [n_rows] token whose logit seeds the row's reference
    unsigned int* sched;      // [2] next item, CTAs that have finished (both zero between launches)
    int tiles_per_row;
    int whole_rows;           // rows [0, whole_rows) are one item each
    int tail_chunks;          // every later row is cut into this many pieces
    long long n_items;        // whole_rows + (n_rows - whole_rows) * tail_chunks
    int cluster_pieces;       // the launch is made of clusters of tail_chunks CTAs, one per row, every
                              // row is cut (whole_rows == 0) and the grid has one CTA per piece
    unsigned int wait_limit;  // polls after which a wait inside the kernel gives up (kWaitLimit)
    // testing aid (aasd_debug_withhold_tile): the copy of this tile of this item is never issued
    long long withhold_item;  // -1: none
    int withhold_tile;
    // sampling kernels only
    SampleJob smp;
    RaceSummary* race_partials;   // [slots x kMaxK] beside the partial records of cut rows
    int full_groups;              // sampling groups that lie wholly inside the vector part of a row
};
constexpr int kRaceSlots = 1024;  // cut-row pieces a sampling launch may have

// Work item -> (row, piece); pieces of a row are balanced ranges of its tiles.  (Item, row and
// tile counts fit 32 bits - the host refuses launches beyond that - and 32-bit divisions are
// several times cheaper than 64-bit ones on a path every item walks.)
__device__ __forceinline__ void decode_item(const StreamJob& job, long long item, int& row, int& chunk) {
    if (item < job.whole_rows) {
        row = (int)item;
        chunk = 0;
    } else {
        const unsigned int j = (unsigned int)(item - job.whole_rows), c = (unsigned int)job.tail_chunks;
        row = job.whole_rows + (int)(j / c);
        chunk = (int)(j % c);
    }
}
__device__ __forceinline__ int chunks_of(const StreamJob& job, int row) {
    return row < job.whole_rows ? 1 : job.tail_chunks;
}
__device__ __forceinline__ int tiles_of(int nvec) { return (int)(((unsigned int)nvec + (kTileBytes / 16 - 1)) / (kTileBytes / 16)); }
// nvec: the row's own vector count (rows that do not start on a 16-byte boundary differ by one)
__device__ __forceinline__ void tile_range(const StreamJob& job, int row, int chunk, int nvec, int& tb, int& te) {
    const int tiles = tiles_of(nvec);
    if (row < job.whole_rows) {
        tb = 0;
        te = tiles;
    } else {
        // chunk < tail_chunks <= 32 and tiles < 2^20: the products stay far inside 32 bits
        const unsigned int c = (unsigned int)job.tail_chunks;
        tb = (int)(((unsigned int)chunk * (unsigned int)tiles) / c);
        te = (int)(((unsigned int)(chunk + 1) * (unsigned int)tiles) / c);
    }
}
// Where a row's vectors begin: rows are streamed from their first 16-byte boundary, the few
// tokens in front of it (none when the row is aligned) and behind the last whole vector are
// left to the finisher.
template <int DT>
__device__ __forceinline__ void row_vectors(const char* rowp, int vocab, int& head, int& nvec) {
    head = (int)(((16u - (unsigned int)((uintptr_t)rowp & 15u)) & 15u) / (unsigned int)Elt<DT>::kSize);
    head = head < vocab ? head : vocab;
    nvec = (vocab - head) / Elt<DT>::kVec;
}

__device__ __forceinline__ bool info_row_ok(unsigned int row, long long n_rows) { return (long long)row < n_rows; }

__device__ __forceinline__ u64 make_vec_key(float vmax, int vec) {
    return ((u64)ordered_bits(vmax) << 32) | (u64)(0xFFFFFFFFu - (unsigned int)vec);
}

// NaN-propagating lower clamp of the logits that feed the exponentials: a -inf entry (a
// masked token) becomes a huge negative finite number, so that its weight is exactly zero
// without 0 * inf, while NaN still reaches the sums and marks the row bad.  The candidates
// for the maximum are taken from the unclamped values.
template <int DT> struct Clamp;
template <> struct Clamp<AASD_F32> {
    static __device__ __forceinline__ unsigned int one(unsigned int w) {
        float r;
        const float lo = -1.0e30f;
        asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(__uint_as_float(w)), "f"(lo));
        return __float_as_uint(r);
    }
    static __device__ __forceinline__ uint4 apply(const uint4& q) {
        return make_uint4(one(q.x), one(q.y), one(q.z), one(q.w));
    }
    static __device__ __forceinline__ float vector_max(const uint4& q) {
        return fmaxf(fmaxf(__uint_as_float(q.x), __uint_as_float(q.y)),
                     fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
    }
};
template <> struct Clamp<AASD_BF16> {
    static constexpr unsigned int kLo2 = 0xF149F149u;   // bf16 pair (-1.0e30, -1.0e30)
    static __device__ __forceinline__ uint4 apply(const uint4& q) {
        uint4 r;
        asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r.x) : "r"(q.x), "r"(kLo2));
        asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r.y) : "r"(q.y), "r"(kLo2));
        asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r.z) : "r"(q.z), "r"(kLo2));
        asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r.w) : "r"(q.w), "r"(kLo2));
        return r;
    }
    static __device__ __forceinline__ float vector_max(const uint4& q) {
        unsigned int a, b, c;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(a) : "r"(q.x), "r"(q.y));
        asm("max.bf16x2 %0, %1, %2;" : "=r"(b) : "r"(q.z), "r"(q.w));
        asm("max.bf16x2 %0, %1, %2;" : "=r"(c) : "r"(a), "r"(b));
        return fmaxf(__uint_as_float(c << 16), __uint_as_float(c & 0xFFFF0000u));
    }
};

// Per-thread state of a consumer: packed fp32 sums and the K best vectors.
template <int DT, int K>
struct TileAccumulator {
    static constexpr int kVec = Elt<DT>::kVec;
    static constexpr int kAcc = kVec / 2;
    float2 S2[kAcc];
    float2 A2[kAcc];
    float best[K];
    int best_vec[K];

    __device__ __forceinline__ void init() {
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            S2[i] = make_float2(0.f, 0.f);
            A2[i] = make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < K; ++j) {
            best[j] = -CUDART_INF_F;
            best_vec[j] = -1;
        }
    }
    template <bool FIN>
    __device__ __forceinline__ void add(const uint4& raw, int vec_index, float c1, float neg_refc) {
        float x[kVec];
        Elt<DT>::unpack(FIN ? raw : Clamp<DT>::apply(raw), x);
        const float2 cc = make_float2(c1, c1);
        const float2 rr = make_float2(neg_refc, neg_refc);
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            float2 t = __ffma2_rn(make_float2(x[2 * i], x[2 * i + 1]), cc, rr);
            float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
            S2[i] = __fadd2_rn(S2[i], e);
            A2[i] = __ffma2_rn(e, t, A2[i]);
        }
        track(raw, vec_index);
    }
    // The vector joins the K best ones if its maximum says so.  ASCENDING: the thread meets its
    // vectors in ascending order, so a new one goes ahead of a kept one only if it is larger
    // ('>' keeps the lower id ahead among equals), and what a slot hands down was ranked above
    // everything below it and stays so whatever the values alone say (equal values: it is the
    // earlier one).  Otherwise (the sampling kernels read a tile's vectors in an order of their
    // own) value and index are compared at every slot.
    template <bool ASCENDING = true>
    __device__ __forceinline__ void track(const uint4& raw, int vec_index) {
        float vmax = Clamp<DT>::vector_max(raw);
        int vi = vec_index;
        bool up = false;
#pragma unroll
        for (int j = 0; j < K; ++j) {
            if (ASCENDING) up = up || vmax > best[j];
            else up = vmax > best[j] || (vmax == best[j] && vmax > -CUDART_INF_F && vi < best_vec[j]);
            const float hi = fmaxf(best[j], vmax);
            const float lo = fminf(best[j], vmax);
            const int hi_i = up ? vi : best_vec[j];
            const int lo_i = up ? best_vec[j] : vi;
            best[j] = hi;
            best_vec[j] = hi_i;
            vmax = lo;
            vi = lo_i;
        }
    }
};

// Kernels that need the best token only (K = 1, no sampling) do not track the vector in
// which a thread met its maximum: a thread keeps the maximum of each tile's logits (one
// packed max per word) and, once per tile, the running maximum with the tile that first
// reached it; the warp reports the maximum and which lanes hold it, and the finisher looks
// the first such vector up among the eight vectors that lane read in that tile.
template <int DT> struct RunMax;
template <> struct RunMax<AASD_BF16> {
    unsigned int m2;   // bf16x2
    __device__ __forceinline__ void init() { m2 = 0xFF80FF80u; }
    __device__ __forceinline__ void update(const uint4& q) {
        unsigned int a, b;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(a) : "r"(q.x), "r"(q.y));
        asm("max.bf16x2 %0, %1, %2;" : "=r"(b) : "r"(q.z), "r"(q.w));
        asm("max.bf16x2 %0, %1, %2;" : "=r"(a) : "r"(a), "r"(b));
        asm("max.bf16x2 %0, %1, %2;" : "=r"(m2) : "r"(m2), "r"(a));
    }
    __device__ __forceinline__ float value() const {
        return fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u));
    }
};
template <> struct RunMax<AASD_F32> {
    float m;
    __device__ __forceinline__ void init() { m = -CUDART_INF_F; }
    __device__ __forceinline__ void update(const uint4& q) {
        m = fmaxf(fmaxf(m, __uint_as_float(q.x)),
                  fmaxf(fmaxf(__uint_as_float(q.y), __uint_as_float(q.z)), __uint_as_float(q.w)));
    }
    __device__ __forceinline__ float value() const { return m; }
};

// The sums of one vector without any maximum tracking.
template <int DT, int K, bool FIN>
__device__ __forceinline__ void add_sums(TileAccumulator<DT, K>& acc, const uint4& raw, float c1, float neg_refc) {
    constexpr int kVec = Elt<DT>::kVec;
    float x[kVec];
    Elt<DT>::unpack(FIN ? raw : Clamp<DT>::apply(raw), x);
    const float2 cc = make_float2(c1, c1);
    const float2 rr = make_float2(neg_refc, neg_refc);
#pragma unroll
    for (int i = 0; i < kVec / 2; ++i) {
        float2 t = __ffma2_rn(make_float2(x[2 * i], x[2 * i + 1]), cc, rr);
        float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
        acc.S2[i] = __fadd2_rn(acc.S2[i], e);
        acc.A2[i] = __ffma2_rn(e, t, acc.A2[i]);
    }
}

// Where the finisher re-reads vectors of the item it finishes: the row in global memory, or,
// when the item's tiles are all still resident (launches of one item per CTA with no more
// tiles than ring stages), the shared-memory ring itself: tile t of the item sits in stage
// t - tb.
struct VectorSource {
    const char* vbase;              // the row's first vector in global memory
    const unsigned char* resident;  // the ring, or nullptr
    int tb;                         // first tile of the item
    __device__ __forceinline__ uint4 load(int v) const {
        constexpr int kTileVecs = kTileBytes / 16;
        if (resident) return lds16(resident + ((size_t)(v / kTileVecs - tb) * kTileVecs + (size_t)(v % kTileVecs)) * 16);
        return __ldg(reinterpret_cast<const uint4*>(vbase) + v);
    }
};

// First vector (lowest index) with maximum m among the vectors thread `tid` of the consumers
// read in tile t: vectors t * 2048 + k * 256 + tid, or, in sampling kernels (GROUPED), the eight
// neighbours t * 2048 + 8 * tid + k.  By a whole warp; -1 if none.
template <int DT, bool GROUPED>
__device__ int first_vector_in_tile(const VectorSource& src, int nvec, int t, int tid, float m) {
    constexpr int kTileVecs = kTileBytes / 16;
    constexpr int kPer = kTileVecs / kConsumers;
    const int lane = threadIdx.x & 31;
    const int step = GROUPED ? 1 : kConsumers, first = GROUPED ? kPer * tid : tid;
    const int v = t * kTileVecs + first + lane * step;
    bool hit = false;
    if (lane < kPer && v < nvec) hit = Clamp<DT>::vector_max(src.load(v)) == m;
    const unsigned int bal = __ballot_sync(0xFFFFFFFFu, hit);
    return bal ? t * kTileVecs + first + (__ffs(bal) - 1) * step : -1;
}
// The same over every vector of tiles [tb, te) (many lanes tie for the maximum).
template <int DT>
__device__ int first_vector_of_range(const VectorSource& src, int nvec, int tb, int te, float m) {
    constexpr int kTileVecs = kTileBytes / 16;
    const int lane = threadIdx.x & 31;
    const int end = min(te * kTileVecs, nvec);
    for (int base = tb * kTileVecs; base < end; base += 32) {
        const int v = base + lane;
        bool hit = false;
        if (v < end) hit = Clamp<DT>::vector_max(src.load(v)) == m;
        const unsigned int bal = __ballot_sync(0xFFFFFFFFu, hit);
        if (bal) return base + __ffs(bal) - 1;
    }
    return -1;
}

// Top-k verification (Sec. 3.3): counts, per thread, the tokens that are ahead of the row's
// draft token d in the order (logit descending, id ascending).  A token with a lower id is
// ahead when its logit is >= x_d, one with a higher id when it is > x_d; ">= x_d" is taken
// as "> the next value below x_d", so every vector needs one comparison per lane with a
// threshold chosen by its position relative to d's own vector.  The vector that holds d is
// compared with "> x_d" and the finisher adds its lower-id ties.
template <int DT> struct AheadCounter;
template <> struct AheadCounter<AASD_BF16> {
    unsigned int thr_gt, thr_ge;   // bf16x2: x_d twice, and the next bf16 below x_d twice
    unsigned int acc;              // bf16x2 running counts of the current tile (exact: <= 16 each)
    int vd;                        // vector index of d
    int count;
    __device__ __forceinline__ void begin_item(int d, float xd, bool valid, int head) {
        count = 0;
        acc = 0;
        vd = d < head ? -1 : (d - head) / 8;   // every vector lies behind a token of the row's head
        unsigned int b = __float_as_uint(xd) >> 16;
        unsigned int below = (b & 0x7FFFu) == 0 ? 0x8001u : ((b & 0x8000u) ? b + 1 : b - 1);
        if (!valid || !(xd > -CUDART_INF_F)) b = below = 0x7F80u;   // +inf: nothing is ahead
        thr_gt = b | (b << 16);
        thr_ge = (below & 0xFFFFu) | (below << 16);
    }
    __device__ __forceinline__ void add(const uint4& q, int vec) {
        const unsigned int thr = vec < vd ? thr_ge : thr_gt;
        unsigned int r;
        asm("set.gt.bf16x2.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(q.x), "r"(thr));
        asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(acc) : "r"(acc), "r"(r));
        asm("set.gt.bf16x2.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(q.y), "r"(thr));
        asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(acc) : "r"(acc), "r"(r));
        asm("set.gt.bf16x2.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(q.z), "r"(thr));
        asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(acc) : "r"(acc), "r"(r));
        asm("set.gt.bf16x2.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(q.w), "r"(thr));
        asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(acc) : "r"(acc), "r"(r));
    }
    // after at most 4 vectors (32 ids): move the packed counts to the integer counter
    __device__ __forceinline__ void end_tile() {
        count += (int)__uint_as_float(acc << 16) + (int)__uint_as_float(acc & 0xFFFF0000u);
        acc = 0;
    }
};
template <> struct AheadCounter<AASD_F32> {
    float thr_gt, thr_ge;
    float acc;
    int vd;
    int count;
    __device__ __forceinline__ void begin_item(int d, float xd, bool valid, int head) {
        count = 0;
        acc = 0.f;
        vd = d < head ? -1 : (d - head) / 4;
        const unsigned int b = __float_as_uint(xd);
        const unsigned int below = (b & 0x7FFFFFFFu) == 0 ? 0x80000001u : ((b & 0x80000000u) ? b + 1 : b - 1);
        thr_gt = xd;
        thr_ge = __uint_as_float(below);
        if (!valid || !(xd > -CUDART_INF_F)) thr_gt = thr_ge = CUDART_INF_F;
    }
    __device__ __forceinline__ void add(const uint4& q, int vec) {
        const float thr = vec < vd ? thr_ge : thr_gt;
        float r;
        asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(__uint_as_float(q.x)), "f"(thr));
        acc += r;
        asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(__uint_as_float(q.y)), "f"(thr));
        acc += r;
        asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(__uint_as_float(q.z)), "f"(thr));
        acc += r;
        asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(__uint_as_float(q.w)), "f"(thr));
        acc += r;
    }
    __device__ __forceinline__ void end_tile() {
        count += (int)acc;
        acc = 0.f;
    }
};

// The sums of one vector in a sampling kernel: the vector's weights are added to the running
// sum of the sampling group the vector belongs to, kept in two halves (`ga` takes the even
// pairs, `gb` the odd ones) so that consecutive additions do not wait for one another.  The
// caller adds a whole group's sum to S at once, and needs it for the group's ratio.
template <int DT, int K, bool FIN>
__device__ __forceinline__ void add_to_group(TileAccumulator<DT, K>& acc, const uint4& raw, float c1, float neg_refc,
                                             float2& ga, float2& gb) {
    constexpr int kVec = Elt<DT>::kVec;
    float x[kVec];
    Elt<DT>::unpack(FIN ? raw : Clamp<DT>::apply(raw), x);
    const float2 cc = make_float2(c1, c1);
    const float2 rr = make_float2(neg_refc, neg_refc);
#pragma unroll
    for (int i = 0; i < kVec / 2; ++i) {
        float2 t = __ffma2_rn(make_float2(x[2 * i], x[2 * i + 1]), cc, rr);
        float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
        if (i & 1) gb = __fadd2_rn(gb, e);
        else ga = __fadd2_rn(ga, e);
        acc.A2[i] = __ffma2_rn(e, t, acc.A2[i]);
    }
}

// exponent and weight of one raw logit exactly as the consumers form them
__device__ __forceinline__ void scalar_term(float x, float c1, float neg_refc, float& e, float& t) {
    float xc;
    const float lo = -1.0e30f;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(xc) : "f"(x), "f"(lo));
    t = fmaf(xc, c1, neg_refc);
    e = ex2_approx(t);
}

// Second, max-centred evaluation of a whole row by one warp: only for rows whose maximum
// lies so far above the provisional reference that the fp32 sums cannot be trusted.
template <int DT>
__device__ void warp_row_centered(const char* rowp, int V, float m, float c1, double& S, double& A) {
    const int lane = threadIdx.x & 31;
    double s = 0.0, a = 0.0;
    for (int i = lane; i < V; i += 32) {
        const float x = Elt<DT>::load(rowp, i);
        float t = (x - m) * c1;
        t = (t < -3.0e38f) ? -3.0e38f : t;   // NaN stays NaN
        const float e = ex2_approx(t);
        s += (double)e;
        a += (double)e * (double)t;
    }
    S = warp_sum_f64(s);
    A = warp_sum_f64(a);
}

// What the finisher hands to the kernel-specific epilogue.
struct FinishedRow {
    RowPartial merged;   // S, A and element-level keys (best tokens)
    float neg_refc;
    bool centered;
};

// Epilogue interface (static functions of a policy type E):
//   E::finish<ND>(args, job, row, rowp, FinishedRow&, ItemInfo&, races, tail_group, Tally&)
//   - entered by the whole finisher warp
//   E::State, E::drain(args, job, State&, Tally&)
//   - what an epilogue carries from one row to the next (verification looks at a row's ticket
//     one row late); drain is called once when the finisher warp has seen its last item
//   E::prefetch(args, row) -> int
//   - a per-row input of the epilogue, loaded by the producer together with the row's reference
//     and handed over in ItemInfo::aux, so that the finisher's serial path has no trip to
//     memory for it
//   ND: keyed draws per row the kernel prepares (0: no sampling)
//   TK: count the tokens ahead of the hinted token (top-k verification)
//   FIN: the logits are expected to hold no -inf: the clamp that makes masked tokens harmless
//        is skipped, and a row that holds one is re-evaluated by the finisher (its sums are NaN)
//   NF: finisher warps.  A row's serial path (look-ups, fp64 evaluation, fence and ticket)
//       takes 5-7 microseconds under load; rows that stream faster than that (below about
//       200 KB) get three finishers, at the price of 80 instead of 94 registers per thread,
//       which long rows, where one finisher is idle 40 % of the time, do not pay.
template <int DT, int K, int ND, bool TK, bool FIN, class E, int NF>
__global__ void __launch_bounds__(stream_threads(NF), 2) stream_kernel(const StreamJob job, const typename E::Args args) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* tiles = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    StreamShared& sh = *reinterpret_cast<StreamShared*>(tiles + (size_t)kStages * kTileBytes);
    constexpr int kVec = Elt<DT>::kVec;
    constexpr int kTileVecs = kTileBytes / 16;
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const RowJob& rj = job.row;
    const float c1 = rj.c1;
    volatile int* abort_flag = &sh.abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sh.full[s], 1);
            mbar_init(&sh.empty[s], kConsumerWarps);
        }
        for (int p = 0; p < kSlots; ++p) {
            mbar_init(&sh.done[p], kConsumerWarps);
            mbar_init(&sh.freeb[p], 1);
        }
        sh.abort_flag = 0;
        mbar_init(&sh.cluster_bar, job.cluster_pieces ? (unsigned int)job.tail_chunks - 1u : 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Where the producer's first item lies: launch constants only, so worked out on this side
    // of the wait for the preceding kernel (and again, for the next item, at the end of each
    // of the producer's iterations).
    int g_row = 0, g_chunk = 0, g_head = 0, g_nvec = 0, g_tb = 0, g_te = 0;
    const char* g_rowp = nullptr;
    auto locate = [&](long long item) {
        decode_item(job, item, g_row, g_chunk);
        g_rowp = row_pointer<DT>(rj, g_row);
        row_vectors<DT>(g_rowp, rj.vocab, g_head, g_nvec);
        tile_range(job, g_row, g_chunk, g_nvec, g_tb, g_te);
    };
    if (warp == kConsumerWarps) locate(blockIdx.x);
    // nobody may signal a barrier of another CTA before that CTA has set it up
    if (job.cluster_pieces) cluster_sync_all();
    pdl_launch_dependents();
    __syncthreads();
    pdl_wait();   // everything above overlapped the end of the preceding kernel

    if (warp < kConsumerWarps) {
        // ------------------------------------------------------------------ consumers
        unsigned int it = 0, seq = 0;
        for (;; ++seq) {
            TileAccumulator<DT, K> acc;
            acc.init();
            GroupRace<(ND > 0 ? ND : 1)> race;
            race.init();
            AheadCounter<DT> ahead;
            ahead.count = 0;
            constexpr bool kLazyMax = (K == 1);   // maximum by value, place found later
            RunMax<DT> tilemax;     // maximum of the current tile's logits
            float m_run = -CUDART_INF_F;   // maximum so far and the tile (within the item) that first reached it
            int m_tile = 0;
            unsigned int row_ctr = 0;
            float neg_refc = 0.f;
            bool alive = true, last = false;
            int tb = 0, te = 1, nvec = 0;
            for (int t = 0; t < te - tb; ++t, ++it) {
                const int s = it % kStages;
                if (!mbar_wait(&sh.full[s], (it / kStages) & 1u, abort_flag, job.wait_limit)) {
                    if (lane == 0) give_up(abort_flag, rj.state);
                    alive = false;
                    break;
                }
                if (t == 0) {
                    // the item's record was written before its first tile was announced
                    const ItemInfo info = sh.ring[seq % kRing];
                    if (info.row == kNoItem) {
                        last = true;
                        ++it;
                        break;
                    }
                    neg_refc = info.neg_refc;
                    row_ctr = (unsigned int)info.row;
                    if (TK) ahead.begin_item(info.hint, info.hint_logit, info.hint >= 0 && info.hint < rj.vocab, info.head);
                    nvec = info.nvec;
                    tile_range(job, info.row, info.chunk, nvec, tb, te);
                }
                const unsigned char* base = tiles + (size_t)s * kTileBytes;
                const int v0 = (tb + t) * kTileVecs;
                const int nv = min(kTileVecs, nvec - v0);
                // (checked build) the tile lies inside the ring and inside the row
                if (!AASD_IN_RANGE(s >= 0 && s < kStages && nv >= 1 && v0 >= 0 && v0 + nv <= nvec &&
                                   (long long)info_row_ok(row_ctr, rj.n_rows), rj.state)) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.empty[s]);   // the stage goes back unread
                    continue;
                }
                if (kLazyMax) tilemax.init();
                if (ND > 0) {
                    // A thread takes the eight neighbouring vectors 8 * tid .. 8 * tid + 7 of the
                    // tile: two sampling groups of bf16 ids (vectors 0-3 and 4-7), one group of
                    // fp32 ids.  So that a quarter-warp covers all shared-memory banks with every
                    // load, load k of a lane takes vector k ^ (lane & 7): bit 2 of the lane index
                    // swaps the two halves, its two low bits permute inside a half, and the
                    // address is one logic operation away from the thread's base; which half a
                    // register holds is known at compile time up to one swap at the end.
                    constexpr int kPer = kTileVecs / kConsumers;
                    constexpr int kVecsPerGroup = kGroup / kVec;           // 4 (bf16) or 8 (fp32)
                    constexpr int kGroupsPerThread = kPer / kVecsPerGroup; // 2 or 1
                    static_assert(kPer == 8 && kGroupsPerThread >= 1, "eight vectors per thread and tile");
                    const int hsel = (lane >> 2) & 1, l7 = lane & 7;
                    // the groups' random variates need their indices only: issued first, the
                    // generator's long dependent chain runs beside the exponentials below
                    const int g0 = (v0 + kPer * tid) * kVec / kGroup;
                    float inv_e[kGroupsPerThread][ND > 0 ? ND : 1];
#pragma unroll
                    for (int gi = 0; gi < kGroupsPerThread; ++gi)
                        GroupRace<(ND > 0 ? ND : 1)>::inverse_variates(g0 + gi, row_ctr, job.smp, inv_e[gi]);
                    uint4 q[kPer];
                    // running sums of the vectors read at k < 4 and at k >= 4, two halves each
                    float2 first = make_float2(0.f, 0.f), second = make_float2(0.f, 0.f);
                    float2 first_b = make_float2(0.f, 0.f), second_b = make_float2(0.f, 0.f);
                    if (nv == kTileVecs) {
#pragma unroll
                        for (int k = 0; k < kPer; ++k)
                            q[k] = lds16(base + (size_t)(kPer * tid + (k ^ l7)) * 16);
#pragma unroll
                        for (int k = 0; k < kPer; ++k) {
                            add_to_group<DT, K, FIN>(acc, q[k], c1, neg_refc, k < 4 ? first : second, k < 4 ? first_b : second_b);
                            if (kLazyMax) tilemax.update(q[k]);
                            else acc.template track<false>(q[k], v0 + kPer * tid + (k ^ l7));
                        }
                    } else {
                        bool ok[kPer];
#pragma unroll
                        for (int k = 0; k < kPer; ++k) {
                            const int v = kPer * tid + (k ^ l7);
                            ok[k] = v < nv;
                            if (ok[k]) q[k] = lds16(base + (size_t)v * 16);
                        }
#pragma unroll
                        for (int k = 0; k < kPer; ++k)
                            if (ok[k]) {
                                add_to_group<DT, K, FIN>(acc, q[k], c1, neg_refc, k < 4 ? first : second, k < 4 ? first_b : second_b);
                                if (kLazyMax) tilemax.update(q[k]);
                                else acc.template track<false>(q[k], v0 + kPer * tid + (k ^ l7));
                            }
                    }
                    first = __fadd2_rn(first, first_b);
                    second = __fadd2_rn(second, second_b);
                    float2 gs[kGroupsPerThread];
                    if (kGroupsPerThread == 2) {
                        gs[0] = hsel ? second : first;    // vectors 0-3 of the thread's share
                        gs[kGroupsPerThread - 1] = hsel ? first : second;
                    } else {
                        gs[0] = __fadd2_rn(first, second);
                    }
#pragma unroll
                    for (int gi = 0; gi < kGroupsPerThread; ++gi) {
                        acc.S2[0] = __fadd2_rn(acc.S2[0], gs[gi]);
                        race.take(gs[gi].x + gs[gi].y, inv_e[gi], g0 + gi, g0 + gi < job.full_groups);
                    }
                } else if (nv == kTileVecs) {
                    uint4 q[kTileVecs / kConsumers];
#pragma unroll
                    for (int k = 0; k < kTileVecs / kConsumers; ++k) q[k] = lds16(base + (size_t)(k * kConsumers + tid) * 16);
#pragma unroll
                    for (int k = 0; k < kTileVecs / kConsumers; ++k) {
                        if (kLazyMax) {
                            add_sums<DT, K, FIN>(acc, q[k], c1, neg_refc);
                            tilemax.update(q[k]);
                        } else {
                            acc.template add<FIN>(q[k], v0 + k * kConsumers + tid, c1, neg_refc);
                        }
                    }
                    if (TK) {
#pragma unroll
                        for (int k = 0; k < kTileVecs / kConsumers; ++k) ahead.add(q[k], v0 + k * kConsumers + tid);
                        ahead.end_tile();
                    }
                } else {
                    for (int v = tid; v < nv; v += kConsumers) {
                        const uint4 q = lds16(base + (size_t)v * 16);
                        if (kLazyMax) {
                            add_sums<DT, K, FIN>(acc, q, c1, neg_refc);
                            tilemax.update(q);
                        } else {
                            acc.template add<FIN>(q, v0 + v, c1, neg_refc);
                        }
                        if (TK) ahead.add(q, v0 + v);
                    }
                    if (TK) ahead.end_tile();
                }
                if (kLazyMax) {
                    const float mt = tilemax.value();
                    const bool up = mt > m_run;   // strict: the earliest tile stays among equals
                    m_tile = up ? t : m_tile;
                    m_run = up ? mt : m_run;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.empty[s]);
            }
            if (!alive) break;
            // warp-level result of the item
            double S = 0.0, A = 0.0;
#pragma unroll
            for (int i = 0; i < TileAccumulator<DT, K>::kAcc; ++i) {
                S += (double)acc.S2[i].x + (double)acc.S2[i].y;
                A += (double)acc.A2[i].x + (double)acc.A2[i].y;
            }
            S = warp_sum_f64(S);
            A = warp_sum_f64(A);
            u64 vk[K];
#pragma unroll
            for (int j = 0; j < K; ++j) vk[j] = acc.best_vec[j] >= 0 ? make_vec_key(acc.best[j], acc.best_vec[j]) : 0ull;
            u64 wk[K];
            if (kLazyMax) {
                // (warp maximum, lanes that hold it); nothing when every logit was -inf or NaN
                const float mt = m_run;
                const float mw = warp_max_f32(mt);
                const unsigned int holders = __ballot_sync(0xFFFFFFFFu, mt == mw);
                wk[0] = mw > -CUDART_INF_F ? (((u64)ordered_bits(mw) << 32) | (u64)holders) : 0ull;
            } else {
#pragma unroll
                for (int r = 0; r < K; ++r) {
                    const u64 m = warp_max_u64(vk[0]);
                    wk[r] = m;
                    if (m != 0 && vk[0] == m) {
#pragma unroll
                        for (int j = 0; j + 1 < K; ++j) vk[j] = vk[j + 1];
                        vk[K - 1] = 0;
                    }
                }
            }
            const int p = seq % kSlots;
            if (!mbar_wait(&sh.freeb[p], ((seq / kSlots) & 1u) ^ 1u, abort_flag, job.wait_limit)) {
                if (lane == 0) give_up(abort_flag, rj.state);
                break;
            }
            if (last) {
                // every finisher warp has to meet the end of the list: it stands in the records
                // of this and the next NF - 1 items
                bool ok = true;
                for (int j = 0; j < NF && ok; ++j) {
                    const unsigned int sq = seq + (unsigned int)j;
                    const int pj = sq % kSlots;
                    if (j > 0) ok = mbar_wait(&sh.freeb[pj], ((sq / kSlots) & 1u) ^ 1u, abort_flag, job.wait_limit);
                    if (ok && lane == 0) mbar_arrive(&sh.done[pj]);
                }
                if (!ok && lane == 0) give_up(abort_flag, rj.state);
                break;
            }
            if (ND > 0) {
#pragma unroll
                for (int j = 0; j < ND; ++j) {
                    u64 mine[kSampleKeep] = {race_key(race.best[j], race.best_g[j]), 0ull, 0ull};
                    u64 top[kSampleKeep];
                    warp_merge_keys<kSampleKeep>(mine, top);
                    const float runner = warp_max_f32(race.runner[j]);
                    if (lane == 0) {
                        RaceSummary& r = sh.race[p][warp][j];
#pragma unroll
                        for (int q = 0; q < kSampleKeep; ++q) r.key[q] = top[q];
                        r.runner = runner;
                    }
                }
            }
            int n_ahead = 0;
            if (TK) n_ahead = __reduce_add_sync(0xFFFFFFFFu, ahead.count);
            if (kLazyMax) {
                sh.max_tile[p][warp][lane] = (unsigned short)m_tile;
                __syncwarp();
            }
            if (lane == 0) {
                WarpPartial& w = sh.wp[p][warp];
                w.ahead = n_ahead;
                w.S = S;
                w.A = A;
#pragma unroll
                for (int j = 0; j < K; ++j) w.key[j] = wk[j];
                mbar_arrive(&sh.done[p]);
            }
        }
        if (job.cluster_pieces) cluster_exit_sync();
        return;
    }

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------- producer
        unsigned int it = 0, seq = 0;
        unsigned int armed = 0;   // bit s: a copy into stage s was issued in the current use
        bool alive = true;
        // The first item of a CTA is its own index (the grid never exceeds the item count);
        // later ones come from the counter, claimed one ahead so that its round trip is
        // hidden behind the copies of the current item.
        long long next = blockIdx.x;
        for (; alive; ++seq) {
            const long long item = next;
            if (item >= job.n_items) {
                // end of the work list: an empty stage use tells the consumers
                if (lane == 0) {
                    const int s = it % kStages;
                    if (mbar_wait(&sh.empty[s], ((it / kStages) & 1u) ^ 1u, abort_flag, job.wait_limit)) {
                        for (int j = 0; j < NF; ++j) sh.ring[(seq + j) % kRing].row = kNoItem;
                        mbar_arrive(&sh.full[s]);
                        // the last CTA to get here leaves the counters ready for the next launch
                        if (!job.cluster_pieces) {
                            __threadfence();
                            if (atomicAdd(job.sched + 1, 1u) == gridDim.x - 1) {
                                job.sched[0] = 0;
                                job.sched[1] = 0;
                            }
                        }
                    } else {
                        alive = false;
                    }
                }
                alive = __shfl_sync(0xFFFFFFFFu, alive ? 1 : 0, 0) != 0;
                break;
            }
            const int row = g_row, chunk = g_chunk, head = g_head, nvec = g_nvec, tb = g_tb, te = g_te;
            const char* rowp = g_rowp;
            const char* vbase = rowp + (size_t)head * Elt<DT>::kSize;
            // The item's first tile is sent off before anything else: the loads that give the
            // row's reference (two dependent trips to memory) then run while the copy is under
            // way.  The tile is announced (the producer's arrival on the stage's barrier, which
            // the phase needs whatever bytes have landed) only after the item's record is written.
            unsigned int first_bytes = 0;
            int first_stage = 0;
            if (lane == 0) {
                first_stage = it % kStages;
                if (!mbar_wait(&sh.empty[first_stage], ((it / kStages) & 1u) ^ 1u, abort_flag, job.wait_limit)) {
                    alive = false;
                } else if (!(item == job.withhold_item && job.withhold_tile == 0)) {   // (testing aid)
                    const long long off = (long long)tb * kTileBytes;
                    const long long left = (long long)nvec * 16 - off;
                    first_bytes = (unsigned int)(left < kTileBytes ? left : kTileBytes);
                    if (!AASD_IN_RANGE(row >= 0 && row < rj.n_rows && off >= 0 && left > 0 &&
                                       (long long)head * Elt<DT>::kSize + (long long)nvec * 16 <= (long long)rj.vocab * Elt<DT>::kSize &&
                                       ((uintptr_t)(vbase + off) & 15u) == 0 && (first_bytes & 15u) == 0, rj.state))
                        first_bytes = 0;
                    else
                    bulk_copy_g2s(tiles + (size_t)first_stage * kTileBytes, vbase + off, first_bytes, &sh.full[first_stage]);
                    armed |= 1u << first_stage;
                }
                // the next item: claimed one ahead, behind this item's first copy (launches of one
                // item per CTA have nothing to claim)
                next = job.cluster_pieces ? job.n_items : (long long)gridDim.x + (long long)atomicAdd(job.sched, 1u);
            }
            // reference of the row: its hinted logit and its first entries
            const int hint = __ldg(job.hint_ids + row);
            const bool hint_ok = hint >= 0 && hint < rj.vocab;
            float r = -CUDART_INF_F;
            if (lane < 4 && lane < rj.vocab) r = Elt<DT>::load(rowp, lane);
            if (lane == 4 && hint_ok) r = Elt<DT>::load(rowp, hint);
            int aux = 0;
            if (lane == 5) aux = E::prefetch(args, row);
            aux = __shfl_sync(0xFFFFFFFFu, aux, 5);
            const float hint_logit = __shfl_sync(0xFFFFFFFFu, r, 4);
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xFFFFFFFFu, r, o));
            r = __shfl_sync(0xFFFFFFFFu, r, 0);
            if (!(fabsf(r) <= 3.0e38f)) r = 0.f;
            if (lane == 0 && alive) {
                ItemInfo& info = sh.ring[seq % kRing];
                info.neg_refc = -(r * c1);
                info.hint = hint;
                info.hint_logit = hint_logit;
                info.row = row;
                info.chunk = chunk;
                info.head = head;
                info.nvec = nvec;
                info.aux = aux;
                if (first_bytes) mbar_arrive_expect_tx(&sh.full[first_stage], first_bytes);
                ++it;
                for (int t = tb + 1; t < te; ++t, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait(&sh.empty[s], ((it / kStages) & 1u) ^ 1u, abort_flag, job.wait_limit)) {
                        alive = false;
                        break;
                    }
                    if (item == job.withhold_item && t - tb == job.withhold_tile) continue;   // testing aid
                    const long long off = (long long)t * kTileBytes;
                    const long long left = (long long)nvec * 16 - off;
                    const unsigned int bytes = (unsigned int)(left < kTileBytes ? left : kTileBytes);
                    if (!AASD_IN_RANGE(off >= 0 && left > 0 && ((uintptr_t)(vbase + off) & 15u) == 0 && (bytes & 15u) == 0,
                                       rj.state))
                        continue;
                    mbar_arrive_expect_tx(&sh.full[s], bytes);
                    bulk_copy_g2s(tiles + (size_t)s * kTileBytes, vbase + off, bytes, &sh.full[s]);
                    armed |= 1u << s;
                }
            }
            alive = __shfl_sync(0xFFFFFFFFu, alive ? 1 : 0, 0) != 0;
            next = __shfl_sync(0xFFFFFFFFu, next, 0);
            if (next < job.n_items) locate(next);
        }
        if (!alive && lane == 0) {
            // give the copies still in flight a bounded time to land before the CTA leaves
            give_up(abort_flag, rj.state);
            for (int back = 1; back <= kStages && back <= (int)it; ++back) {
                const unsigned int j = it - back;
                const int s = j % kStages;
                if (armed & (1u << s)) {
                    for (unsigned int w = 0; w < job.wait_limit; ++w)
                        if (mbar_try_wait(&sh.full[s], (j / kStages) & 1u)) break;
                }
            }
        }
        if (job.cluster_pieces) cluster_exit_sync();
        return;
    }

    // ------------------------------------------------------------------------ finishers
    // the items go round the NF finisher warps
    Tally tally;   // lane 0's running counters, flushed when the warp leaves
    tally.clear();
    typename E::State estate;
    E::init(estate);
    for (unsigned int seq = (unsigned int)(warp - kConsumerWarps - 1);; seq += NF) {
        const int p = seq % kSlots;
        if (!mbar_wait(&sh.done[p], (seq / kSlots) & 1u, abort_flag, job.wait_limit)) {
            if (lane == 0) give_up(abort_flag, rj.state);
            break;
        }
        const ItemInfo info = sh.ring[seq % kRing];
        if (info.row == kNoItem) break;
        const long long row = info.row;
        const int chunk = info.chunk;
        const int chunks = chunks_of(job, info.row);
        const char* rowp = row_pointer<DT>(rj, row);
        const int head = info.head, nvec = info.nvec;            // the row's vectors: tokens head + 0 ...
        const char* vbase = rowp + (size_t)head * Elt<DT>::kSize;
        double S = 0.0, A = 0.0;
        u64 vk[K];
#pragma unroll
        for (int j = 0; j < K; ++j) vk[j] = 0;
        RaceSummary races[ND > 0 ? ND : 1];   // per draw, the same in every lane once merged
        long long n_ahead = 0;
        if (lane < kConsumerWarps) {
            const WarpPartial& w = sh.wp[p][lane];
            S = w.S;
            A = w.A;
            if (TK) n_ahead = w.ahead;
#pragma unroll
            for (int j = 0; j < K; ++j) vk[j] = w.key[j];
        }
        if (ND > 0) {
#pragma unroll
            for (int j = 0; j < ND; ++j) {
                u64 mine[kSampleKeep] = {0ull, 0ull, 0ull};
                float runner = -1.f;
                if (lane < kConsumerWarps) {
                    const RaceSummary& r = sh.race[p][lane][j];
#pragma unroll
                    for (int q = 0; q < kSampleKeep; ++q) mine[q] = r.key[q];
                    runner = r.runner;
                }
                warp_merge_keys<kSampleKeep>(mine, races[j].key);
                races[j].runner = warp_max_f32(runner);
            }
        }
        unsigned short my_tiles[kConsumerWarps];   // lane l: the tile of lane l of every consumer warp
        if (K == 1) {
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) my_tiles[w] = sh.max_tile[p][w][lane];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.freeb[p]);
        static_assert(kConsumerWarps == 8, "the eight warp partials sit in lanes 0-7");
        S = octet_sum_f64(S);
        A = octet_sum_f64(A);
        if (TK) n_ahead = warp_sum_i64(n_ahead);
        u64 mk[K];   // merged vector keys, identical in every lane
        // One item per CTA whose tiles all fit the ring (the small launches whose rows are cut
        // into one cluster each): the tiles are still in shared memory, so the finisher finds the
        // maximum's place there and hands on the best token itself instead of its vector: no
        // trip to global memory on its way.
        int item_tb, item_te;
        tile_range(job, info.row, info.chunk, nvec, item_tb, item_te);
        const bool resident = K == 1 && job.cluster_pieces && (tiles_of(nvec) + chunks - 1) / chunks <= kStages;
        const VectorSource vsrc{vbase, resident ? tiles : nullptr, item_tb};
        if (K == 1) {
            // the consumers reported (maximum, lanes holding it) per warp: find the first vector
            // of the item that attains the maximum
            const unsigned int top = (unsigned int)(vk[0] >> 32);
            const unsigned int best = __reduce_max_sync(0xFFFFFFFFu, top);
            mk[0] = 0;
            if (best != 0) {
                const float m = unordered_bits(best);
                const unsigned int mine = (lane < kConsumerWarps && top == best) ? (unsigned int)vk[0] : 0u;
                int n_holders = __reduce_add_sync(0xFFFFFFFFu, __popc(mine));
                const int tb = item_tb, te = item_te;
                int vfirst = 0x7FFFFFFF;
                if (n_holders <= 16) {
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        unsigned int lanes = __shfl_sync(0xFFFFFFFFu, mine, w);
                        while (lanes) {
                            const int l = __ffs(lanes) - 1;
                            lanes &= lanes - 1;
                            const int t = tb + (int)__shfl_sync(0xFFFFFFFFu, (unsigned int)my_tiles[w], l);
                            const int v = first_vector_in_tile<DT, (ND > 0)>(vsrc, nvec, t, w * 32 + l, m);
                            if (v >= 0 && v < vfirst) vfirst = v;
                        }
                    }
                } else {
                    const int v = first_vector_of_range<DT>(vsrc, nvec, tb, te, m);
                    if (v >= 0) vfirst = v;
                }
                if (vfirst != 0x7FFFFFFF) {
                    mk[0] = make_vec_key(m, vfirst);
                    if (resident) {
                        // the best token of that vector: the lowest id that holds the maximum
                        float x[kVec];
                        Elt<DT>::unpack(vsrc.load(vfirst), x);
                        int first_i = kVec - 1;
#pragma unroll
                        for (int i = kVec - 1; i >= 0; --i) first_i = (x[i] == m) ? i : first_i;
                        mk[0] = make_key(m, head + vfirst * kVec + first_i);
                    }
                }
            }
        } else {
#pragma unroll
            for (int r = 0; r < K; ++r) {
                const u64 m = warp_max_u64(vk[0]);
                mk[r] = m;
                if (m != 0 && vk[0] == m) {
#pragma unroll
                    for (int j = 0; j + 1 < K; ++j) vk[j] = vk[j + 1];
                    vk[K - 1] = 0;
                }
            }
        }
        if (chunks > 1 && job.cluster_pieces) {
            // The pieces of the row are the CTAs of this cluster (rank = piece): the others
            // write their records into the first CTA's shared memory and signal its barrier;
            // the first CTA waits for them and carries on.  No trip through global memory.
            if (chunk != 0) {
                if (lane == 0 && AASD_IN_RANGE(chunk > 0 && chunk < kMaxCluster, rj.state)) {
                    const unsigned int dst = cluster_map(&sh.cluster_piece[chunk], 0);
                    cluster_store_u64(dst + (unsigned int)offsetof(RowPartial, S), (u64)__double_as_longlong(S));
                    cluster_store_u64(dst + (unsigned int)offsetof(RowPartial, A), (u64)__double_as_longlong(A));
#pragma unroll
                    for (int j = 0; j < kMaxK; ++j)
                        cluster_store_u64(dst + (unsigned int)(offsetof(RowPartial, key) + 8 * j), j < K ? mk[j] : 0ull);
                    cluster_store_u64(dst + (unsigned int)offsetof(RowPartial, ahead), (u64)n_ahead);
                    cluster_mbar_arrive(cluster_map(&sh.cluster_bar, 0));
                }
                continue;
            }
            if (lane == 0) {
                RowPartial& mine = sh.cluster_piece[0];
                mine.S = S;
                mine.A = A;
#pragma unroll
                for (int j = 0; j < kMaxK; ++j) mine.key[j] = j < K ? mk[j] : 0ull;
                mine.ahead = n_ahead;
            }
            if (!mbar_wait_cluster(&sh.cluster_bar, 0u, abort_flag, job.wait_limit)) {
                if (lane == 0) give_up(abort_flag, rj.state);
                break;
            }
            __syncwarp();
            S = 0.0;
            A = 0.0;
            n_ahead = 0;
#pragma unroll
            for (int j = 0; j < K; ++j) vk[j] = 0;
            if (lane < chunks) {
                const RowPartial& q = sh.cluster_piece[lane];
                S = q.S;
                A = q.A;
                if (TK) n_ahead = q.ahead;
#pragma unroll
                for (int j = 0; j < K; ++j) key_insert<K>(vk, q.key[j]);
            }
            static_assert(kMaxCluster <= 8, "a cluster's pieces sit in lanes 0-7");
            S = octet_sum_f64(S);
            A = octet_sum_f64(A);
            if (TK) n_ahead = warp_sum_i64(n_ahead);
#pragma unroll
            for (int r = 0; r < K; ++r) {
                const u64 m = warp_max_u64(vk[0]);
                mk[r] = m;
                if (m != 0 && vk[0] == m) {
#pragma unroll
                    for (int j = 0; j + 1 < K; ++j) vk[j] = vk[j + 1];
                    vk[K - 1] = 0;
                }
            }
        } else if (chunks > 1) {
            // pieces of a row meet in global memory; the last one to arrive carries on
            RowPartial* slots = rj.partials + (row - job.whole_rows) * chunks;
            int last = 0;
            if (lane == 0 && AASD_IN_RANGE((row - job.whole_rows) * chunks + chunk >= 0 &&
                                           (row - job.whole_rows + 1) * chunks <= (ND > 0 ? kRaceSlots : kPartialSlots) &&
                                           row < rj.n_rows, rj.state)) {
                RowPartial mine;
                mine.S = S;
                mine.A = A;
#pragma unroll
                for (int j = 0; j < kMaxK; ++j) mine.key[j] = j < K ? mk[j] : 0ull;
                mine.ahead = n_ahead;
                slots[chunk] = mine;
                if (ND > 0) {
                    RaceSummary* rp = job.race_partials + ((row - job.whole_rows) * chunks + chunk) * kMaxK;
#pragma unroll
                    for (int j = 0; j < ND; ++j) rp[j] = races[j];
                }
                __threadfence();
                const unsigned int t = atomicAdd(&rj.row_tickets[row], 1u);
                last = (t == (unsigned int)chunks - 1);
                if (last) rj.row_tickets[row] = 0;
            }
            last = __shfl_sync(0xFFFFFFFFu, last, 0);
            if (!last) continue;
            __threadfence();
            S = 0.0;
            A = 0.0;
            n_ahead = 0;
#pragma unroll
            for (int j = 0; j < K; ++j) vk[j] = 0;
            for (int c = lane; c < chunks; c += 32) {
                const RowPartial* q = slots + c;
                S += __ldcg(&q->S);
                A += __ldcg(&q->A);
                if (TK) n_ahead += __ldcg(&q->ahead);
#pragma unroll
                for (int j = 0; j < K; ++j) key_insert<K>(vk, __ldcg(&q->key[j]));
            }
            S = warp_sum_f64(S);
            A = warp_sum_f64(A);
            if (TK) n_ahead = warp_sum_i64(n_ahead);
#pragma unroll
            for (int r = 0; r < K; ++r) {
                const u64 m = warp_max_u64(vk[0]);
                mk[r] = m;
                if (m != 0 && vk[0] == m) {
#pragma unroll
                    for (int j = 0; j + 1 < K; ++j) vk[j] = vk[j + 1];
                    vk[K - 1] = 0;
                }
            }
            if (ND > 0) {
#pragma unroll
                for (int j = 0; j < ND; ++j) {
                    u64 mine[kSampleKeep] = {0ull, 0ull, 0ull};
                    float runner = -1.f;
                    for (int c = lane; c < chunks; c += 32) {
                        const RaceSummary* rp = job.race_partials + ((row - job.whole_rows) * chunks + c) * kMaxK + j;
#pragma unroll
                        for (int q = 0; q < kSampleKeep; ++q) key_insert<kSampleKeep>(mine, __ldcg(&rp->key[q]));
                        runner = fmaxf(runner, __ldcg(&rp->runner));
                    }
                    warp_merge_keys<kSampleKeep>(mine, races[j].key);
                    races[j].runner = warp_max_f32(runner);
                }
            }
        }
        // Best tokens: they lie inside the K best vectors; plus the tokens outside the vectors
        // (in front of the row's first 16-byte boundary and behind its last whole vector: fewer
        // than two vectors' worth together).
        u64 ek[K];
#pragma unroll
        for (int j = 0; j < K; ++j) ek[j] = 0;
        float ts = 0.f, ta = 0.f;
        {
            u64 mine = 0;
#pragma unroll
            for (int j = 0; j < K; ++j)
                if (lane == j) mine = mk[j];
            if (resident) {
                if (lane == 0 && mine != 0) key_insert<K>(ek, mine);   // already the row's best token
            } else if (lane < K && mine != 0 && AASD_IN_RANGE(key_id(mine) >= 0 && key_id(mine) < nvec, rj.state)) {
                const int vec = key_id(mine);
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(vbase) + vec);
                float x[kVec];
                Elt<DT>::unpack(q, x);
#pragma unroll
                for (int i = 0; i < kVec; ++i)
                    if (x[i] > -CUDART_INF_F) key_insert<K>(ek, make_key(x[i], head + vec * kVec + i));
            }
            static_assert(kMaxK + 2 * (16 / 2 - 1) <= 32, "one lane per token outside the vectors");
            const int j = lane - K;
            const int i = j < head ? j : nvec * kVec + j;   // head tokens first, then the tail
            if (lane >= K && i < rj.vocab) {
                const float x = Elt<DT>::load(rowp, i);
                float e, t;
                scalar_term(x, c1, info.neg_refc, e, t);
                ts = e;
                ta = e * t;
                if (x > -CUDART_INF_F) key_insert<K>(ek, make_key(x, i));
            }
        }
        if (head > 0 || nvec * kVec < rj.vocab) {     // (no token outside the vectors: nothing to add)
            S += warp_sum_f64((double)ts);
            A += warp_sum_f64((double)ta);
        }
        FinishedRow fr;
#pragma unroll
        for (int r = 0; r < kMaxK; ++r) fr.merged.key[r] = 0;
#pragma unroll
        for (int r = 0; r < K; ++r) {
            const u64 m = warp_max_u64(ek[0]);
            fr.merged.key[r] = m;
            if (m != 0 && ek[0] == m) {
#pragma unroll
                for (int j = 0; j + 1 < K; ++j) ek[j] = ek[j + 1];
                ek[K - 1] = 0;
            }
        }
        fr.neg_refc = info.neg_refc;
        fr.centered = false;
        const u64 k0 = fr.merged.key[0];
        const float m = key_value(k0);
        if (k0 != 0 && fabsf(m) <= 3.0e38f) {
            const float shift = fmaf(m, c1, info.neg_refc);
            if (!(S > 0.0) || !(S <= 1.0e300) || !(fabs(A) <= 1.0e300) || !(fabsf(shift) <= kRedoShift)) {
                warp_row_centered<DT>(rowp, rj.vocab, m, c1, S, A);
                fr.neg_refc = -m;
                fr.centered = true;
                tally.redo += 1;
            }
        }
        fr.merged.S = S;
        fr.merged.A = A;
        fr.merged.ahead = 0;
        if (TK) {
            // what the consumers could not see: lower-id ties inside d's own vector, and the
            // ids of the ragged tail
            const int d = info.hint;
            long long extra = 0;
            if (d >= 0 && d < rj.vocab && info.hint_logit > -CUDART_INF_F) {
                const float xd = info.hint_logit;
                if (d >= head && d < head + nvec * kVec) {
                    const int i = head + (d - head) / kVec * kVec + lane;
                    if (lane < kVec && i < d && Elt<DT>::load(rowp, i) == xd) extra += 1;
                }
                // the tokens outside the vectors, one per lane
                const int i = lane < head ? lane : nvec * kVec + lane;
                if (i < rj.vocab) {
                    const float x = Elt<DT>::load(rowp, i);
                    extra += (x > xd || (x == xd && i < d)) ? 1 : 0;
                }
            }
            fr.merged.ahead = n_ahead + warp_sum_i64(extra);
        }
        // ids beyond the last complete group of the vector part were not raced (sampling
        // launches take aligned rows only: head == 0)
        const int tail_group = (ND > 0 && job.full_groups * kGroup < rj.vocab) ? job.full_groups : -1;
        E::template finish<ND>(args, rj, row, rowp, fr, info, races, tail_group, estate, tally);
    }
    E::drain(args, rj, estate, tally);
    if (lane == 0) tally.flush(rj.state);
    if (job.cluster_pieces) cluster_exit_sync();
}

// Epilogues are entered by the whole finisher warp.
template <int DT>
struct VerifyEpilogue {
    using Args = VerifyArgs;
    using State = PendingRow;
    static __device__ __forceinline__ void init(State& st) { st.valid = 0; }
    template <int ND>
    static __device__ void finish(const VerifyArgs& a, const RowJob& job, int64_t row, const char* rowp,
                                  const FinishedRow& fr, const ItemInfo& info, const RaceSummary* races, int tail_group,
                                  State& previous, Tally& tally) {
        int sampled = AASD_NONE;
        if (ND > 0 && !partial_bad(fr.merged))
            sampled = warp_sample_decide<DT>(rowp, job.vocab, (unsigned int)row, 0, a.smp, races[0], tail_group,
                                             fr.centered, tally.recheck, tally.exhaustive);
        // this row's evaluation and ticket first, then the previous row's ticket, which has had
        // a whole row's time to come back
        PendingRow mine;
        verify_row_warp<DT>(a, job, row, fr.merged, fr.neg_refc, fr.centered, info.hint, info.hint_logit,
                            (unsigned int)info.aux, sampled, mine, tally);
        if (previous.valid) verify_complete_warp(a, job, previous, tally);
        previous = mine;
    }
    static __device__ void drain(const VerifyArgs& a, const RowJob& job, State& previous, Tally& tally) {
        if (previous.valid) verify_complete_warp(a, job, previous, tally);
        previous.valid = 0;
    }
    // the row's flag byte
    static __device__ __forceinline__ int prefetch(const VerifyArgs& a, int64_t row) {
        return a.draft_flags ? (int)__ldg(a.draft_flags + row) : (int)AASD_FLAG_CONDITIONAL;
    }
};
template <int DT>
struct AlignEpilogue {
    using Args = AlignArgs;
    struct State {};
    static __device__ __forceinline__ void init(State&) {}
    static __device__ __forceinline__ void drain(const AlignArgs&, const RowJob&, State&, Tally&) {}
    template <int ND>
    static __device__ void finish(const AlignArgs& a, const RowJob& job, int64_t row, const char* rowp,
                                  const FinishedRow& fr, const ItemInfo& info, const RaceSummary* races, int tail_group,
                                  State&, Tally& tally) {
        // next_ids holds validated tokens only, so the hint is the row's next token
        int draws[kMaxK];
#pragma unroll
        for (int j = 0; j < kMaxK; ++j) draws[j] = AASD_NONE;
        if (ND > 0 && align_wants_draws(a, fr.merged, info.hint)) {
#pragma unroll
            for (int j = 0; j < ND; ++j)
                if (j < a.k_extra)
                    draws[j] = warp_sample_decide<DT>(rowp, job.vocab, (unsigned int)row, j, a.smp, races[j], tail_group,
                                                      fr.centered, tally.recheck, tally.exhaustive);
        }
        align_finish_warp<DT>(a, job, row, rowp, fr.merged, fr.neg_refc, fr.centered, info.hint, info.hint_logit, draws,
                              tally);
    }
    static __device__ __forceinline__ int prefetch(const AlignArgs&, int64_t) { return 0; }
};

}  // namespace aasd
