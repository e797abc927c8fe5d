// Draft trees (Eq. 2, Sec. 3.2) and their verification (Sec. 3.3).
//
// A tree is a range of nodes; node 0 of a tree is its root (the last token of the current
// sequence, no draft token), every other node carries a draft token and the index of its
// parent inside the tree, and parents precede their children.  Row v of the logits is the
// target distribution that follows node v, so the token of node v is judged with the
// statistics of its parent's row.  Verification therefore runs in two phases inside one
// launch: every row is reduced to its statistics by the streaming pass, and the warp that
// delivers the last row of a tree evaluates the tree's nodes, applies the prefix rule along
// the paths and emits the deepest passing path.
#pragma once

#include "aasd_stream.cuh"

namespace aasd {

// ---- building the tree from the flat candidates -----------------------------------------

struct TreeBuildArgs {
    const int32_t* draft_ids;     // [n_seqs x max_cands x draft_len]
    const uint8_t* draft_flags;   // same shape
    const int32_t* cand_len;      // [n_seqs x max_cands]
    const int32_t* n_cands;       // [n_seqs]
    int max_cands, draft_len;
    int cap;                      // node slots per tree: 1 + max_cands * draft_len
    int32_t* node_token;          // [n_seqs x cap]
    int32_t* node_parent;
    uint8_t* node_flags;
    int32_t* node_depth;
    int32_t* n_nodes;             // [n_seqs]
};

#ifdef AASD_HOST_TU   // not a template: compiled in the host translation unit only
// One warp per sequence.  The candidates are walked in order; at each depth the warp looks
// for the child that carries the same token (lowest node index, found with a ballot over
// the nodes made so far, which live in shared memory) or appends a new node.
__global__ void __launch_bounds__(32) tree_build_kernel(const TreeBuildArgs a) {
    extern __shared__ int s_nodes[];   // token[cap], parent[cap]
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    const int cap = a.cap;
    int* s_tok = s_nodes;
    int* s_par = s_nodes + cap;
    int32_t* tok = a.node_token + (int64_t)b * cap;
    int32_t* par = a.node_parent + (int64_t)b * cap;
    uint8_t* fl = a.node_flags + (int64_t)b * cap;
    int32_t* dep = a.node_depth + (int64_t)b * cap;
    for (int v = lane; v < cap; v += 32) {
        tok[v] = AASD_NONE;
        par[v] = AASD_NONE;
        fl[v] = 0;
        dep[v] = 0;
    }
    if (lane == 0) {
        s_tok[0] = AASD_NONE;
        s_par[0] = AASD_NONE;
    }
    __syncwarp();
    int n = 1;
    const int nc = min(a.n_cands[b], a.max_cands);
    for (int c = 0; c < nc; ++c) {
        const int32_t* d = a.draft_ids + ((int64_t)b * a.max_cands + c) * a.draft_len;
        const uint8_t* f = a.draft_flags + ((int64_t)b * a.max_cands + c) * a.draft_len;
        const int L = min(a.cand_len[(int64_t)b * a.max_cands + c], a.draft_len);
        int u = 0, depth = 0;
        for (int i = 0; i < L; ++i) {
            const int t = d[i];
            if (t == AASD_NONE) break;
            int child = AASD_NONE;
            for (int base = 1; base < n && child == AASD_NONE; base += 32) {
                const int v = base + lane;
                const bool hit = v < n && s_par[v] == u && s_tok[v] == t;
                const unsigned int bal = __ballot_sync(0xFFFFFFFFu, hit);
                if (bal) child = base + __ffs(bal) - 1;
            }
            ++depth;
            if (child == AASD_NONE) {
                child = n++;
                if (lane == 0) {
                    s_tok[child] = t;
                    s_par[child] = u;
                    tok[child] = t;
                    par[child] = u;
                    dep[child] = depth;
                    fl[child] = f[i];
                }
            } else if (lane == 0) {
                fl[child] |= f[i];
            }
            __syncwarp();
            u = child;
        }
    }
    if (lane == 0) a.n_nodes[b] = n;
}
#endif

// ---- verification ----------------------------------------------------------------------------

// What phase two needs to know about a row.
struct TreeRowStat {
    double S, H, pmax;
    float neg_refc, m;
    int own;     // the target's own token of the row (argmax or keyed draw), NONE on a bad row
    int flags;   // bit 0: bad row, bit 1: sums are max-centred
    int ahead;   // top-k mode: tokens ahead of the row's hinted token (its first child's), -1: not counted
    int pad;
};

struct TreeArgs {
    RowJob job;
    const int32_t* node_token;
    const int32_t* node_parent;
    const uint8_t* node_flags;    // NULL: every node conditional-eligible
    const int32_t* tree_offsets;  // [n_trees + 1]
    int n_trees;
    float alpha, beta;
    int mode;
    int top_k;                    // TOP_K mode
    int emit_stride;
    SampleJob smp;
    int32_t* hint;                // scratch [n_rows]: token of each row's first child
    TreeRowStat* stats;           // scratch [n_rows]
    unsigned int* tree_tickets;   // scratch [n_trees]
    uint8_t* node_ok;             // scratch [n_rows]: the node's own accept bit
    aasd_tree_out out;
};

#ifdef AASD_HOST_TU   // not a template: compiled in the host translation unit only
// hint[row of parent] = token of the parent's first child (rows without children keep NONE,
// set by the host).  Also checks the shape: a parent precedes its child.
__global__ void tree_hint_kernel(const TreeArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= a.job.n_rows) return;
    const int t = find_segment(a.tree_offsets, a.n_trees, g);
    const int64_t lo = a.tree_offsets[t];
    const int v = (int)(g - lo);
    if (v == 0) return;
    const int p = a.node_parent[g];
    if (p < 0 || p >= v) {
        atomicOr(&a.job.state->status, AASD_STATUS_BAD_OFFSETS);
        return;
    }
    for (int u = p + 1; u < v; ++u)
        if (a.node_parent[lo + u] == p) return;   // an earlier sibling is the first child
    const int tok = a.node_token[g];
    if (tok >= 0 && tok < a.job.vocab) a.hint[lo + p] = tok;
}
#endif

// Results of trees without nodes (between the offsets of their neighbours).
__device__ inline void write_empty_tree(const TreeArgs& a, int t) {
    if (a.out.best_node) a.out.best_node[t] = AASD_NONE;
    if (a.out.n_accept) a.out.n_accept[t] = 0;
    if (a.out.n_emit) a.out.n_emit[t] = 0;
    if (a.out.emit_ids)
        for (int i = 0; i < a.emit_stride; ++i) a.out.emit_ids[(int64_t)t * a.emit_stride + i] = AASD_NONE;
}
#ifdef AASD_HOST_TU   // not a template: compiled in the host translation unit only
__global__ void tree_empty_kernel(const TreeArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < a.n_trees) write_empty_tree(a, t);
}
#endif

// Row epilogue, entered by a whole warp.  Phase one (lane 0): the row's statistics.  Phase
// two (the warp that completes the tree): nodes, paths, result.
// Tokens of a row that are ahead of token d (raw logit xd) in the order (logit descending, id
// ascending), counted by a whole warp going over the row: the slow, exact way.
template <int DT>
__device__ int warp_count_ahead(const char* rowp, int V, int d, float xd) {
    int n = 0;
    for (int i = threadIdx.x & 31; i < V; i += 32) {
        const float x = Elt<DT>::load(rowp, i);
        n += (x > xd || (x == xd && i < d)) ? 1 : 0;
    }
    return __reduce_add_sync(0xFFFFFFFFu, n);
}

// ahead: the streaming pass's count for the row's hinted token (top-k mode), or -1.
template <int DT>
__device__ void tree_finish_warp(const TreeArgs& a, const RowJob& job, int64_t row, const RowPartial& merged,
                                 float neg_refc, bool centered, int sampled, int ahead, Tally& tally) {
    const int lane = threadIdx.x & 31;
    int t = 0, last = 0;
    int64_t lo = 0, hi = 0;
    double my_prob;
    RowFinal f = finish_row_warp(merged, job.c1, neg_refc, centered, key_value(merged.key[0]), my_prob);
    f.pmax = __shfl_sync(0xFFFFFFFFu, my_prob, 0);
    if (lane == 0) {
        const double lin = (double)a.alpha * f.H + (double)a.beta;
        TreeRowStat st;
        st.S = f.S;
        st.H = f.H;
        st.pmax = f.pmax;
        st.neg_refc = neg_refc;
        st.m = f.m;
        st.own = f.bad ? AASD_NONE : (a.mode == AASD_VERIFY_STRICT_SAMPLED ? sampled : f.top1);
        st.flags = (f.bad ? 1 : 0) | (centered ? 2 : 0);
        st.ahead = ahead;
        st.pad = 0;
        a.stats[row] = st;
        if (a.out.entropy) a.out.entropy[row] = (float)f.H;
        if (a.out.pmax) a.out.pmax[row] = (float)f.pmax;
        if (a.out.argmax) a.out.argmax[row] = f.top1;
        if (a.out.threshold) a.out.threshold[row] = f.bad ? 0.f : (float)fmin(lin, f.pmax);
        if (a.out.sampled) a.out.sampled[row] = f.bad ? AASD_NONE : sampled;
        tally.rows += 1;
        if (f.bad) {
            tally.bad += 1;
            tally.status |= AASD_STATUS_BAD_ROW;
        }
        t = find_segment(a.tree_offsets, a.n_trees, row);
        lo = a.tree_offsets[t];
        hi = a.tree_offsets[t + 1];
        // empty trees own no row: their neighbours write their (empty) result
        if (row == lo)
            for (int e = t - 1; e >= 0 && a.tree_offsets[e] == a.tree_offsets[e + 1]; --e) write_empty_tree(a, e);
        if (row == job.n_rows - 1)
            for (int e = t + 1; e < a.n_trees; ++e) write_empty_tree(a, e);
        __threadfence();
        const unsigned int k = atomicAdd(&a.tree_tickets[t], 1u);
        last = (k == (unsigned int)(hi - lo) - 1u);
        if (last) a.tree_tickets[t] = 0;
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    t = __shfl_sync(0xFFFFFFFFu, t, 0);
    lo = __shfl_sync(0xFFFFFFFFu, lo, 0);
    hi = __shfl_sync(0xFFFFFFFFu, hi, 0);
    __threadfence();
    const int n = (int)(hi - lo);

    // every node's own accept bit, judged with its parent's row (Eq. 3-6 / top-k / strict)
    unsigned int n_near = 0, n_acc = 0, status = 0;
    for (int base = 0; base < n; base += 32) {
        const int v = base + lane;
        const int64_t g = lo + v;
        const int p = (v == 0 || v >= n) ? AASD_NONE : a.node_parent[g];
        double pt = 0.0;
        bool acc = false, rank_wanted = false;
        int d = AASD_NONE, n_ahead = AASD_NONE;
        float x = 0.f;
        if (p >= 0 && p < v) {
            const TreeRowStat* ps = a.stats + lo + p;
            d = a.node_token[g];
            const bool d_ok = d >= 0 && d < job.vocab;
            if (!d_ok && d != AASD_NONE) status |= AASD_STATUS_ID_RANGE;
            const int pflags = __ldcg(&ps->flags);
            if (d_ok && !(pflags & 1)) {
                x = Elt<DT>::load(row_pointer<DT>(job, lo + p), d);
                RowFinal f;
                f.c1 = (double)job.c1;
                f.neg_refc = (double)__ldcg(&ps->neg_refc);
                f.centered = (pflags & 2) != 0;
                f.S = __ldcg(&ps->S);
                pt = f.prob(x);
                const unsigned int flag = a.node_flags ? a.node_flags[g] : AASD_FLAG_CONDITIONAL;
                if (a.mode == AASD_VERIFY_CONDITIONAL && (flag & AASD_FLAG_CONDITIONAL)) {
                    const double lin = (double)a.alpha * __ldcg(&ps->H) + (double)a.beta;
                    const bool at_max = (x == __ldcg(&ps->m));
                    acc = at_max || (pt >= lin);
                    if (!at_max && fabs(pt - lin) <= 1.0e-6) n_near += 1;
                } else if (a.mode == AASD_VERIFY_TOP_K && (flag & AASD_FLAG_CONDITIONAL)) {
                    rank_wanted = x > -CUDART_INF_F;     // a masked token has no rank and never passes
                } else {
                    acc = (d == __ldcg(&ps->own));
                }
                if (a.mode == AASD_VERIFY_TOP_K && x > -CUDART_INF_F) {
                    // the streaming pass counted for the parent's first child; siblings are counted below
                    const int counted = __ldcg(&ps->ahead);
                    if (counted >= 0 && d == __ldcg(a.hint + lo + p)) n_ahead = counted;
                    else n_ahead = -2;   // to be counted
                }
            }
        }
        if (a.mode == AASD_VERIFY_TOP_K) {
            unsigned int todo = __ballot_sync(0xFFFFFFFFu, n_ahead == -2);
            while (todo) {
                const int l = __ffs(todo) - 1;
                todo &= todo - 1;
                const int pp = __shfl_sync(0xFFFFFFFFu, p, l), dd = __shfl_sync(0xFFFFFFFFu, d, l);
                const float xx = __shfl_sync(0xFFFFFFFFu, x, l);
                const int cnt = warp_count_ahead<DT>(row_pointer<DT>(job, lo + pp), job.vocab, dd, xx);
                if (lane == l) n_ahead = cnt;
            }
            if (rank_wanted) acc = n_ahead >= 0 && n_ahead < a.top_k;
        }
        if (v < n) {
            if (a.out.p_token) a.out.p_token[g] = (float)pt;
            if (a.out.accept) a.out.accept[g] = acc ? 1 : 0;
            if (a.out.n_greater) a.out.n_greater[g] = (a.mode == AASD_VERIFY_TOP_K && n_ahead >= 0) ? n_ahead : AASD_NONE;
            a.node_ok[g] = acc ? 1 : 0;
            n_acc += acc ? 1 : 0;
        }
    }
    __syncwarp();
    n_near = __reduce_add_sync(0xFFFFFFFFu, n_near);
    n_acc = __reduce_add_sync(0xFFFFFFFFu, n_acc);
    status = __reduce_or_sync(0xFFFFFFFFu, status);
    tally.near += n_near;
    tally.accepted += n_acc;
    tally.status |= status;

    // prefix rule along the paths: a node passes when it and all its ancestors are accepted;
    // the deepest passing node wins, ties to the lowest index: key = (depth + 1, ~node)
    u64 key = 0;
    for (int v = lane; v < n; v += 32) {
        bool good = true;
        int depth = 0;
        for (int u = v; u != 0 && good; ++depth) {
            good = __ldcg(a.node_ok + lo + u) != 0;
            u = a.node_parent[lo + u];
            if (depth > n) good = false;   // malformed parents: never loops for ever
        }
        if (good) {
            const u64 k = ((u64)(unsigned int)(depth + 1) << 32) | (u64)(0xFFFFFFFFu - (unsigned int)v);
            key = k > key ? k : key;
        }
    }
    key = warp_max_u64(key);
    if (lane != 0) return;
    const int best = (int)(0xFFFFFFFFu - (unsigned int)key);
    const int depth = (int)(key >> 32) - 1;
    const int stride = a.emit_stride;
    int32_t* e = a.out.emit_ids ? a.out.emit_ids + (int64_t)t * stride : nullptr;
    const int own = __ldcg(&a.stats[lo + best].own);
    int ne = min(depth, stride);
    if (own != AASD_NONE && depth < stride) ne = depth + 1;
    if (e) {
        for (int i = ne; i < stride; ++i) e[i] = AASD_NONE;
        if (own != AASD_NONE && depth < stride) e[depth] = own;
        int pos = depth - 1;
        for (int u = best; u != 0; u = a.node_parent[lo + u], --pos)
            if (pos < stride) e[pos] = a.node_token[lo + u];
    }
    if (a.out.best_node) a.out.best_node[t] = best;
    if (a.out.n_accept) a.out.n_accept[t] = depth;
    if (a.out.n_emit) a.out.n_emit[t] = ne;
}

// Epilogue of the streaming kernel (entered by the whole finisher warp).
template <int DT>
struct TreeEpilogue {
    using Args = TreeArgs;
    struct State {};
    static __device__ __forceinline__ void init(State&) {}
    static __device__ __forceinline__ void drain(const TreeArgs&, const RowJob&, State&, Tally&) {}
    template <int ND>
    static __device__ void finish(const TreeArgs& a, const RowJob& job, int64_t row, const char* rowp,
                                  const FinishedRow& fr, const ItemInfo& info, const RaceSummary* races, int tail_group,
                                  State&, Tally& tally) {
        int sampled = AASD_NONE;
        if (ND > 0 && !partial_bad(fr.merged))
            sampled = warp_sample_decide<DT>(rowp, job.vocab, (unsigned int)row, 0, a.smp, races[0], tail_group,
                                             fr.centered, tally.recheck, tally.exhaustive);
        // top-k mode: the streaming pass counted the tokens ahead of the hinted token (exact when
        // the hint is a token of the vocabulary that is not masked)
        const bool counted = a.mode == AASD_VERIFY_TOP_K && info.hint >= 0 && info.hint < job.vocab &&
                             info.hint_logit > -CUDART_INF_F;
        tree_finish_warp<DT>(a, job, row, fr.merged, fr.neg_refc, fr.centered, sampled,
                             counted ? (int)fr.merged.ahead : -1, tally);
    }
    static __device__ __forceinline__ int prefetch(const TreeArgs&, int64_t) { return 0; }
};

// Plain-load kernel for layouts whose rows are not 16-byte aligned.
template <int DT>
__global__ void __launch_bounds__(kThreads) tree_kernel(const TreeArgs a) {
    __shared__ BlockScratch sc;
    pdl_launch_dependents();
    pdl_wait();
    const RowJob& job = a.job;
    const int64_t row = blockIdx.x / job.chunks;
    const int chunk = blockIdx.x % job.chunks;
    const char* rowp = row_pointer<DT>(job, row);
    float neg_refc;
    bool centered;
    if (!row_reduce<DT, 1>(job, row, chunk, __ldg(a.hint + row), rowp, neg_refc, centered, sc)) return;
    if (threadIdx.x >= 32) return;
    Tally tally;
    tally.clear();
    int sampled = AASD_NONE;
    if (a.mode == AASD_VERIFY_STRICT_SAMPLED && !partial_bad(sc.merged)) {
        sampled = warp_sample_exhaustive<DT>(rowp, job.vocab, (unsigned int)row, 0, a.smp);
        tally.exhaustive += 1;
    }
    tree_finish_warp<DT>(a, job, row, sc.merged, neg_refc, centered, sampled, -1, tally);
    if (threadIdx.x == 0) tally.flush(job.state);
}

}  // namespace aasd
