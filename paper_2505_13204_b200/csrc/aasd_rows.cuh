// Streaming kernels over logits rows: alignment sampling and conditional verification.
#pragma once

#include "aasd_device.cuh"
#include "aasd_sampler.cuh"

namespace aasd {

// What every row kernel needs to know about the logits block and the scratch memory.
struct RowJob {
    const void* logits;
    int64_t row_stride;     // elements
    int64_t n_rows;
    int vocab;
    int vector_ok;          // rows are 16-byte aligned: take the vector path
    int nvec;               // whole vectors per row (vector path)
    int stream_nvec;        // whole vectors every row has from its first 16-byte boundary on, whatever
                            // its alignment (the streaming kernel's planning figure; 0: rows too short)
    int vec_elts;           // logits per 16-byte vector
    int chunks;             // CTAs per row
    int vec_per_chunk;      // vectors per chunk (multiple of 8)
    float c1;               // inv_temperature * log2(e)
    RowPartial* partials;   // [n_rows x chunks] when chunks > 1
    unsigned int* row_tickets;
    DeviceState* state;
};

struct BlockScratch {
    double S[kWarps];
    double A[kWarps];
    u64 keys[kWarps][kMaxK];
    RowPartial merged;
    int flag;
};

template <int DT>
__device__ __forceinline__ const char* row_pointer(const RowJob& job, int64_t row) {
    return static_cast<const char*>(job.logits) + row * job.row_stride * (int64_t)Elt<DT>::kSize;
}

// Provisional reference of a row: the hinted token's logit (the draft token / the prompt's
// next token, very often the row maximum) and the first few entries.  Any finite value is
// valid; a good one keeps the exponents small.
template <int DT>
__device__ __forceinline__ float provisional_ref(const char* row, int vocab, int hint) {
    float r = -CUDART_INF_F;
    const int n = vocab < 4 ? vocab : 4;
    for (int i = 0; i < n; ++i) r = fmaxf(r, Elt<DT>::load(row, i));
    if (hint >= 0) r = fmaxf(r, Elt<DT>::load(row, hint));
    if (!(fabsf(r) <= 3.0e38f)) r = 0.f;   // NaN, +-inf
    return r;
}

// The part of a row a CTA streams: 16-byte vectors [vbeg, vend) counted from the 16-byte
// aligned address vbase, whose first element is token vid0 of the row, and the scalar
// elements [s1beg, s1end) and [s2beg, s2end) in front of and behind them.  A row that starts
// on a 16-byte boundary has vbase = row, vid0 = 0 and nothing in front; any other row is
// peeled up to its first boundary.
struct RowSpan {
    const char* vbase;
    int vid0, vbeg, vend, s1beg, s1end, s2beg, s2end;
};
// Elements [beg, end) of a row at an arbitrary (element-aligned) address.
template <int DT>
__device__ __forceinline__ RowSpan peeled_span(const char* row, int beg, int end) {
    constexpr int kVec = Elt<DT>::kVec, kSize = Elt<DT>::kSize;
    const uintptr_t addr = (uintptr_t)row + (uintptr_t)beg * kSize;
    int head = (int)(((16u - (unsigned int)(addr & 15u)) & 15u) / kSize);
    if (head > end - beg) head = end - beg;
    const int nv = (end - beg - head) / kVec;
    RowSpan sp;
    sp.vbase = row + (size_t)(beg + head) * kSize;
    sp.vid0 = beg + head;
    sp.vbeg = 0;
    sp.vend = nv;
    sp.s1beg = beg;
    sp.s1end = beg + head;
    sp.s2beg = beg + head + nv * kVec;
    sp.s2end = end;
    return sp;
}

// Streams a span of a row and leaves the CTA-wide result in sc.merged (valid for every
// thread after the closing barrier).
template <int DT, int K, bool SAFE>
__device__ void block_row_pass(const char* row, const RowSpan& sp, float c1, float neg_refc, BlockScratch& sc) {
    constexpr int kVec = Elt<DT>::kVec;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int vbeg = sp.vbeg, vend = sp.vend;
    RowAccumulator<DT, K, SAFE> acc;
    acc.init();

    const uint4* vrow = reinterpret_cast<const uint4*>(sp.vbase);
    int v = vbeg + tid;
    for (; v + 3 * kThreads < vend; v += 4 * kThreads) {
        uint4 q0 = load_stream16(vrow + v);
        uint4 q1 = load_stream16(vrow + v + kThreads);
        uint4 q2 = load_stream16(vrow + v + 2 * kThreads);
        uint4 q3 = load_stream16(vrow + v + 3 * kThreads);
        acc.add_vector(q0, v, c1, neg_refc);
        acc.add_vector(q1, v + kThreads, c1, neg_refc);
        acc.add_vector(q2, v + 2 * kThreads, c1, neg_refc);
        acc.add_vector(q3, v + 3 * kThreads, c1, neg_refc);
    }
    for (; v < vend; v += kThreads) {
        uint4 q = load_stream16(vrow + v);
        acc.add_vector(q, v, c1, neg_refc);
    }

    // the thread's best tokens: they lie inside its K best vectors
    u64 ek[K];
#pragma unroll
    for (int j = 0; j < K; ++j) ek[j] = 0;
#pragma unroll
    for (int j = 0; j < K; ++j) {
        if (acc.best_vec[j] >= 0) {
            uint4 q = __ldg(vrow + acc.best_vec[j]);
            float x[kVec];
            Elt<DT>::unpack(q, x);
#pragma unroll
            for (int i = 0; i < kVec; ++i)
                if (x[i] > -CUDART_INF_F) key_insert<K>(ek, make_key(x[i], sp.vid0 + acc.best_vec[j] * kVec + i));
        }
    }
    double S, A;
    acc.totals(S, A);
    // scalar parts: what lies in front of the first 16-byte boundary and the ragged tail
    {
        float s = 0.f, a = 0.f;
        for (int i = sp.s1beg + tid; i < sp.s1end; i += kThreads) {
            float xv = Elt<DT>::load(row, i);
            acc.add_scalar(xv, c1, neg_refc, s, a);
            if (xv > -CUDART_INF_F) key_insert<K>(ek, make_key(xv, i));
        }
        for (int i = sp.s2beg + tid; i < sp.s2end; i += kThreads) {
            float xv = Elt<DT>::load(row, i);
            acc.add_scalar(xv, c1, neg_refc, s, a);
            if (xv > -CUDART_INF_F) key_insert<K>(ek, make_key(xv, i));
        }
        S += (double)s;
        A += (double)a;
    }

    S = warp_sum_f64(S);
    A = warp_sum_f64(A);
#pragma unroll
    for (int r = 0; r < K; ++r) {
        u64 m = warp_max_u64(ek[0]);
        if (lane == 0) sc.keys[warp][r] = m;
        if (m != 0 && ek[0] == m) {
#pragma unroll
            for (int j = 0; j + 1 < K; ++j) ek[j] = ek[j + 1];
            ek[K - 1] = 0;
        }
    }
    if (lane == 0) {
        sc.S[warp] = S;
        sc.A[warp] = A;
    }
    __syncthreads();
    if (warp == 0) {
        double s = lane < kWarps ? sc.S[lane] : 0.0;
        double a = lane < kWarps ? sc.A[lane] : 0.0;
        s = warp_sum_f64(s);
        a = warp_sum_f64(a);
        u64 k = 0;
        if (lane < kWarps * K) k = sc.keys[lane / K][lane % K];
#pragma unroll
        for (int r = 0; r < K; ++r) {
            u64 m = warp_max_u64(k);
            if (lane == 0) sc.merged.key[r] = m;
            if (m != 0 && k == m) k = 0;
        }
        if (lane == 0) {
            sc.merged.S = s;
            sc.merged.A = a;
#pragma unroll
            for (int r = K; r < kMaxK; ++r) sc.merged.key[r] = 0;
        }
    }
    __syncthreads();
}

// Whole-row driver used by both kernels.  Returns true in the one CTA that holds the
// finished row (every CTA when chunks == 1); sc.merged then holds the row's sums and best
// tokens.  The exponents behind the sums are fma(x, c1, neg_refc) when `centered` is false
// and (x - max) * c1 (with neg_refc = -max) when the second pass ran.
template <int DT, int K>
__device__ bool row_reduce(const RowJob& job, int64_t row, int chunk, int hint, const char* rowp,
                           float& neg_refc, bool& centered, BlockScratch& sc) {
    centered = false;
    constexpr int kVec = Elt<DT>::kVec;
    const int tid = threadIdx.x;
    const int V = job.vocab;
    const float c1 = job.c1;
    neg_refc = -(provisional_ref<DT>(rowp, V, hint) * c1);

    RowSpan sp;
    if (job.vector_ok) {
        sp.vbase = rowp;
        sp.vid0 = 0;
        sp.vbeg = chunk * job.vec_per_chunk;
        sp.vend = min(job.nvec, sp.vbeg + job.vec_per_chunk);
        if (sp.vbeg > sp.vend) sp.vbeg = sp.vend;
        sp.s1beg = sp.s1end = 0;
        sp.s2beg = sp.s2end = 0;
        if (chunk == 0) {
            sp.s2beg = job.nvec * kVec;
            sp.s2end = V;
        }
    } else {
        // unaligned layout: split the elements themselves, then peel each share up to its
        // first 16-byte boundary
        int per = (V + job.chunks - 1) / job.chunks;
        const int beg = min(V, chunk * per);
        sp = peeled_span<DT>(rowp, beg, min(V, beg + per));
    }
    block_row_pass<DT, K, false>(rowp, sp, c1, neg_refc, sc);

    if (job.chunks > 1) {
        RowPartial* slots = job.partials + row * job.chunks;
        if (tid == 0) {
            slots[chunk] = sc.merged;
            __threadfence();
            unsigned int t = atomicAdd(&job.row_tickets[row], 1u);
            sc.flag = (t == (unsigned int)job.chunks - 1);
        }
        __syncthreads();
        if (!sc.flag) return false;
        __threadfence();
        if (tid < 32) {
            double s = 0.0, a = 0.0;
            u64 k[K];
#pragma unroll
            for (int j = 0; j < K; ++j) k[j] = 0;
            if (tid < job.chunks) {
                const RowPartial* p = slots + tid;
                s = __ldcg(&p->S);
                a = __ldcg(&p->A);
#pragma unroll
                for (int j = 0; j < K; ++j) k[j] = __ldcg(&p->key[j]);
            }
            s = warp_sum_f64(s);
            a = warp_sum_f64(a);
#pragma unroll
            for (int r = 0; r < K; ++r) {
                u64 m = warp_max_u64(k[0]);
                if (tid == 0) sc.merged.key[r] = m;
                if (m != 0 && k[0] == m) {
#pragma unroll
                    for (int j = 0; j + 1 < K; ++j) k[j] = k[j + 1];
                    k[K - 1] = 0;
                }
            }
            if (tid == 0) {
                sc.merged.S = s;
                sc.merged.A = a;
                job.row_tickets[row] = 0;   // ready for the next call
            }
        }
        __syncthreads();
    }

    // Second pass when the provisional reference was too far from the maximum for the
    // fp32 sums to be trusted (overflow, underflow to zero, -inf entries, large shift).
    const u64 k0 = sc.merged.key[0];
    const float m = key_value(k0);
    bool redo = false;
    if (k0 != 0 && fabsf(m) <= 3.0e38f) {
        const double S = sc.merged.S, A = sc.merged.A;
        const float shift = fmaf(m, c1, neg_refc);
        redo = !(S > 0.0) || !(S <= 1.0e300) || !(fabs(A) <= 1.0e300) || !(fabsf(shift) <= kRedoShift);
    }
    __syncthreads();   // everyone has read sc.merged
    if (redo) {
        neg_refc = -m;
        centered = true;
        RowSpan all = peeled_span<DT>(rowp, 0, V);   // an aligned row peels nothing
        block_row_pass<DT, K, true>(rowp, all, c1, neg_refc, sc);
        if (tid == 0) atomicAdd(&job.state->counters[kCntRedo], 1ull);
    }
    return true;
}

// Scalars of a finished row (Eq. 5-6), evaluated in double by one thread.
struct RowFinal {
    bool bad;
    float m;        // raw logit of the best token
    int top1;
    double S;       // relative to the reference
    double H;       // nats
    double pmax;
    double c1;
    double neg_refc;
    bool centered;
    // probability of a token from its raw logit, with the exponent the streaming pass used
    __device__ double prob(float x) const {
        const double t = centered ? ((double)x + neg_refc) * c1 : (double)x * c1 + neg_refc;
        return fmin(exp2(t) / S, 1.0);   // (S comes from fp32 sums: a lone spike may land a hair above 1)
    }
};

// A row is bad when it held NaN or +inf, or nothing but -inf.
__device__ inline bool partial_bad(const RowPartial& p) {
    const float m = key_value(p.key[0]);
    return (p.key[0] == 0) || !(fabsf(m) <= 3.0e38f) || !(p.S > 0.0) || !(p.S <= 1.0e300) || !(fabs(p.A) <= 1.0e300);
}

__device__ inline RowFinal finish_row(const RowPartial& p, float c1, float neg_refc, bool centered) {
    RowFinal f;
    f.c1 = (double)c1;
    f.neg_refc = (double)neg_refc;
    f.centered = centered;
    f.m = key_value(p.key[0]);
    f.top1 = key_id(p.key[0]);
    f.S = p.S;
    f.bad = partial_bad(p);
    if (f.bad) {
        f.top1 = AASD_NONE;
        f.H = 0.0;
        f.pmax = 0.0;
        f.S = 1.0;
        return f;
    }
    f.H = fmax(log(p.S) - kLn2 * (p.A / p.S), 0.0);   // (and its entropy a hair below 0)
    f.pmax = f.prob(f.m);
    return f;
}

// The same by a whole warp, with the probabilities of up to 31 tokens of the row alongside:
// lane l < 31 hands in the raw logit of a token (`my_x`; anything where it has none) and
// gets the token's probability back in `my_prob`.  All the fp64 work of a row - the logarithm
// of Eq. 5 and the exponentials of the probabilities - is one exponential per lane, evaluated
// by all lanes at once instead of one after the other by one lane: lane 31 evaluates
// 2^-y0 for y0 = lg2.approx(S), which turns log2(S) = y0 + log2(S * 2^-y0) into a three-term
// series in S * 2^-y0 - 1 (|.| < 2^-21, truncation below 1e-27); the divisions by S are
// multiplications by one reciprocal.  Results differ from finish_row's by a few fp64 ulps.
__device__ inline RowFinal finish_row_warp(const RowPartial& p, float c1, float neg_refc, bool centered, float my_x,
                                           double& my_prob) {
    RowFinal f;
    f.c1 = (double)c1;
    f.neg_refc = (double)neg_refc;
    f.centered = centered;
    f.m = key_value(p.key[0]);
    f.top1 = key_id(p.key[0]);
    f.S = p.S;
    f.bad = partial_bad(p);     // the same in every lane: p is
    my_prob = 0.0;
    if (f.bad) {
        f.top1 = AASD_NONE;
        f.H = 0.0;
        f.pmax = 0.0;
        f.S = 1.0;
        return f;
    }
    const int lane = threadIdx.x & 31;
    float y0;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y0) : "f"((float)p.S));
    if (!(fabsf(y0) <= 1.0e30f)) y0 = 0.f;      // S outside float's range: the series would not hold ...
    const double t = lane == 31 ? -(double)y0
                                : (centered ? ((double)my_x + f.neg_refc) * f.c1 : (double)my_x * f.c1 + f.neg_refc);
    const double e = exp2(t);
    const double inv_s = 1.0 / p.S;
    my_prob = fmin(e * inv_s, 1.0);   // a probability (Eq. 4, 6): the fp32 sums may put a lone spike a hair above 1
    const double u = __shfl_sync(0xFFFFFFFFu, e, 31) * p.S - 1.0;
    constexpr double kInvLn2 = 1.4426950408889634;
    double log2_s = (double)y0 + u * (kInvLn2 + u * (-0.5 * kInvLn2 + u * (kInvLn2 / 3.0)));
    if (!(fabs(u) <= 1.0e-3)) log2_s = log2(p.S);   // ... so take the library's logarithm there
    f.H = fmax(kLn2 * (log2_s - p.A * inv_s), 0.0);   // an entropy: likewise never below 0
    return f;
}

// ---- conditional verification -----------------------------------------------------------------

// Optional tail of a verification launch: once the last candidate of a sequence is done,
// choose the longest passing candidate (Sec. 3.3) and append what it emits to the
// sequence's history (Algorithm 1).  Regular layout only: cands_per_seq candidates per
// sequence, rows_per_cand rows per candidate.
struct SeqTail {
    int enabled;
    int cands_per_seq;
    int rows_per_seq;            // cands_per_seq * rows per candidate
    int emit_stride;
    unsigned int* seq_tickets;   // [n_seqs], zero between launches
    int32_t* best_cand;
    int32_t* n_emit;
    int32_t* emit_ids;
    int32_t* hist_ids;
    const int32_t* hist_offsets;
    int32_t* hist_len;
    // alignment sampling on generated context: table rows of the emitted tokens
    int32_t* table_ids;                 // NULL: off
    int32_t* table_n;
    const int32_t* table_row_offsets;   // [n_seqs] table row of each sequence's first position
    int table_k;                        // row width of table_ids
};

constexpr int kRowExtraInts = 1 + kMaxK;   // per row: how many tokens rank above its draft token, and which

struct VerifyArgs {
    RowJob job;
    const int32_t* draft_ids;
    const uint8_t* draft_flags;
    const int32_t* cand_offsets;   // NULL: regular candidates of rows_per_cand rows
    int n_cands;
    int rows_per_cand;
    float alpha, beta;
    int mode;
    unsigned int* cand_tickets;
    u64* row_state;                // scratch [n_rows]: the row's own token << 32 | its accept bit
    int32_t* row_extra;            // scratch [n_rows x kRowExtraInts] or NULL: (count, ids) ranked above the row's draft token
    SampleJob smp;                 // STRICT_SAMPLED: the row's own token is a keyed draw
    int top_k;                     // TOP_K mode
    unsigned int hints;            // AASD_HINT_*
    SeqTail seq;
    aasd_verify_out out;
};

// Candidate that owns row r: the last c with cand_offsets[c] <= r.
__device__ inline int find_segment(const int32_t* offsets, int n, int64_t r) {
    int lo = 0, hi = n;   // invariant: offsets[lo] <= r < offsets[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if ((int64_t)__ldg(offsets + mid) <= r) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ inline void write_empty_candidate(const VerifyArgs& a, int c) {
    if (a.out.accept_len) a.out.accept_len[c] = 0;
    if (a.out.next_token) a.out.next_token[c] = AASD_NONE;
}

// What a finished row adds to the running counters and the status word.  The streaming
// kernel keeps one per CTA in registers and flushes it when the CTA leaves.
struct Tally {
    unsigned int rows, bad, redo, near, accepted, recheck, exhaustive, status;
    __device__ void clear() { rows = bad = redo = near = accepted = recheck = exhaustive = status = 0; }
    __device__ void flush(DeviceState* st) const {
        if (rows) atomicAdd(&st->counters[kCntRows], (u64)rows);
        if (bad) atomicAdd(&st->counters[kCntBad], (u64)bad);
        if (redo) atomicAdd(&st->counters[kCntRedo], (u64)redo);
        if (near) atomicAdd(&st->counters[kCntNear], (u64)near);
        if (accepted) atomicAdd(&st->counters[kCntAccepted], (u64)accepted);
        if (recheck) atomicAdd(&st->counters[kCntRecheck], (u64)recheck);
        if (exhaustive) atomicAdd(&st->counters[kCntExact], (u64)exhaustive);
        if (status) atomicOr(&st->status, status);
    }
};

// Eq. 4-6 for one row, by one thread, once the row's sums and best token are known: writes
// the row's outputs and its accept bit / own token for the prefix rule.  d is the row's
// draft id as given, xd its raw logit (read only when d lies inside the vocabulary), sampled
// the row's keyed draw in STRICT_SAMPLED mode (NONE otherwise, and on a bad row).  In TOP_K
// mode merged.ahead is the number of tokens ahead of d in the order (logit desc, id asc).
// What the prefix rule needs of the row goes out first and the row's ticket (the counter of
// its candidate) is taken right behind it, so that the stores of the row's outputs, which
// nobody inside the launch reads, are under way while the ticket travels.  Returns the
// ticket's value.
// flag: the row's draft-token flag byte (AASD_FLAG_CONDITIONAL when the call has no flags).
// f: the row's scalars (finish_row_warp), pd_in: the draft token's probability from the same call.
template <int DT>
__device__ unsigned int verify_row(const VerifyArgs& a, const RowJob& job, int64_t row, const RowPartial& merged,
                                   const RowFinal& f, double pd_in, int d, float xd, unsigned int flag, int sampled,
                                   unsigned int* ticket, Tally& tally) {
    const bool d_ok = d >= 0 && d < job.vocab;
    if (!AASD_IN_RANGE(row >= 0 && row < job.n_rows && (f.bad || (f.top1 >= 0 && f.top1 < job.vocab)), job.state)) return 0xFFFFFFFFu;
    const double lin = (double)a.alpha * f.H + (double)a.beta;
    const double thr = f.bad ? 0.0 : fmin(lin, f.pmax);
    const int own = a.mode == AASD_VERIFY_STRICT_SAMPLED ? sampled : f.top1;   // NONE on a bad row
    double pd = 0.0;
    bool acc = false, near = false;
    if (f.bad) tally.status |= AASD_STATUS_BAD_ROW;
    if (!d_ok && d != AASD_NONE) tally.status |= AASD_STATUS_ID_RANGE;
    if (d_ok && !f.bad) {
        pd = pd_in;
        if (a.mode == AASD_VERIFY_CONDITIONAL && (flag & AASD_FLAG_CONDITIONAL)) {
            const bool at_max = (xd == f.m);
            acc = at_max || (pd >= lin);
            near = !at_max && fabs(pd - lin) <= 1.0e-6;
        } else if (a.mode == AASD_VERIFY_TOP_K && (flag & AASD_FLAG_CONDITIONAL)) {
            acc = xd > -CUDART_INF_F && merged.ahead < (long long)a.top_k;
        } else {
            acc = (d == own);
        }
    }
    a.row_state[row] = ((u64)(unsigned int)own << 32) | (acc ? 1ull : 0ull);
    if (a.row_extra) {
        // Fig. 2's rule with the draft token in the place of the prompt's next token
        int n = 0, ids[kMaxK];
#pragma unroll
        for (int j = 0; j < kMaxK; ++j) ids[j] = AASD_NONE;
        if (d_ok && !f.bad) {
            const int width = a.seq.table_k < kMaxK ? a.seq.table_k : kMaxK;
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) {
                const u64 k = merged.key[j];
                if (j >= width || k == 0) break;
                const float xv = key_value(k);
                const int id = key_id(k);
                if (xv > xd || (xv == xd && id < d)) {
#pragma unroll
                    for (int q = 0; q < kMaxK; ++q)
                        if (q == n) ids[q] = id;
                    ++n;
                }
            }
        }
        int32_t* x = a.row_extra + row * kRowExtraInts;
        x[0] = n;
#pragma unroll
        for (int j = 0; j < kMaxK; ++j) x[1 + j] = ids[j];
    }
    const unsigned int t = take_ticket(ticket);
    if (a.out.n_greater)
        a.out.n_greater[row] = (a.mode == AASD_VERIFY_TOP_K && d_ok && !f.bad && xd > -CUDART_INF_F)
                                   ? (int)merged.ahead : AASD_NONE;
    if (a.out.p_draft) a.out.p_draft[row] = (float)pd;
    if (a.out.entropy) a.out.entropy[row] = (float)f.H;
    if (a.out.pmax) a.out.pmax[row] = (float)f.pmax;
    if (a.out.argmax) a.out.argmax[row] = f.top1;
    if (a.out.threshold) a.out.threshold[row] = (float)thr;
    if (a.out.accept) a.out.accept[row] = acc ? 1 : 0;
    if (a.out.sampled) a.out.sampled[row] = f.bad ? AASD_NONE : sampled;
    tally.rows += 1;
    tally.bad += f.bad ? 1 : 0;
    tally.near += near ? 1 : 0;
    tally.accepted += acc ? 1 : 0;
    return t;
}

// Candidate of a row and its row range; results of the empty candidates next to it (they
// own no row, so a neighbour writes them).
__device__ inline int candidate_of_row(const VerifyArgs& a, int64_t n_rows, int64_t row, int64_t& lo, int64_t& hi) {
    int c;
    if (a.cand_offsets) {
        c = find_segment(a.cand_offsets, a.n_cands, row);
        lo = a.cand_offsets[c];
        hi = a.cand_offsets[c + 1];
        if (row == lo)
            for (int e = c - 1; e >= 0 && a.cand_offsets[e] == a.cand_offsets[e + 1]; --e)
                write_empty_candidate(a, e);
        if (row == n_rows - 1)
            for (int e = c + 1; e < a.n_cands; ++e) write_empty_candidate(a, e);
    } else {
        c = (int)(row / a.rows_per_cand);
        lo = (int64_t)c * a.rows_per_cand;
        hi = lo + a.rows_per_cand;
    }
    return c;
}

// A row whose ticket has been taken but not looked at yet: what the warp needs to complete the
// row's candidate once the ticket's value is in (lane 0's copy counts).
struct PendingRow {
    int valid;
    int c;
    int64_t lo, hi;
    unsigned int ticket;
    int whole_sequence;   // the ticket counts the rows of the candidate's whole sequence (see below)
};

// A launch that also selects and appends (SeqTail) with sequences of at most 32 rows counts
// rows per sequence instead of rows per candidate: one ticket per row, and the warp that takes
// a sequence's last one does everything for it with the rows' records in its lanes.
__device__ __forceinline__ bool sequence_tickets(const VerifyArgs& a) {
    return a.seq.enabled && a.seq.rows_per_seq <= 32;
}

// Row epilogue of verification, first half, run by a whole warp: lane 0 evaluates the row
// (Eq. 4-6), writes its outputs and takes the ticket of its candidate.
template <int DT>
__device__ void verify_row_warp(const VerifyArgs& a, const RowJob& job, int64_t row, const RowPartial& merged,
                                float neg_refc, bool centered, int d, float xd, unsigned int flag, int sampled,
                                PendingRow& pending, Tally& tally) {
    pending.valid = 1;
    pending.c = 0;
    pending.lo = pending.hi = 0;
    pending.ticket = 0;
    pending.whole_sequence = 0;
    // the row's scalars by the whole warp: lane 0 asks for the best token's probability
    // (Delta of Eq. 6), lane 1 for the draft token's (Eq. 4)
    const int lane_id = threadIdx.x & 31;
    double my_prob;
    RowFinal f = finish_row_warp(merged, job.c1, neg_refc, centered, lane_id == 1 ? xd : key_value(merged.key[0]), my_prob);
    f.pmax = __shfl_sync(0xFFFFFFFFu, my_prob, 0);
    const double pd = __shfl_sync(0xFFFFFFFFu, my_prob, 1);
    if (lane_id == 0) {
        int64_t lo = 0, hi = 0;
        int c = candidate_of_row(a, job.n_rows, row, lo, hi);
        if (!AASD_IN_RANGE(c >= 0 && c < a.n_cands && lo >= 0 && lo <= row && row < hi && hi <= job.n_rows, job.state)) c = 0, hi = lo = 0;
        pending.whole_sequence = sequence_tickets(a) ? 1 : 0;
        unsigned int* ticket = pending.whole_sequence ? &a.seq.seq_tickets[c / a.seq.cands_per_seq] : &a.cand_tickets[c];
        pending.ticket = verify_row<DT>(a, job, row, merged, f, pd, d, xd, flag, sampled, ticket, tally);
        pending.c = c;
        pending.lo = lo;
        pending.hi = hi;
    }
}

// Second half: the warp that took a candidate's last ticket applies the prefix rule with one
// load per lane, and, when that completes a sequence, selects and appends.  The streaming
// kernel runs it one row late, so that the ticket's trip to memory is hidden behind the next
// row's work.
__device__ inline void verify_complete_warp(const VerifyArgs& a, const RowJob& job, const PendingRow& pending, Tally& tally);

template <int DT>
__device__ void verify_finish_warp(const VerifyArgs& a, const RowJob& job, int64_t row, const RowPartial& merged,
                                   float neg_refc, bool centered, int d, float xd, unsigned int flag, int sampled,
                                   Tally& tally) {
    PendingRow pending;
    verify_row_warp<DT>(a, job, row, merged, neg_refc, centered, d, xd, flag, sampled, pending, tally);
    verify_complete_warp(a, job, pending, tally);
}

// Emission of a finished sequence b: the winning candidate's accepted draft tokens and the
// target's own token go to emit_ids and to the history, their extras to the alignment table.
// draft_token(i): token i of the winning candidate.
template <class DraftToken>
__device__ __forceinline__ void emit_and_append(const VerifyArgs& a, int b, int best, int best_a, int nt, int off, int cap,
                                                int len, DraftToken draft_token, Tally& tally) {
    const int lane = threadIdx.x & 31;
    const int stride = a.seq.emit_stride;
    int32_t* e = a.seq.emit_ids + (int64_t)b * stride;
    int ne = 0;
    if (best != AASD_NONE) {
        ne = min(best_a, stride);
        if (nt != AASD_NONE && ne < stride) ne += 1;
    }
    for (int base = 0; base < stride; base += 32) {
        const int i = base + lane;
        const int drafted = draft_token(i < best_a ? i : 0);     // (a shuffle: every lane takes part)
        if (i < stride) {
            int tok = AASD_NONE;
            if (i < ne) tok = (i < best_a) ? drafted : nt;
            e[i] = tok;
            if (i < ne && len + i < cap) a.seq.hist_ids[off + len + i] = tok;
        }
    }
    if (a.seq.table_ids) {
        // table rows of the emitted tokens: position len + i has row (first row) + len + i - 1
        const int64_t row0 = (int64_t)a.seq.table_row_offsets[b] + len - 1;
        const int K = a.seq.table_k;
        for (int i = lane; i < ne; i += 32) {
            if (len + i >= cap || len + i < 1) continue;
            int n = 0, ids[kMaxK];
#pragma unroll
            for (int j = 0; j < kMaxK; ++j) ids[j] = AASD_NONE;
            if (i < best_a) {
                const int32_t* x = a.row_extra + ((int64_t)best * a.rows_per_cand + i) * kRowExtraInts;
                n = __ldcg(x);
#pragma unroll
                for (int j = 0; j < kMaxK; ++j) ids[j] = __ldcg(x + 1 + j);
            }
            a.seq.table_n[row0 + i] = n;
#pragma unroll
            for (int j = 0; j < kMaxK; ++j)
                if (j < K) a.seq.table_ids[(row0 + i) * K + j] = ids[j];
        }
    }
    __syncwarp();
    if (lane == 0) {
        a.seq.best_cand[b] = best;
        a.seq.n_emit[b] = ne;
        a.seq.hist_len[b] = min(len + ne, cap);
        if (len + ne > cap) tally.status |= AASD_STATUS_HIST_OVERFLOW;
    }
}

// Everything a finished sequence of at most 32 rows needs, with row i of the sequence in lane
// i: the prefix rule per candidate (Sec. 2.1), the longest passing candidate (Sec. 3.3), the
// emission and the history update (Algorithm 1).  One trip to memory for the rows' records.
__device__ inline void verify_complete_sequence(const VerifyArgs& a, int b, Tally& tally) {
    const int lane = threadIdx.x & 31;
    const int cps = a.seq.cands_per_seq, rpc = a.rows_per_cand, rps = a.seq.rows_per_seq;
    const int64_t row0 = (int64_t)b * rps;
    const u64 st = lane < rps ? __ldcg(a.row_state + row0 + lane) : 1ull;
    const int dtok = lane < rps ? __ldg(a.draft_ids + row0 + lane) : AASD_NONE;
    const int off = a.seq.hist_offsets[b];
    const int cap = a.seq.hist_offsets[b + 1] - off;
    const int len = a.seq.hist_len[b];
    const unsigned int rejected = __ballot_sync(0xFFFFFFFFu, lane < rps && (st & 1ull) == 0);
    const int own = (int)(unsigned int)(st >> 32);
    const unsigned int seg_mask = rpc >= 32 ? 0xFFFFFFFFu : ((1u << rpc) - 1u);
    int best = AASD_NONE, best_a = -1, nt = AASD_NONE;
    for (int j = 0; j < cps; ++j) {
        const unsigned int seg = (rejected >> (j * rpc)) & seg_mask;
        const int n = seg ? __ffs(seg) - 1 : rpc;              // leading accepted rows
        int next = __shfl_sync(0xFFFFFFFFu, own, j * rpc + (seg ? n : 0));
        next = seg ? next : AASD_NONE;                          // the own token of the first row that does not pass
        if (lane == 0) {
            if (a.out.accept_len) a.out.accept_len[b * cps + j] = n;
            if (a.out.next_token) a.out.next_token[b * cps + j] = next;
        }
        if (n > best_a) {      // ties go to the lower candidate
            best_a = n;
            best = b * cps + j;
            nt = next;
        }
    }
    if (best == AASD_NONE) best_a = 0;
    const int first_row = (best - b * cps) * rpc;
    emit_and_append(a, b, best, best_a, nt, off, cap, len,
                    [&](int i) { return __shfl_sync(0xFFFFFFFFu, dtok, best == AASD_NONE ? 0 : first_row + i); }, tally);
}

__device__ inline void verify_complete_warp(const VerifyArgs& a, const RowJob& job, const PendingRow& pending, Tally& tally) {
    const int lane = threadIdx.x & 31;
    int c = pending.c, last = 0;
    int64_t lo = pending.lo, hi = pending.hi;
    if (__shfl_sync(0xFFFFFFFFu, pending.whole_sequence, 0)) {
        int b = 0;
        if (lane == 0) {
            b = c / a.seq.cands_per_seq;
            last = (pending.ticket == (unsigned int)a.seq.rows_per_seq - 1u);
            if (last) a.seq.seq_tickets[b] = 0;
        }
        last = __shfl_sync(0xFFFFFFFFu, last, 0);
        if (!last) return;
        b = __shfl_sync(0xFFFFFFFFu, b, 0);
        // lane 0's ticket acquired what the other rows' warps released; the warp barrier hands
        // that on to the other lanes, whose loads go to L2 (no fence, which would also wait for
        // this warp's own stores)
        __syncwarp();
        verify_complete_sequence(a, b, tally);
        return;
    }
    if (lane == 0) {
        last = (pending.ticket == (unsigned int)(hi - lo) - 1u);
        if (last) a.cand_tickets[c] = 0;
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    c = __shfl_sync(0xFFFFFFFFu, c, 0);
    lo = __shfl_sync(0xFFFFFFFFu, lo, 0);
    hi = __shfl_sync(0xFFFFFFFFu, hi, 0);
    __syncwarp();   // (as above: lane 0's ticket acquired the other rows' records)
    int64_t n = hi - lo;   // leading accepted rows
    int next = AASD_NONE;  // the own token of the first row that does not pass
    for (int64_t base = lo; base < hi; base += 32) {
        const int64_t r = base + lane;
        const u64 st = r < hi ? __ldcg(a.row_state + r) : 1ull;
        const unsigned int bal = __ballot_sync(0xFFFFFFFFu, (st & 1ull) == 0);
        if (bal) {
            const int first = __ffs(bal) - 1;
            n = base - lo + first;
            next = (int)(unsigned int)(__shfl_sync(0xFFFFFFFFu, st, first) >> 32);
            break;
        }
    }
    if (lane == 0) {
        if (a.out.accept_len) a.out.accept_len[c] = (int)n;
        if (a.out.next_token) a.out.next_token[c] = next;
    }
    if (!a.seq.enabled) return;

    // The warp that completes a sequence's last candidate selects and appends.
    const int cps = a.seq.cands_per_seq;
    const int b = c / cps;
    if (cps > 1) {     // a sequence with a single candidate is complete with it: no second ticket
        if (lane == 0) {
            const unsigned int t = take_ticket(&a.seq.seq_tickets[b]);
            last = (t == (unsigned int)cps - 1u);
            if (last) a.seq.seq_tickets[b] = 0;
        }
        last = __shfl_sync(0xFFFFFFFFu, last, 0);
        if (!last) return;
        __syncwarp();
    }
    // longest accepted prefix, ties to the lowest candidate: key = (length + 1, ~candidate)
    u64 key = 0;
    for (int j = lane; j < cps; j += 32) {
        const int cj = b * cps + j;
        const u64 k = ((u64)(unsigned int)(__ldcg(a.out.accept_len + cj) + 1) << 32) | (u64)(0xFFFFFFFFu - (unsigned int)cj);
        key = k > key ? k : key;
    }
    key = warp_max_u64(key);
    int best = AASD_NONE, best_a = 0;
    if (key != 0) {
        best = (int)(0xFFFFFFFFu - (unsigned int)key);
        best_a = (int)(key >> 32) - 1;
    }
    const int off = a.seq.hist_offsets[b];
    const int cap = a.seq.hist_offsets[b + 1] - off;
    const int len = a.seq.hist_len[b];
    const int nt = best != AASD_NONE ? __ldcg(a.out.next_token + best) : AASD_NONE;
    emit_and_append(a, b, best, best_a, nt, off, cap, len,
                    [&](int i) { return best != AASD_NONE ? a.draft_ids[(int64_t)best * a.rows_per_cand + i] : AASD_NONE; }, tally);
}

// One CTA (or `chunks` CTAs) per row with plain vector / scalar loads: the path for logits
// whose rows are not 16-byte aligned.
// K: how many of the row's best tokens are kept (1, or the table's width when the step also
// enters the emitted tokens into the alignment table).
template <int DT, int K = 1>
__global__ void __launch_bounds__(kThreads) verify_kernel(const VerifyArgs a) {
    __shared__ BlockScratch sc;
    pdl_launch_dependents();
    pdl_wait();
    const RowJob& job = a.job;
    const int64_t row = blockIdx.x / job.chunks;
    const int chunk = blockIdx.x % job.chunks;
    const char* rowp = row_pointer<DT>(job, row);
    const int d = __ldg(a.draft_ids + row);
    const bool d_ok = d >= 0 && d < job.vocab;
    float neg_refc;
    bool centered;
    if (!row_reduce<DT, K>(job, row, chunk, d_ok ? d : -1, rowp, neg_refc, centered, sc)) return;
    if (threadIdx.x >= 32) return;
    const float xd = d_ok ? Elt<DT>::load(rowp, d) : 0.f;
    Tally tally;
    tally.clear();
    int sampled = AASD_NONE;
    if (a.mode == AASD_VERIFY_STRICT_SAMPLED && !partial_bad(sc.merged)) {
        // this layout takes the definition as it stands: every group scored in fp64
        sampled = warp_sample_exhaustive<DT>(rowp, job.vocab, (unsigned int)row, 0, a.smp);
        tally.exhaustive += 1;
    }
    if (a.mode == AASD_VERIFY_TOP_K) {
        // and counts the tokens ahead of the draft token by going over the row once more
        long long n = 0;
        if (d_ok)
            for (int i = threadIdx.x; i < job.vocab; i += 32) {
                const float x = Elt<DT>::load(rowp, i);
                n += (x > xd || (x == xd && i < d)) ? 1 : 0;
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xFFFFFFFFu, n, o);
        sc.merged.ahead = n;
        __syncwarp();
    }
    const unsigned int flag = a.draft_flags ? a.draft_flags[row] : AASD_FLAG_CONDITIONAL;
    verify_finish_warp<DT>(a, job, row, sc.merged, neg_refc, centered, d, xd, flag, sampled, tally);
    if (threadIdx.x == 0) tally.flush(job.state);
}

#ifdef AASD_HOST_TU   // not a template: compiled in the host translation unit only
// Candidates of a call without rows.
__global__ void verify_empty_kernel(const VerifyArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < a.n_cands) write_empty_candidate(a, c);
}
#endif

// ---- alignment sampling ---------------------------------------------------------------------------

struct AlignArgs {
    RowJob job;
    const int32_t* prompt_ids;
    const int32_t* seq_offsets;
    int n_seqs;
    int k_extra;
    int mode;
    unsigned int hints;   // AASD_HINT_*
    int32_t* next_ids;   // scratch [n_rows]: the prompt's next token of every row
    SampleJob smp;       // GUMBEL mode: the extras are keyed draws
    aasd_align_out out;
};

#ifdef AASD_HOST_TU   // not a template: compiled in the host translation unit only
// next_ids[t] = prompt_ids[t+1] unless t is the last row of its sequence.
__global__ void align_next_kernel(const AlignArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= a.job.n_rows) return;
    int b = find_segment(a.seq_offsets, a.n_seqs, t);
    int nxt = AASD_NONE;
    if (t + 1 < (int64_t)a.seq_offsets[b + 1]) {
        nxt = a.prompt_ids[t + 1];
        if (nxt < 0 || nxt >= a.job.vocab) {
            nxt = AASD_NONE;
            atomicOr(&a.job.state->status, AASD_STATUS_ID_RANGE);
        }
    }
    a.next_ids[t] = nxt;
}
#endif

// Does the row take keyed draws?  GUMBEL mode, a usable row, and a next token that is not the
// greedy one (Sec. 2.3: only misaligned positions get extra tokens).
__device__ inline bool align_wants_draws(const AlignArgs& a, const RowPartial& merged, int next) {
    if (a.mode != AASD_ALIGN_GUMBEL || a.k_extra == 0 || partial_bad(merged)) return false;
    return !(next != AASD_NONE && next == key_id(merged.key[0]));
}

// Row epilogue of alignment sampling (Sec. 2.3 alignment test, Fig. 2 extras): entered by a whole
// warp for the row's fp64 scalars, finished by lane 0.
// next is the prompt's next token of the row (validated, or NONE), xn its raw logit.  In
// GUMBEL mode draws[j] / draw_logits[j] are the row's keyed draws (NONE where not drawn).
__device__ inline void align_row(const AlignArgs& a, const RowJob& job, int64_t row, const RowPartial& merged,
                                 float neg_refc, bool centered, int next, float xn_in, const int* draws,
                                 const float* draw_logits, Tally& tally) {
    // the row's scalars and every probability the row may report, by the whole warp: lane 0 the
    // best token's, lane 1 the next token's, lanes 2 .. 2+K-1 the listed tokens' (TOPK) or the
    // draws' (GUMBEL)
    const int lane_id = threadIdx.x & 31;
    float my_x = key_value(merged.key[0]);
    if (lane_id == 1) my_x = xn_in;
#pragma unroll
    for (int j = 0; j < kMaxK; ++j)
        if (lane_id == 2 + j) my_x = a.mode == AASD_ALIGN_GUMBEL ? draw_logits[j] : key_value(merged.key[j]);
    double my_prob;
    RowFinal f = finish_row_warp(merged, job.c1, neg_refc, centered, my_x, my_prob);
    f.pmax = __shfl_sync(0xFFFFFFFFu, my_prob, 0);
    const double p_next = __shfl_sync(0xFFFFFFFFu, my_prob, 1);
    double p_listed[kMaxK];
#pragma unroll
    for (int j = 0; j < kMaxK; ++j) p_listed[j] = __shfl_sync(0xFFFFFFFFu, my_prob, 2 + j);
    if (lane_id != 0) return;
    const int KE = a.k_extra;
    int ids[kMaxK];
    float ps[kMaxK];
    int n = 0;
    for (int j = 0; j < kMaxK; ++j) {
        ids[j] = AASD_NONE;
        ps[j] = 0.f;
    }
    double pn = 0.0;
    bool aligned = false;
    if (!f.bad) {
        float xn = 0.f;
        if (next != AASD_NONE) {
            xn = xn_in;
            pn = p_next;
            aligned = (next == f.top1);
        }
        if (a.mode == AASD_ALIGN_GUMBEL) {
            // distinct draws other than the prompt's own token, in draw order
            for (int j = 0; j < KE && !aligned; ++j) {
                const int tok = draws[j];
                if (tok == AASD_NONE || tok == next) continue;
                bool dup = false;
                for (int q = 0; q < n; ++q) dup |= (ids[q] == tok);
                if (dup) continue;
                ids[n] = tok;
                ps[n] = (float)p_listed[j];
                ++n;
            }
        } else {
            // the listed tokens that rank above the next token (Fig. 2)
            for (int j = 0; j < KE; ++j) {
                const u64 k = merged.key[j];
                if (k == 0) break;
                const float xv = key_value(k);
                const int id = key_id(k);
                if (next == AASD_NONE || xv > xn || (xv == xn && id < next)) {
                    ids[n] = id;
                    ps[n] = (float)p_listed[j];
                    ++n;
                }
            }
        }
    }
    for (int j = 0; j < KE; ++j) {
        if (a.out.align_ids) a.out.align_ids[row * KE + j] = ids[j];
        if (a.out.align_p) a.out.align_p[row * KE + j] = ps[j];
    }
    if (a.out.n_extra) a.out.n_extra[row] = n;
    if (a.out.p_next) a.out.p_next[row] = (float)pn;
    if (a.out.top1) a.out.top1[row] = f.top1;
    if (a.out.entropy) a.out.entropy[row] = (float)f.H;
    if (a.out.pmax) a.out.pmax[row] = (float)f.pmax;
    if (a.out.aligned) a.out.aligned[row] = aligned ? 1 : 0;
    tally.rows += 1;
    if (f.bad) {
        tally.bad += 1;
        tally.status |= AASD_STATUS_BAD_ROW;
    }
}

// Entered by a whole warp with the draws already made (the same values in every lane).
template <int DT>
__device__ void align_finish_warp(const AlignArgs& a, const RowJob& job, int64_t row, const char* rowp,
                                  const RowPartial& merged, float neg_refc, bool centered, int next, float xn,
                                  const int (&draws)[kMaxK], Tally& tally) {
    float dx[kMaxK];
    for (int j = 0; j < kMaxK; ++j)
        dx[j] = (a.mode == AASD_ALIGN_GUMBEL && j < a.k_extra && draws[j] >= 0) ? Elt<DT>::load(rowp, draws[j]) : 0.f;
    align_row(a, job, row, merged, neg_refc, centered, next, xn, draws, dx, tally);
}

template <int DT, int K>
__global__ void __launch_bounds__(kThreads) align_kernel(const AlignArgs a) {
    __shared__ BlockScratch sc;
    pdl_launch_dependents();
    pdl_wait();
    const RowJob& job = a.job;
    const int64_t row = blockIdx.x / job.chunks;
    const int chunk = blockIdx.x % job.chunks;
    const char* rowp = row_pointer<DT>(job, row);
    const int next = __ldg(a.next_ids + row);
    float neg_refc;
    bool centered;
    if (!row_reduce<DT, K>(job, row, chunk, next, rowp, neg_refc, centered, sc)) return;
    if (threadIdx.x >= 32) return;
    const float xn = next != AASD_NONE ? Elt<DT>::load(rowp, next) : 0.f;
    Tally tally;
    tally.clear();
    int draws[kMaxK];
    for (int j = 0; j < kMaxK; ++j) draws[j] = AASD_NONE;
    if (align_wants_draws(a, sc.merged, next)) {
        // this layout takes the definition as it stands: every group scored in fp64
        for (int j = 0; j < a.k_extra; ++j) {
            draws[j] = warp_sample_exhaustive<DT>(rowp, job.vocab, (unsigned int)row, j, a.smp);
            tally.exhaustive += 1;
        }
    }
    align_finish_warp<DT>(a, job, row, rowp, sc.merged, neg_refc, centered, next, xn, draws, tally);
    if (threadIdx.x == 0) tally.flush(job.state);
}

}  // namespace aasd
