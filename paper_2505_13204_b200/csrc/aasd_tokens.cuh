// Integer kernels on token buffers: suffix-match drafting, candidate selection, append.
#pragma once

#include "aasd_device.cuh"

namespace aasd {

constexpr int kMaxCands = 64;   // candidates per sequence a draft call can emit
constexpr int kExtScan = 32;    // depths per main whose extra counts are fetched in parallel
constexpr int kDraftThreads = 1024;   // one CTA per sequence: long histories want many lanes
constexpr int kDraftThreadsBatch = 256;   // batches with more sequences than SMs: CTAs share an SM, and the
                                          // step is made of instructions every warp issues, so fewer warps each
constexpr int kHitWords = 128;        // places per window of the lookup = 32 * kHitWords
constexpr int kMatchBytes = 32768;    // histories up to this many tokens keep their match lengths in shared memory

struct DraftArgs {
    aasd_draft_in in;
    aasd_draft_params p;
    aasd_draft_out out;
    DeviceState* state;
};

// A place of the external pool in the lists of places (history places are >= 1).
__device__ __forceinline__ int pool_place(int p) { return -2 - p; }
__device__ __forceinline__ bool is_pool_place(int code) { return code <= -2; }
__device__ __forceinline__ int place_of(int code) { return code <= -2 ? -2 - code : code; }

// One CTA per sequence.  Every place p of the sequence's token buffer (the index right after a
// possible key occurrence, with a continuation behind it) is scored by the length of the common
// suffix of the tokens in front of it and the key; the places that reach the best length are
// the lookup result of Algorithm 1's dictionary for the longest key that has one (Sec. 3.1:
// longer keys first).  An external pool (a second token buffer shared by all sequences, NONE
// between its documents) is scored the same way and its places come after the sequence's own.
// The places are found in two sweeps: the best length (block-wide maximum), then one bit per
// place that reaches it, written by warp ballots into a bit field in shared memory (a window
// of 4096 places at a time, from the top down, until enough places are found) from which one
// warp reads the places off in descending order.  A history of more than one window whose
// lengths are all kept in shared memory takes one pass instead: a word of hit bits per thread,
// a block-wide count from the top down, and every thread writes its own places.
template <int NT>
__global__ void __launch_bounds__(NT) draft_kernel(const DraftArgs a) {
    constexpr int kWarps = NT / 32;
    __shared__ int s_rec[AASD_MAX_NGRAM];
    __shared__ int s_pos[kMaxCands];        // places of the mains (pool places encoded)
    __shared__ int s_len[kMaxCands];        // and how many tokens follow them
    __shared__ unsigned int s_hits[kHitWords];
    __shared__ __align__(16) unsigned char s_m[kMatchBytes];   // match length of every place of the history (short histories)
    __shared__ int s_count;
    __shared__ int s_kstar;
    __shared__ unsigned char s_next[kMaxCands * kExtScan];
    __shared__ int s_alt[kMaxCands];         // alternatives: (main << 16) | (extra slot << 12)
    __shared__ int s_alt_depth[kMaxCands];   // and their depth
    __shared__ int s_total;

    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.p.n, draft_len = a.p.draft_len, max_cands = a.p.max_cands, K = a.p.k_extra;
    const int32_t* h = a.in.hist_ids + a.in.hist_offsets[b];
    const int len = a.in.hist_len[b];
    const int plen = min(a.in.prompt_len[b], len);
    const bool have_align = a.in.align_ids != nullptr && a.in.align_n != nullptr && K > 0;
    const bool match_align = have_align && (a.p.flags & AASD_DRAFT_MATCH_ALIGN);
    const int64_t arow0 = have_align ? (int64_t)a.in.align_row_offsets[b] : 0;
    const int32_t* pool = a.in.pool_ids;
    const int pool_len = pool != nullptr ? a.in.pool_len : 0;
    const bool have_pool_align = pool_len > 0 && a.in.pool_align_ids != nullptr && a.in.pool_align_n != nullptr && K > 0;

    // The tokens in front of the first places each thread looks at do not depend on the key:
    // they are asked for together with it, so that both cross the memory system at once.
    constexpr int kBatch = 8;
    int front[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
        const int p = 1 + tid + u * NT;
        front[u] = p < len ? h[p - 1] : AASD_NONE;
    }
    int rl;
    if (a.in.recent_ids) {
        // (slot tid of the key is read whether it counts or not: one trip instead of two)
        const int slot = tid < n ? a.in.recent_ids[(int64_t)b * n + tid] : AASD_NONE;
        rl = max(0, min(n, a.in.recent_len[b]));
        if (tid < rl) s_rec[tid] = slot;
    } else {
        rl = min(n, len);
        if (tid < rl) s_rec[tid] = h[len - rl + tid];
    }
    if (tid == 0) {
        s_count = 0;
        s_kstar = 0;
        s_m[0] = 0;   // no place 0: the bit field below reads whole words
    }
    __syncthreads();

    auto n_ext = [&](int q) -> int {
        if (!have_align || q < 1 || q >= plen) return 0;
        return min(K, max(0, a.in.align_n[arow0 + q - 1]));
    };
    auto ext = [&](int q, int s) -> int { return a.in.align_ids[(arow0 + q - 1) * K + s]; };
    auto n_pool_ext = [&](int q) -> int {
        if (!have_pool_align || q < 1 || q >= pool_len) return 0;
        return min(K, max(0, a.in.pool_align_n[q - 1]));
    };
    auto pool_ext = [&](int q, int s) -> int { return a.in.pool_align_ids[(int64_t)(q - 1) * K + s]; };
    auto match_len_at = [&](int p) -> int {
        const int lim = min(min(n, p), rl);
        int m = 0;
        for (int j = 1; j <= lim; ++j) {
            const int q = p - j, want = s_rec[rl - j];
            bool ok = (h[q] == want);
            if (!ok && j == 1 && match_align) {
                const int ne = n_ext(q);
                for (int s = 0; s < ne; ++s) ok |= (ext(q, s) == want);
            }
            if (!ok) break;
            m = j;
        }
        return m;
    };
    // a place of the pool: NONE equals no key token (keys hold tokens, and a key slot that is
    // NONE must not match a document boundary), and a place on a boundary has no continuation
    auto pool_match_len_at = [&](int p) -> int {
        if (pool[p] == AASD_NONE) return 0;
        const int lim = min(min(n, p), rl);
        int m = 0;
        for (int j = 1; j <= lim; ++j) {
            const int t = pool[p - j];
            if (t == AASD_NONE || t != s_rec[rl - j]) break;
            m = j;
        }
        return m;
    };

    // sweep 1: the longest key that occurs at a place with a continuation (the lengths are kept
    // for sweep 2 when the history is short enough)
    const bool cached = len <= kMatchBytes;
    int best = 0;
    {
        // A place matches at all only if the token in front of it is the key's last one (or, with
        // the table, one of that position's extras): the tokens of eight places are fetched
        // together, so that their trips to memory overlap, and the full comparison runs for
        // the few places that pass this test.
        const int want_last = rl > 0 ? s_rec[rl - 1] : AASD_NONE;
        for (int base = 1 + tid; base < len; base += kBatch * NT) {
            if (base != 1 + tid) {
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int p = base + u * NT;
                    front[u] = p < len ? h[p - 1] : AASD_NONE;
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int p = base + u * NT;
                if (p >= len) break;
                const int m = (rl > 0 && (front[u] == want_last || match_align)) ? match_len_at(p) : 0;
                if (cached) s_m[p] = (unsigned char)m;
                best = max(best, m);
            }
        }
    }
    for (int p = 1 + tid; p < pool_len; p += NT) best = max(best, pool_match_len_at(p));
    best = __reduce_max_sync(0xFFFFFFFFu, best);
    if (lane == 0 && best > 0) atomicMax(&s_kstar, best);
    __syncthreads();
    const int kstar = s_kstar;

    // sweep 2: its places, the sequence's own first, most recent first within a source, in
    // windows of 32 * kHitWords places from the top down
    if (kstar > 0) {
        for (int src = 0; src < 2; ++src) {
            if (src == 0 && cached && len > 32 * kHitWords && len <= 32 * NT) {
                // (a history of a single window measured no slower by the windows below)
                // Every place's length is in shared memory: thread t turns places 32 t .. 32 t + 31
                // into a word of hit bits (byte compares, four at a time), a block-wide count
                // from the top down gives each word the rank of its highest place, and the
                // threads whose places rank among the first max_cands write them: one barrier,
                // whatever the history's length.
                const int lo = 32 * tid;
                unsigned int bits = 0;
                if (lo < len) {
                    const uint4* src16 = reinterpret_cast<const uint4*>(s_m + lo);
                    const uint4 q0 = src16[0], q1 = src16[1];
                    const unsigned int w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
                    const unsigned int want = 0x01010101u * (unsigned int)kstar;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const unsigned int eq = (__vcmpeq4(w[i], want) >> 7) & 0x01010101u;   // bit 0 of each equal byte
                        bits |= ((eq * 0x01020408u) >> 24 & 0xFu) << (4 * i);
                    }
                    const int valid = min(32, len - lo);
                    if (valid < 32) bits &= (1u << valid) - 1u;
                    if (tid == 0) bits &= ~1u;
                }
                const int mine = __popc(bits);
                int incl = mine;   // hits of this lane and of the lanes above it
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int dn = __shfl_down_sync(0xFFFFFFFFu, incl, o);
                    if (lane + o < 32) incl += dn;
                }
                if (lane == 0) s_hits[warp] = (unsigned int)incl;   // the warp's hits
                __syncthreads();
                const int others = lane < kWarps ? (int)s_hits[lane] : 0;
                const int above = __reduce_add_sync(0xFFFFFFFFu, lane > warp ? others : 0);
                const int all = __reduce_add_sync(0xFFFFFFFFu, others);
                int rank = above + incl - mine;
                unsigned int left = bits;
                while (left && rank < max_cands) {
                    const int bit = 31 - __clz(left);    // the highest place of the word first
                    left &= ~(1u << bit);
                    if (!AASD_IN_RANGE(rank >= 0 && rank < kMaxCands && lo + bit >= 1 && lo + bit < len, a.state)) break;
                    s_pos[rank++] = lo + bit;
                }
                if (tid == 0) s_count = min(all, max_cands);
                __syncthreads();
                continue;
            }
            const int top = src == 0 ? len : pool_len;     // places 1 .. top - 1
            for (int hi = top; hi > 1 && s_count < max_cands; hi -= 32 * kHitWords) {
                const int lo = max(1, hi - 32 * kHitWords);   // window [lo, hi)
                const int words = (hi - lo + 31) / 32;
                for (int wd = warp; wd < words; wd += kWarps) {
                    const int p = lo + wd * 32 + lane;
                    const bool hit = p < hi && (src == 0 ? (cached ? (int)s_m[p] : match_len_at(p)) : pool_match_len_at(p)) == kstar;
                    const unsigned int bal = __ballot_sync(0xFFFFFFFFu, hit);
                    if (lane == 0) s_hits[wd] = bal;
                }
                __syncthreads();
                if (warp == 0) {
                    int count = s_count;
                    for (int base = words - 1; base >= 0 && count < max_cands; base -= 32) {
                        const int wd = base - lane;              // lane 0 takes the highest word
                        const unsigned int bits = wd >= 0 ? s_hits[wd] : 0u;
                        const int mine = __popc(bits);
                        int incl = mine;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                            if (lane >= o) incl += up;
                        }
                        int rank = count + incl - mine;          // places of higher words come first
                        unsigned int left = bits;
                        while (left && rank < max_cands) {
                            const int bit = 31 - __clz(left);    // the highest place of the word first
                            left &= ~(1u << bit);
                            const int p = lo + wd * 32 + bit;
                            if (!AASD_IN_RANGE(rank >= 0 && rank < kMaxCands && p >= 1 && p < top && wd >= 0 && wd < kHitWords,
                                               a.state))
                                break;
                            s_pos[rank++] = src == 0 ? p : pool_place(p);
                        }
                        count += __shfl_sync(0xFFFFFFFFu, incl, 31);
                    }
                    if (lane == 0) s_count = min(count, max_cands);
                }
                __syncthreads();
            }
        }
    }
    const int n_main = min(s_count, max_cands);

    int32_t* d_ids = a.out.draft_ids + (int64_t)b * max_cands * draft_len;
    uint8_t* d_fl = a.out.draft_flags + (int64_t)b * max_cands * draft_len;
    int32_t* c_len = a.out.cand_len + (int64_t)b * max_cands;
    int32_t* c_pos = a.out.cand_pos + (int64_t)b * max_cands;
    // how many tokens follow each main: up to draft_len, to the end of its buffer, and in the
    // pool to the end of the document
    for (int c = tid; c < n_main; c += NT) {
        const int code = s_pos[c], p = place_of(code);
        int L;
        if (!is_pool_place(code)) {
            L = min(draft_len, len - p);
        } else {
            L = 0;
            while (L < draft_len && p + L < pool_len && pool[p + L] != AASD_NONE) ++L;
        }
        s_len[c] = L;
    }
    __syncthreads();
    for (int i = tid; i < max_cands * draft_len; i += NT) {
        const int c = i / draft_len, j = i % draft_len;
        int tok = AASD_NONE;
        unsigned int fl = 0;
        if (c < n_main && j < s_len[c]) {
            const int code = s_pos[c], q = place_of(code) + j;
            if (!AASD_IN_RANGE(q >= 0 && q < (is_pool_place(code) ? pool_len : len), a.state)) continue;
            if (!is_pool_place(code)) {
                tok = h[q];
                fl = (q < plen) ? AASD_FLAG_CONDITIONAL : 0u;
            } else {
                tok = pool[q];      // not input context: verified strictly
            }
        }
        d_ids[i] = tok;
        d_fl[i] = (uint8_t)fl;
    }
    for (int c = tid; c < max_cands; c += NT) {
        c_len[c] = c < n_main ? s_len[c] : 0;
        c_pos[c] = c < n_main ? s_pos[c] : AASD_NONE;
    }
    // how many extras each (main, depth) has: fetched by all threads at once, so that the
    // serial walk below does not pay a trip to memory per step
    const bool any_table = have_align || have_pool_align;
    const int scan = min(draft_len, kExtScan);
    auto extras_at = [&](int c, int depth) -> int {
        const int code = s_pos[c], q = place_of(code) + depth;
        return is_pool_place(code) ? n_pool_ext(q) : n_ext(q);
    };
    if (any_table && n_main < max_cands) {
        for (int i = tid; i < n_main * scan; i += NT) {
            const int c = i / scan, depth = i % scan;
            s_next[c * kExtScan + depth] = (unsigned char)(depth < s_len[c] ? extras_at(c, depth) : 0);
        }
    }
    __syncthreads();

    // alternatives: a main's prefix plus one alignment-sampled token (Sec. 3.2), in
    // (main, depth, extra slot) order while slots remain.  One thread lays the list out from
    // the counts in shared memory; all threads then write the tokens.
    if (tid == 0) {
        int total = n_main;
        for (int c = 0; c < n_main && total < max_cands && any_table; ++c) {
            const int L = s_len[c];
            for (int i = 0; i < L && total < max_cands; ++i) {
                const int ne = i < scan ? (int)s_next[c * kExtScan + i] : extras_at(c, i);
                for (int s = 0; s < ne && total < max_cands; ++s) {
                    s_alt[total] = (c << 16) | (s << 12) | 0;   // main and extra slot; the depth goes beside
                    s_alt_depth[total] = i;
                    ++total;
                }
            }
        }
        s_total = total;
        a.out.n_cands[b] = total;
        a.out.match_len[b] = kstar;
    }
    __syncthreads();
    const int total = s_total;
    for (int i = tid; i < (total - n_main) * draft_len; i += NT) {
        const int slot = n_main + i / draft_len, q = i % draft_len;
        const int c = s_alt[slot] >> 16, es = (s_alt[slot] >> 12) & 15, depth = s_alt_depth[slot];
        const int code = s_pos[c], p = place_of(code);
        const bool from_pool = is_pool_place(code);
        if (q < depth) {
            d_ids[slot * draft_len + q] = from_pool ? pool[p + q] : h[p + q];
            d_fl[slot * draft_len + q] = (uint8_t)((!from_pool && p + q < plen) ? AASD_FLAG_CONDITIONAL : 0u);
        } else if (q == depth) {
            d_ids[slot * draft_len + q] = from_pool ? pool_ext(p + depth, es) : ext(p + depth, es);
            d_fl[slot * draft_len + q] = (uint8_t)(AASD_FLAG_CONDITIONAL | AASD_FLAG_EXTRA);
            c_len[slot] = depth + 1;
            c_pos[slot] = code;
        }
    }
}

// Read-only stream over a buffer (measurement aid): every 16-byte word is loaded once.
__global__ void __launch_bounds__(256) probe_read_kernel(const uint4* __restrict__ p, size_t n, unsigned int* sink) {
    pdl_launch_dependents();
    pdl_wait();
    unsigned int acc = 0;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t st = (size_t)gridDim.x * blockDim.x;
    for (; i + 3 * st < n; i += 4 * st) {
        const uint4 a = load_stream16(p + i), b = load_stream16(p + i + st), c = load_stream16(p + i + 2 * st),
                    d = load_stream16(p + i + 3 * st);
        acc += a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
    }
    for (; i < n; i += st) {
        const uint4 a = load_stream16(p + i);
        acc += a.x ^ a.y ^ a.z ^ a.w;
    }
    if (acc == 0x9E3779B9u) atomicAdd(sink, acc);   // keeps the loads alive, practically never taken
}

struct SelectArgs {
    const int32_t* accept_len;
    const int32_t* next_token;
    const int32_t* draft_ids;
    const int32_t* cand_offsets;
    int rows_per_cand;
    const int32_t* seq_cand_offsets;
    int cands_per_seq;
    int n_seqs;
    int emit_stride;
    int32_t* best_cand;
    int32_t* n_emit;
    int32_t* emit_ids;
};

// Longest passing candidate per sequence (Sec. 3.3), ties to the lowest index.
__global__ void select_kernel(const SelectArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= a.n_seqs) return;
    const int lo = a.seq_cand_offsets ? a.seq_cand_offsets[b] : b * a.cands_per_seq;
    const int hi = a.seq_cand_offsets ? a.seq_cand_offsets[b + 1] : lo + a.cands_per_seq;
    int best = AASD_NONE, best_a = -1;
    for (int c = lo; c < hi; ++c) {
        const int v = a.accept_len[c];
        if (v > best_a) {
            best_a = v;
            best = c;
        }
    }
    int32_t* e = a.emit_ids + (int64_t)b * a.emit_stride;
    int ne = 0;
    if (best != AASD_NONE) {
        const int64_t d0 = a.cand_offsets ? (int64_t)a.cand_offsets[best] : (int64_t)best * a.rows_per_cand;
        for (int i = 0; i < best_a && ne < a.emit_stride; ++i) e[ne++] = a.draft_ids[d0 + i];
        const int nt = a.next_token[best];
        if (nt != AASD_NONE && ne < a.emit_stride) e[ne++] = nt;
    }
    for (int i = ne; i < a.emit_stride; ++i) e[i] = AASD_NONE;
    a.best_cand[b] = best;
    a.n_emit[b] = ne;
}

struct AppendArgs {
    int32_t* hist_ids;
    const int32_t* hist_offsets;
    int32_t* hist_len;
    const int32_t* emit_ids;
    const int32_t* n_emit;
    int n_seqs;
    int emit_stride;
    DeviceState* state;
};

// q <- q + y (Algorithm 1), in place, clipped at the buffer's capacity.
__global__ void append_kernel(const AppendArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= a.n_seqs) return;
    const int off = a.hist_offsets[b];
    const int cap = a.hist_offsets[b + 1] - off;
    int len = a.hist_len[b];
    const int ne = min(a.n_emit[b], a.emit_stride);
    for (int i = 0; i < ne; ++i) {
        if (len >= cap) {
            atomicOr(&a.state->status, AASD_STATUS_HIST_OVERFLOW);
            break;
        }
        a.hist_ids[off + len] = a.emit_ids[(int64_t)b * a.emit_stride + i];
        ++len;
    }
    a.hist_len[b] = len;
}

}  // namespace aasd
