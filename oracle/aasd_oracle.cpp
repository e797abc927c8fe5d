// CPU oracle for the AASD draft-and-verify path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision statement of
// what the method computes, written from the paper (Alignment-Augmented Speculative
// Decoding: alignment sampling, context-aware drafting, conditional verification).  Only
// the tests, the smoke check and the benchmark's cpu_baseline / reference legs may call
// it.  It shares no code, header, table or constant generator with the CUDA path.
//
// Every floating-point quantity is computed in IEEE double with libm exp/log; fp32 and
// bf16 inputs are widened exactly.  There is no blocking or reordering beyond the
// definitions: sums run over the vocabulary in index order.
//
// Pins (tests/test_oracle_*.py): closed forms of softmax/entropy (uniform, one spike,
// (1/2,1/4,1/8,1/8)), hand-computed thresholds of Eq. 5, the worked alignment examples of
// Sec. 2.3 and Fig. 2, brute-force sorts and 2^len accept patterns on tiny inputs, a
// dictionary of Algorithm 1 and a naive double loop for the lookup, published Philox4x32-10 known-answer
// vectors and a chi-square test of the sampler against the exact softmax; top-k verification
// against a full stable sort and the two extreme rows of Sec. 3.3; the draft tree against the
// set of distinct candidate prefixes, tree verification against the longest passing flat
// candidate over all root-to-leaf paths and against plain sampled decoding along the tree.
// Parity unpinned: the end-to-end mean acceptance length of the closed-loop driver (it
// is a statistic of the synthetic inputs; the paper's figures need its datasets and
// model weights).
//
// Build: g++ -O2 -std=c++17 -fopenmp -shared -fPIC aasd_oracle.cpp -o liboracle.so
// (-O2 without -ffast-math: no reassociation, no contraction that changes results
// beyond what IEEE double already allows).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <map>
#include <vector>

namespace {

constexpr int32_t NONE = -1;

// ---------------------------------------------------------------------------------
// Input widening.  dtype 0 = IEEE fp32, dtype 1 = bfloat16 stored as raw uint16
// (bfloat16 is the upper half of an fp32 bit pattern).
// ---------------------------------------------------------------------------------
struct Rows {
    const void* base;
    int dtype;
    int64_t row_stride;  // in elements
    double at(int64_t row, int64_t i) const {
        int64_t off = row * row_stride + i;
        if (dtype == 0) {
            return (double)static_cast<const float*>(base)[off];
        }
        uint32_t bits = (uint32_t)static_cast<const uint16_t*>(base)[off] << 16;
        float f;
        std::memcpy(&f, &bits, 4);
        return (double)f;
    }
};

// ---------------------------------------------------------------------------------
// O-R: per-row statistics (Eq. 5 and Eq. 6).
//   y_i = x_i * invT, m = max y, argmax = lowest id attaining m,
//   S = sum exp(y_i - m), p_i = exp(y_i - m)/S, Delta = max_i p_i = 1/S,
//   H = -sum p_i ln p_i (0 ln 0 := 0) = ln S - (sum e^{y_i-m}(y_i-m))/S   [nats].
// A row holding NaN or +inf, or nothing but -inf, is "bad".
// ---------------------------------------------------------------------------------
struct RowStats {
    bool bad;
    double m;
    int32_t argmax;
    double S;
    double H;
    double pmax;
};

RowStats row_stats(const Rows& X, int64_t row, int64_t V, double invT) {
    RowStats r{};
    r.bad = false;
    r.m = -std::numeric_limits<double>::infinity();
    r.argmax = NONE;
    for (int64_t i = 0; i < V; ++i) {
        double y = X.at(row, i) * invT;
        if (std::isnan(y) || y == std::numeric_limits<double>::infinity()) r.bad = true;
        if (y > r.m) {
            r.m = y;
            r.argmax = (int32_t)i;
        }
    }
    if (r.argmax == NONE) r.bad = true;  // every entry was -inf (or V == 0)
    if (r.bad) {
        r.m = 0;
        r.argmax = NONE;
        r.S = 0;
        r.H = 0;
        r.pmax = 0;
        return r;
    }
    double S = 0.0, A = 0.0;
    for (int64_t i = 0; i < V; ++i) {
        double t = X.at(row, i) * invT - r.m;
        if (t == -std::numeric_limits<double>::infinity()) continue;  // p = 0, 0 ln 0 = 0
        double e = std::exp(t);
        S += e;
        A += e * t;
    }
    r.S = S;
    r.H = std::log(S) - A / S;
    r.pmax = 1.0 / S;
    return r;
}

inline double prob_of(const Rows& X, int64_t row, int64_t id, double invT, const RowStats& r) {
    return std::exp(X.at(row, id) * invT - r.m) / r.S;
}

// Total order on the tokens of a row: larger logit first, equal logits by lower id.
inline bool ahead(double ya, int64_t ia, double yb, int64_t ib) {
    return ya > yb || (ya == yb && ia < ib);
}

// ---------------------------------------------------------------------------------
// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
// easy as 1, 2, 3", SC'11), the oracle's own copy.
// ---------------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    uint32_t c[4] = {ctr_in[0], ctr_in[1], ctr_in[2], ctr_in[3]};
    uint32_t k[2] = {key_in[0], key_in[1]};
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k[0] += 0x9E3779B9u;
            k[1] += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k[0];
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k[1];
        uint32_t n3 = (uint32_t)p0;
        c[0] = n0;
        c[1] = n1;
        c[2] = n2;
        c[3] = n3;
    }
    for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// 32-bit word -> open-interval uniform -> standard Gumbel variate.
inline double gumbel_of(uint32_t r) {
    double u = ((double)r + 0.5) * (1.0 / 4294967296.0);
    return -std::log(-std::log(u));
}

// Counter domains: which call and which stage of the sampler a word belongs to.
enum : uint32_t {
    DOM_ALIGN_GROUP = 2,
    DOM_ALIGN_ELEM = 3,
    DOM_VERIFY_GROUP = 4,
    DOM_VERIFY_ELEM = 5,
};

constexpr int64_t GROUP = 32;

// ---------------------------------------------------------------------------------
// O-S: hierarchical Gumbel-max sampler, an exact sampler of softmax(y).
// The vocabulary is cut into groups of 32 consecutive ids.  Group stage: every group g
// gets the score Lambda_g + G, Lambda_g = ln sum_{i in g} e^{y_i}; the best score wins
// (ties: lowest g).  Element stage inside the winning group: score y_i + G', best wins
// (ties: lowest id).  By max-stability of the Gumbel law the winner is distributed as
// softmax(y).  Draw j (0 <= j < 4) uses word j of the Philox output, so up to four draws
// share the same counters:
//   group words   = philox(ctr = (g, row, step, domain_group), key = seed)
//   element words = philox(ctr = (i, row, step, domain_elem ), key = seed)
// ---------------------------------------------------------------------------------
int32_t sample_row(const Rows& X, int64_t row, int64_t V, double invT, uint64_t seed,
                   uint32_t row_ctr, uint32_t step, uint32_t dom_group, uint32_t dom_elem,
                   int draw) {
    const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    const double NEG_INF = -std::numeric_limits<double>::infinity();
    int64_t n_groups = (V + GROUP - 1) / GROUP;
    double best = NEG_INF;
    int64_t best_g = -1;
    for (int64_t g = 0; g < n_groups; ++g) {
        int64_t lo = g * GROUP, hi = std::min(V, lo + GROUP);
        double gm = NEG_INF;
        for (int64_t i = lo; i < hi; ++i) gm = std::max(gm, X.at(row, i) * invT);
        if (gm == NEG_INF) continue;  // empty group: probability 0
        double s = 0.0;
        for (int64_t i = lo; i < hi; ++i) s += std::exp(X.at(row, i) * invT - gm);
        double lambda = gm + std::log(s);
        uint32_t ctr[4] = {(uint32_t)g, row_ctr, step, dom_group};
        uint32_t w[4];
        philox4x32_10(ctr, key, w);
        double score = lambda + gumbel_of(w[draw]);
        if (score > best) {
            best = score;
            best_g = g;
        }
    }
    if (best_g < 0) return NONE;
    int64_t lo = best_g * GROUP, hi = std::min(V, lo + GROUP);
    double ebest = NEG_INF;
    int32_t winner = NONE;
    for (int64_t i = lo; i < hi; ++i) {
        double y = X.at(row, i) * invT;
        if (y == NEG_INF) continue;
        uint32_t ctr[4] = {(uint32_t)i, row_ctr, step, dom_elem};
        uint32_t w[4];
        philox4x32_10(ctr, key, w);
        double score = y + gumbel_of(w[draw]);
        if (score > ebest) {
            ebest = score;
            winner = (int32_t)i;
        }
    }
    return winner;
}

}  // namespace

extern "C" {

// Raw generator access for the known-answer pins.
void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

double oracle_gumbel_of(uint32_t r) { return gumbel_of(r); }

// Row statistics of R rows (Eq. 5-6).  Outputs have R entries; any may be NULL.
void oracle_row_stats(const void* logits, int dtype, int64_t R, int64_t V, int64_t row_stride,
                      double invT, int threads, double* m, int32_t* argmax, double* S,
                      double* H, double* pmax, uint8_t* bad) {
    Rows X{logits, dtype, row_stride};
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
    for (int64_t r = 0; r < R; ++r) {
        RowStats st = row_stats(X, r, V, invT);
        if (m) m[r] = st.m;
        if (argmax) argmax[r] = st.argmax;
        if (S) S[r] = st.S;
        if (H) H[r] = st.H;
        if (pmax) pmax[r] = st.pmax;
        if (bad) bad[r] = st.bad ? 1 : 0;
    }
}

// Full softmax of one row (for the brute-force pins only).
void oracle_softmax_row(const void* logits, int dtype, int64_t row, int64_t V,
                        int64_t row_stride, double invT, double* p_out) {
    Rows X{logits, dtype, row_stride};
    RowStats st = row_stats(X, row, V, invT);
    for (int64_t i = 0; i < V; ++i) p_out[i] = st.bad ? 0.0 : prob_of(X, row, i, invT, st);
}

// One draw of the sampler O-S (for the distribution pins).  kind: 0 = align, 1 = verify.
int32_t oracle_sample_row(const void* logits, int dtype, int64_t row, int64_t V,
                          int64_t row_stride, double invT, uint64_t seed, uint32_t row_ctr,
                          uint32_t step, int kind, int draw) {
    Rows X{logits, dtype, row_stride};
    return sample_row(X, row, V, invT, seed, row_ctr, step,
                      kind == 0 ? DOM_ALIGN_GROUP : DOM_VERIFY_GROUP,
                      kind == 0 ? DOM_ALIGN_ELEM : DOM_VERIFY_ELEM, draw);
}

// ---------------------------------------------------------------------------------
// O-A: alignment sampling over prefill logits (Sec. 2.3, Sec. 3.2, Fig. 2).
// Row t of a sequence holds the distribution of the token that follows prompt token t,
// so next_t = prompt[t+1] (NONE for the last row of a sequence).  The prompt token is
// "aligned" iff it equals the greedy choice of its row.
// mode 0 (TOPK): the extras of row t are those of the row's K best tokens that are ahead
//   of next_t in the order (logit desc, id asc): n_extra = min(rank(next_t), K); all K
//   when next_t is NONE.
// mode 1 (GUMBEL): aligned rows get none; otherwise K draws j = 0..K-1 of the sampler
//   (counters: row = global row index, step = stream_tag), keeping the distinct values
//   different from next_t in draw order.
// Outputs (any may be NULL): align_ids [rows x K] (NONE padded), align_p [rows x K]
// (0 padded), n_extra, p_next (0 when next is NONE), top1, entropy, pmax, aligned, bad.
// ---------------------------------------------------------------------------------
int oracle_align_sample(const void* logits, int dtype, const int32_t* prompt_ids,
                        const int32_t* seq_offsets, int32_t B, int64_t V, int64_t row_stride,
                        double invT, int K, int mode, uint64_t seed, uint32_t stream_tag,
                        int threads, int32_t* align_ids, double* align_p, int32_t* n_extra,
                        double* p_next, int32_t* top1, double* entropy, double* pmax,
                        uint8_t* aligned, uint8_t* bad) {
    if (K < 0 || K > 4 || B < 0 || V <= 0) return 1;
    Rows X{logits, dtype, row_stride};
    for (int32_t b = 0; b < B; ++b) {
        int64_t lo = seq_offsets[b], hi = seq_offsets[b + 1];
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
        for (int64_t t = lo; t < hi; ++t) {
            RowStats st = row_stats(X, t, V, invT);
            int32_t next = (t + 1 < hi) ? prompt_ids[t + 1] : NONE;
            if (next < 0 || next >= V) next = NONE;
            int32_t ids[4] = {NONE, NONE, NONE, NONE};
            double ps[4] = {0, 0, 0, 0};
            int n = 0;
            bool is_aligned = false;
            double pn = 0.0;
            if (!st.bad) {
                is_aligned = (next != NONE && next == st.argmax);
                if (next != NONE) pn = prob_of(X, t, next, invT, st);
                if (mode == 0) {
                    // K best tokens by repeated selection under the total order.
                    int32_t best[4] = {NONE, NONE, NONE, NONE};
                    for (int k = 0; k < K; ++k) {
                        int64_t pick = -1;
                        double py = 0;
                        for (int64_t i = 0; i < V; ++i) {
                            bool taken = false;
                            for (int q = 0; q < k; ++q) taken |= (best[q] == (int32_t)i);
                            if (taken) continue;
                            double y = X.at(t, i) * invT;
                            // a masked token (probability 0) cannot be drawn from the
                            // distribution, so it is never an extra
                            if (y == -std::numeric_limits<double>::infinity()) continue;
                            if (pick < 0 || ahead(y, i, py, pick)) {
                                pick = i;
                                py = y;
                            }
                        }
                        best[k] = (int32_t)pick;
                    }
                    double yn = (next != NONE) ? X.at(t, next) * invT : 0.0;
                    for (int k = 0; k < K; ++k) {
                        if (best[k] == NONE) break;
                        double yk = X.at(t, best[k]) * invT;
                        if (next == NONE || ahead(yk, best[k], yn, next)) {
                            ids[n] = best[k];
                            ps[n] = prob_of(X, t, best[k], invT, st);
                            ++n;
                        }
                    }
                } else if (!is_aligned) {
                    for (int j = 0; j < K; ++j) {
                        int32_t tok = sample_row(X, t, V, invT, seed, (uint32_t)t, stream_tag,
                                                 DOM_ALIGN_GROUP, DOM_ALIGN_ELEM, j);
                        if (tok == NONE || tok == next) continue;
                        bool dup = false;
                        for (int q = 0; q < n; ++q) dup |= (ids[q] == tok);
                        if (dup) continue;
                        ids[n] = tok;
                        ps[n] = prob_of(X, t, tok, invT, st);
                        ++n;
                    }
                }
            }
            for (int k = 0; k < K; ++k) {
                if (align_ids) align_ids[t * K + k] = ids[k];
                if (align_p) align_p[t * K + k] = ps[k];
            }
            if (n_extra) n_extra[t] = n;
            if (p_next) p_next[t] = pn;
            if (top1) top1[t] = st.argmax;
            if (entropy) entropy[t] = st.H;
            if (pmax) pmax[t] = st.pmax;
            if (aligned) aligned[t] = is_aligned ? 1 : 0;
            if (bad) bad[t] = st.bad ? 1 : 0;
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------------
// O-D: context-aware drafting (Sec. 3.1, Algorithm 1).
// The draft pool of Algorithm 1 holds, for every k-gram (k <= n) of the current sequence, the
// places right after its occurrences; the lookup tries the last k tokens of the sequence as
// the key for k = n, n-1, ..., 1 and stops at the first k that has a place (Sec. 3.1: longer
// keys first).  Written out as a definition: the match length of a place p (an index into the
// token sequence, 1 <= p < len, so that a continuation exists) is the largest k <= min(n, p,
// recent_len) such that the k tokens in front of p equal the key's last k tokens; k* is the
// largest match length of any place, and the lookup result is every place that reaches it.
// With match_align != 0 the token right in front of p may also be one of the alignment
// extras stored for that prompt position (extras of position q live in align row q-1).
// An external pool (Limitations: "most existing retrieval-based speculative decoding") is a
// second token sequence, shared by all sequences and owned by the caller, that is looked up
// the same way: its places compete with the history's for k*, a NONE token inside it separates
// documents (it matches nothing and ends a continuation), and its tokens are not input
// context, so they are verified strictly (flag 0).  The pool may carry an alignment table of
// its own (extras of pool position q in row q-1): those extras are alignment-sampled tokens
// like any other (flags 3).
// Candidates: the places of the history in descending order, then those of the pool in
// descending order, at most max_cands ("mains"), each continued by up to draft_len tokens of
// its source; then, while slots remain, alternatives in (main, depth i, extra slot s) order =
// the main's first i tokens plus extra s of position p+i.  Token flags: bit0 = eligible for
// conditional verification (history index < prompt_len, or an alignment extra), bit1 =
// alignment extra.
// Outputs per sequence b: draft_ids/draft_flags [max_cands x draft_len] (NONE / 0 padded),
// cand_len, cand_pos (place of the main a candidate derives from: p for the history,
// -2 - p for the pool; NONE for unused slots) [max_cands], n_cands, match_len (k*, 0 when
// nothing matched).
// ---------------------------------------------------------------------------------
int oracle_draft(const int32_t* hist_ids, const int32_t* hist_offsets, const int32_t* hist_len,
                 const int32_t* prompt_len, const int32_t* align_ids, const int32_t* align_n,
                 const int32_t* align_row_offsets, int K, const int32_t* recent_ids,
                 const int32_t* recent_len, int32_t B, int n, int draft_len, int max_cands,
                 int match_align, const int32_t* pool_ids, int32_t pool_len,
                 const int32_t* pool_align_ids, const int32_t* pool_align_n, int32_t* draft_ids,
                 uint8_t* draft_flags, int32_t* cand_len, int32_t* cand_pos, int32_t* n_cands,
                 int32_t* match_len) {
    if (n < 1 || draft_len < 1 || max_cands < 1 || B < 0 || pool_len < 0) return 1;
    const bool have_align = (align_ids != nullptr && align_n != nullptr && K > 0);
    const bool have_pool = (pool_ids != nullptr && pool_len > 0);
    const bool have_pool_align = have_pool && pool_align_ids != nullptr && pool_align_n != nullptr && K > 0;
    for (int32_t b = 0; b < B; ++b) {
        const int32_t* h = hist_ids + hist_offsets[b];
        const int32_t len = hist_len[b];
        const int32_t plen = prompt_len[b];
        const int32_t* rec = recent_ids + (int64_t)b * n;
        const int32_t rl = std::max<int32_t>(0, std::min<int32_t>(n, recent_len[b]));
        const int64_t arow0 = have_align ? (int64_t)align_row_offsets[b] : 0;
        // extras stored for prompt position q / pool position q
        auto n_ext = [&](int32_t q) -> int {
            if (!have_align || q < 1 || q >= plen) return 0;
            return align_n[arow0 + q - 1];
        };
        auto ext = [&](int32_t q, int s) -> int32_t { return align_ids[(arow0 + q - 1) * K + s]; };
        auto n_pool_ext = [&](int32_t q) -> int {
            if (!have_pool_align || q < 1 || q >= pool_len) return 0;
            return pool_align_n[q - 1];
        };
        auto pool_ext = [&](int32_t q, int s) -> int32_t { return pool_align_ids[(int64_t)(q - 1) * K + s]; };
        // match length of place p of the history
        auto hist_match = [&](int32_t p) -> int {
            int m = 0;
            for (int k = 1; k <= std::min<int>(std::min<int>(n, p), rl); ++k) {
                const int32_t q = p - k, want = rec[rl - k];
                bool same = (h[q] == want);
                if (!same && k == 1 && match_align)
                    for (int s = 0; s < n_ext(q); ++s) same |= (ext(q, s) == want);
                if (!same) break;
                m = k;
            }
            return m;
        };
        // and of place p of the pool (NONE separates documents: it equals no key token)
        auto pool_match = [&](int32_t p) -> int {
            int m = 0;
            for (int k = 1; k <= std::min<int>(std::min<int>(n, p), rl); ++k) {
                const int32_t t = pool_ids[p - k];
                if (t == NONE || t != rec[rl - k]) break;
                m = k;
            }
            return m;
        };
        int kstar = 0;
        for (int32_t p = 1; p < len; ++p) kstar = std::max(kstar, hist_match(p));
        if (have_pool)
            for (int32_t p = 1; p < pool_len; ++p)
                if (pool_ids[p] != NONE) kstar = std::max(kstar, pool_match(p));
        // places that reach k*: (source, p), history first, most recent first within a source
        std::vector<std::pair<int, int32_t>> found;
        if (kstar > 0) {
            for (int32_t p = len - 1; p >= 1; --p)
                if (hist_match(p) == kstar) found.push_back({0, p});
            if (have_pool)
                for (int32_t p = pool_len - 1; p >= 1; --p)
                    if (pool_ids[p] != NONE && pool_match(p) == kstar) found.push_back({1, p});
        }

        int32_t* d_ids = draft_ids + (int64_t)b * max_cands * draft_len;
        uint8_t* d_fl = draft_flags + (int64_t)b * max_cands * draft_len;
        int32_t* c_len = cand_len + (int64_t)b * max_cands;
        int32_t* c_pos = cand_pos + (int64_t)b * max_cands;
        for (int64_t i = 0; i < (int64_t)max_cands * draft_len; ++i) {
            d_ids[i] = NONE;
            d_fl[i] = 0;
        }
        for (int c = 0; c < max_cands; ++c) {
            c_len[c] = 0;
            c_pos[c] = NONE;
        }
        const int n_main = std::min<int>((int)found.size(), max_cands);
        int total = 0;
        for (int c = 0; c < n_main; ++c) {
            const bool from_pool = found[c].first == 1;
            const int32_t p = found[c].second;
            int32_t L = 0;
            if (!from_pool) {
                L = std::min<int32_t>(draft_len, len - p);
                for (int32_t i = 0; i < L; ++i) {
                    d_ids[c * draft_len + i] = h[p + i];
                    d_fl[c * draft_len + i] = (p + i < plen) ? 1 : 0;
                }
            } else {
                while (L < draft_len && p + L < pool_len && pool_ids[p + L] != NONE) {
                    d_ids[c * draft_len + L] = pool_ids[p + L];
                    d_fl[c * draft_len + L] = 0;
                    ++L;
                }
            }
            c_len[c] = L;
            c_pos[c] = from_pool ? -2 - p : p;
            ++total;
        }
        for (int c = 0; c < n_main && total < max_cands; ++c) {
            const bool from_pool = found[c].first == 1;
            const int32_t p = found[c].second;
            for (int32_t i = 0; i < c_len[c] && total < max_cands; ++i) {
                const int ne = from_pool ? n_pool_ext(p + i) : n_ext(p + i);
                for (int s = 0; s < ne && total < max_cands; ++s) {
                    int slot = total++;
                    for (int32_t q = 0; q < i; ++q) {
                        d_ids[slot * draft_len + q] = d_ids[c * draft_len + q];
                        d_fl[slot * draft_len + q] = d_fl[c * draft_len + q];
                    }
                    d_ids[slot * draft_len + i] = from_pool ? pool_ext(p + i, s) : ext(p + i, s);
                    d_fl[slot * draft_len + i] = 3;
                    c_len[slot] = i + 1;
                    c_pos[slot] = c_pos[c];
                }
            }
        }
        n_cands[b] = total;
        match_len[b] = kstar;
    }
    return 0;
}

// ---------------------------------------------------------------------------------
// O-V: verification of draft rows (Eq. 3-6, prefix rule of Sec. 2.1, Sec. 3.3).
// Row r carries a draft id d and a flag byte f (flags == NULL: every row conditional).
//   d == NONE (or outside the vocabulary)      -> reject
//   mode 0 CONDITIONAL and f.bit0              -> delta = min(alpha*H + beta, Delta);
//        accept iff p_d >= delta, evaluated as (y_d == m) or (p_d >= alpha*H + beta)
//   otherwise strict: accept iff d == the target's own token of that row, which is the
//        argmax (modes 0 and 1 STRICT_GREEDY) or the row's sampled token (mode 2
//        STRICT_SAMPLED: draw 0 of the sampler, counters row = r, step = step).
//   mode 3 TOP_K (the alternative the paper argues against in Sec. 3.3 and ablates with
//        k = 5 in Sec. 4.4) and f.bit0 -> accept iff fewer than top_k tokens are ahead of d
//        in the order (logit desc, id asc), i.e. d is one of the row's top_k tokens; a
//        token of probability 0 (logit -inf) never passes; tokens without f.bit0 strict
//        greedy as in mode 0.
// n_greater[r] = number of tokens ahead of d in that order (NONE when d is NONE or masked).
// Candidates are CSR ranges of rows (cand_offsets[C+1]); accept_len = number of leading
// accepted rows; next_token = the target's own token of row accept_len when that row
// exists, else NONE.  near[r] = 1 when a conditional decision has
// |p_d - (alpha*H+beta)| <= 1e-6 and the Delta clause does not decide it.
// ---------------------------------------------------------------------------------
int oracle_verify(const void* logits, int dtype, const int32_t* draft_ids,
                  const uint8_t* draft_flags, const int32_t* cand_offsets, int32_t C, int64_t V,
                  int64_t row_stride, double alpha, double beta, double invT, int mode,
                  uint64_t seed, uint32_t step, int top_k, int threads, double* p_draft,
                  double* entropy, double* pmax, int32_t* argmax, double* threshold, uint8_t* accept,
                  int32_t* sampled, uint8_t* near, uint8_t* bad, int32_t* n_greater,
                  int32_t* accept_len, int32_t* next_token) {
    if (C < 0 || V <= 0 || mode < 0 || mode > 3) return 1;
    Rows X{logits, dtype, row_stride};
    const int64_t R = cand_offsets[C];
    std::vector<uint8_t> acc(R, 0);
    std::vector<int32_t> own(R, NONE);
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
    for (int64_t r = 0; r < R; ++r) {
        RowStats st = row_stats(X, r, V, invT);
        int32_t d = draft_ids[r];
        if (d < 0 || d >= V) d = NONE;
        uint8_t f = draft_flags ? draft_flags[r] : 1;
        double pd = 0.0, thr = 0.0;
        int32_t smp = NONE;
        bool a = false, is_near = false;
        int32_t ahead_of_d = NONE;
        if (!st.bad && d != NONE) {
            double yd = X.at(r, d) * invT;
            if (yd != -std::numeric_limits<double>::infinity()) {   // a masked token has no rank
                ahead_of_d = 0;
                for (int64_t i = 0; i < V; ++i)
                    if (i != d && ahead(X.at(r, i) * invT, i, yd, d)) ++ahead_of_d;
            }
        }
        if (!st.bad) {
            if (mode == 2)
                smp = sample_row(X, r, V, invT, seed, (uint32_t)r, step, DOM_VERIFY_GROUP,
                                 DOM_VERIFY_ELEM, 0);
            own[r] = (mode == 2) ? smp : st.argmax;
            double lin = alpha * st.H + beta;
            thr = std::min(lin, st.pmax);
            if (d != NONE) {
                pd = prob_of(X, r, d, invT, st);
                if (mode == 0 && (f & 1)) {
                    bool at_max = (X.at(r, d) * invT == st.m);
                    a = at_max || (pd >= lin);
                    is_near = !at_max && std::fabs(pd - lin) <= 1e-6;
                } else if (mode == 3 && (f & 1)) {
                    a = ahead_of_d != NONE && ahead_of_d < top_k;
                } else {
                    a = (d == own[r]);
                }
            }
        }
        acc[r] = a ? 1 : 0;
        if (p_draft) p_draft[r] = pd;
        if (entropy) entropy[r] = st.H;
        if (pmax) pmax[r] = st.pmax;
        if (argmax) argmax[r] = st.argmax;
        if (threshold) threshold[r] = thr;
        if (accept) accept[r] = acc[r];
        if (sampled) sampled[r] = smp;
        if (near) near[r] = is_near ? 1 : 0;
        if (bad) bad[r] = st.bad ? 1 : 0;
        if (n_greater) n_greater[r] = ahead_of_d;
    }
    for (int32_t c = 0; c < C; ++c) {
        int64_t lo = cand_offsets[c], hi = cand_offsets[c + 1];
        int32_t a = 0;
        while (lo + a < hi && acc[lo + a]) ++a;
        if (accept_len) accept_len[c] = a;
        if (next_token) next_token[c] = (lo + a < hi) ? own[lo + a] : NONE;
    }
    return 0;
}

// ---------------------------------------------------------------------------------
// O-T: the draft tree of Eq. 2 (Sec. 3.2): the candidate n-grams of a sequence, expanded
// by alignment sampling, are merged into one tree.  Node 0 of a tree is its root (the last
// token of the current sequence; it carries no draft token).  The candidates are walked in
// order; at each depth the walk moves to the child that carries the same token (children
// are searched in creation order) or creates it, so nodes are numbered in creation order
// and a parent always precedes its children.  A node reached by several candidates keeps
// the OR of their token flags.
// Inputs per sequence b: draft_ids/draft_flags [max_cands x draft_len], cand_len, n_cands as
// oracle_draft writes them.  Outputs per sequence, max_nodes = 1 + max_cands*draft_len slots:
// node_token (NONE for the root and unused slots), node_parent (index inside the tree, NONE
// for the root and unused slots), node_flags, node_depth, and n_nodes[b].
// ---------------------------------------------------------------------------------
int oracle_tree_build(const int32_t* draft_ids, const uint8_t* draft_flags, const int32_t* cand_len,
                      const int32_t* n_cands, int32_t B, int max_cands, int draft_len,
                      int32_t* node_token, int32_t* node_parent, uint8_t* node_flags,
                      int32_t* node_depth, int32_t* n_nodes) {
    if (B < 0 || max_cands < 1 || draft_len < 1) return 1;
    const int64_t cap = 1 + (int64_t)max_cands * draft_len;
    for (int32_t b = 0; b < B; ++b) {
        int32_t* tok = node_token + b * cap;
        int32_t* par = node_parent + b * cap;
        uint8_t* fl = node_flags + b * cap;
        int32_t* dep = node_depth + b * cap;
        for (int64_t v = 0; v < cap; ++v) {
            tok[v] = NONE;
            par[v] = NONE;
            fl[v] = 0;
            dep[v] = 0;
        }
        int32_t n = 1;  // the root
        for (int32_t c = 0; c < n_cands[b]; ++c) {
            const int32_t* d = draft_ids + ((int64_t)b * max_cands + c) * draft_len;
            const uint8_t* f = draft_flags + ((int64_t)b * max_cands + c) * draft_len;
            int32_t u = 0;
            for (int32_t i = 0; i < cand_len[(int64_t)b * max_cands + c]; ++i) {
                if (d[i] == NONE) break;
                int32_t child = NONE;
                for (int32_t v = 1; v < n && child == NONE; ++v)
                    if (par[v] == u && tok[v] == d[i]) child = v;
                if (child == NONE) {
                    child = n++;
                    tok[child] = d[i];
                    par[child] = u;
                    dep[child] = dep[u] + 1;
                }
                fl[child] |= f[i];
                u = child;
            }
        }
        n_nodes[b] = n;
    }
    return 0;
}

// ---------------------------------------------------------------------------------
// O-VT: verification of draft trees (Eq. 2, Sec. 3.3).  Row v of the logits is the target
// distribution P_M(. | F(v)) that follows node v, F(v) being the path from the root to v;
// so the token of node v is judged by the row of its parent, with the rules of O-V (modes
// 0-2).  A node passes when it and all its ancestors are accepted (prefix rule, Sec. 2.1);
// the result of a tree is its deepest passing node (ties: lowest node index; the root when
// nothing passes): "the longest draft candidate that passes verification".  Mode 3 (TOP_K,
// the alternative of Sec. 3.3): an eligible node passes iff fewer than top_k tokens of its
// parent's row are ahead of its token in the order (logit desc, id asc) and the token is not
// masked; n_greater[node] is that count (NONE for roots, NONE / masked tokens, bad rows).  Emitted: the
// tokens on the path to that node, followed by the target's own token of that node's row.
// Trees are CSR ranges of nodes (tree_offsets[T+1]); node_parent holds indices inside the
// tree (NONE for the root, which is node 0 of its tree); parents precede children.
// Per row: entropy, pmax, argmax, threshold, sampled, bad.  Per node: p_token, accept (the
// node's own bit; 0 for roots), near.  Per tree: best_node (inside the tree), n_accept
// (its depth), n_emit, emit_ids [T x emit_stride] (NONE padded, clipped at emit_stride).
// ---------------------------------------------------------------------------------
int oracle_verify_tree(const void* logits, int dtype, const int32_t* node_token,
                       const int32_t* node_parent, const uint8_t* node_flags,
                       const int32_t* tree_offsets, int32_t T, int64_t V, int64_t row_stride,
                       double alpha, double beta, double invT, int mode, uint64_t seed, uint32_t step,
                       int top_k, int threads, int emit_stride, double* p_token, double* entropy, double* pmax,
                       int32_t* argmax, double* threshold, uint8_t* accept, int32_t* sampled,
                       uint8_t* near, uint8_t* bad, int32_t* n_greater, int32_t* best_node, int32_t* n_accept,
                       int32_t* n_emit, int32_t* emit_ids) {
    if (T < 0 || V <= 0 || mode < 0 || mode > 3 || emit_stride < 1) return 1;
    Rows X{logits, dtype, row_stride};
    const int64_t R = tree_offsets[T];
    std::vector<RowStats> st(R);
    std::vector<int32_t> own(R, NONE);
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
    for (int64_t r = 0; r < R; ++r) {
        st[r] = row_stats(X, r, V, invT);
        int32_t smp = NONE;
        if (!st[r].bad && mode == 2)
            smp = sample_row(X, r, V, invT, seed, (uint32_t)r, step, DOM_VERIFY_GROUP, DOM_VERIFY_ELEM, 0);
        own[r] = st[r].bad ? NONE : (mode == 2 ? smp : st[r].argmax);
        if (entropy) entropy[r] = st[r].H;
        if (pmax) pmax[r] = st[r].pmax;
        if (argmax) argmax[r] = st[r].argmax;
        if (threshold) threshold[r] = st[r].bad ? 0.0 : std::min(alpha * st[r].H + beta, st[r].pmax);
        if (sampled) sampled[r] = smp;
        if (bad) bad[r] = st[r].bad ? 1 : 0;
    }
    for (int32_t t = 0; t < T; ++t) {
        const int64_t lo = tree_offsets[t], hi = tree_offsets[t + 1];
        const int64_t n = hi - lo;
        std::vector<uint8_t> ok(n, 0);
        std::vector<int32_t> depth(n, 0);
        int32_t best = 0;
        for (int64_t v = 0; v < n; ++v) {
            const int64_t g = lo + v;
            const int32_t par = node_parent[g];
            double pt = 0.0;
            bool a = false, is_near = false;
            int32_t ahead_of_d = NONE;
            if (v == 0 || par < 0 || par >= v) {   // the root (or a malformed node: never passes)
                ok[v] = (v == 0);
            } else {
                const RowStats& ps = st[lo + par];
                int32_t d = node_token[g];
                if (d < 0 || d >= V) d = NONE;
                const uint8_t f = node_flags ? node_flags[g] : 1;
                if (!ps.bad && d != NONE) {
                    pt = prob_of(X, lo + par, d, invT, ps);
                    const double yd = X.at(lo + par, d) * invT;
                    if (yd != -std::numeric_limits<double>::infinity()) {   // a masked token has no rank
                        ahead_of_d = 0;
                        for (int64_t i = 0; i < V; ++i)
                            if (i != d && ahead(X.at(lo + par, i) * invT, i, yd, d)) ++ahead_of_d;
                    }
                    if (mode == 0 && (f & 1)) {
                        const double lin = alpha * ps.H + beta;
                        const bool at_max = (X.at(lo + par, d) * invT == ps.m);
                        a = at_max || (pt >= lin);
                        is_near = !at_max && std::fabs(pt - lin) <= 1e-6;
                    } else if (mode == 3 && (f & 1)) {
                        a = ahead_of_d != NONE && ahead_of_d < top_k;
                    } else {
                        a = (d == own[lo + par]);
                    }
                }
                depth[v] = depth[par] + 1;
                ok[v] = a && ok[par];
                if (ok[v] && depth[v] > depth[best]) best = (int32_t)v;
            }
            if (p_token) p_token[g] = pt;
            if (accept) accept[g] = a ? 1 : 0;
            if (near) near[g] = is_near ? 1 : 0;
            if (n_greater) n_greater[g] = ahead_of_d;
        }
        if (n == 0) {
            if (best_node) best_node[t] = NONE;
            if (n_accept) n_accept[t] = 0;
            if (n_emit) n_emit[t] = 0;
            for (int i = 0; i < emit_stride; ++i) emit_ids[(int64_t)t * emit_stride + i] = NONE;
            continue;
        }
        std::vector<int32_t> path;
        for (int32_t v = best; v != 0; v = node_parent[lo + v]) path.push_back(node_token[lo + v]);
        std::reverse(path.begin(), path.end());
        if (own[lo + best] != NONE) path.push_back(own[lo + best]);
        int32_t ne = 0;
        for (int i = 0; i < emit_stride; ++i) {
            int32_t tok = NONE;
            if (i < (int)path.size()) {
                tok = path[i];
                ++ne;
            }
            emit_ids[(int64_t)t * emit_stride + i] = tok;
        }
        if (best_node) best_node[t] = best;
        if (n_accept) n_accept[t] = depth[best];
        if (n_emit) n_emit[t] = ne;
    }
    return 0;
}

// ---------------------------------------------------------------------------------
// Selection (Sec. 3.3, last sentence): per sequence the candidate with the longest
// accepted prefix wins (ties: lowest candidate index).  Emitted tokens = its accepted
// draft ids followed by its next_token when that is not NONE.
// seq_cand_offsets[B+1] is a CSR over candidates; emit_ids is [B x emit_stride].
// A sequence without candidates emits nothing and gets best_cand = NONE.
// ---------------------------------------------------------------------------------
int oracle_select(const int32_t* accept_len, const int32_t* next_token, const int32_t* draft_ids,
                  const int32_t* cand_offsets, const int32_t* seq_cand_offsets, int32_t B,
                  int emit_stride, int32_t* best_cand, int32_t* n_emit, int32_t* emit_ids) {
    for (int32_t b = 0; b < B; ++b) {
        int32_t lo = seq_cand_offsets[b], hi = seq_cand_offsets[b + 1];
        int32_t best = NONE, best_a = -1;
        for (int32_t c = lo; c < hi; ++c)
            if (accept_len[c] > best_a) {
                best_a = accept_len[c];
                best = c;
            }
        for (int i = 0; i < emit_stride; ++i) emit_ids[(int64_t)b * emit_stride + i] = NONE;
        int32_t ne = 0;
        if (best != NONE) {
            for (int32_t i = 0; i < best_a && ne < emit_stride; ++i)
                emit_ids[(int64_t)b * emit_stride + ne++] = draft_ids[cand_offsets[best] + i];
            if (next_token[best] != NONE && ne < emit_stride)
                emit_ids[(int64_t)b * emit_stride + ne++] = next_token[best];
        }
        best_cand[b] = best;
        n_emit[b] = ne;
    }
    return 0;
}

// ---------------------------------------------------------------------------------
// Append (Algorithm 1, q <- q + y): emitted tokens join the history in place.  The
// capacity of sequence b is hist_offsets[b+1] - hist_offsets[b]; tokens beyond it are
// dropped and overflow[b] is set.
// ---------------------------------------------------------------------------------
int oracle_append(int32_t* hist_ids, const int32_t* hist_offsets, int32_t* hist_len,
                  const int32_t* emit_ids, const int32_t* n_emit, int32_t B, int emit_stride,
                  uint8_t* overflow) {
    for (int32_t b = 0; b < B; ++b) {
        int32_t cap = hist_offsets[b + 1] - hist_offsets[b];
        if (overflow) overflow[b] = 0;
        for (int32_t i = 0; i < n_emit[b]; ++i) {
            if (hist_len[b] >= cap) {
                if (overflow) overflow[b] = 1;
                break;
            }
            hist_ids[hist_offsets[b] + hist_len[b]] = emit_ids[(int64_t)b * emit_stride + i];
            hist_len[b] += 1;
        }
    }
    return 0;
}

}  // extern "C"
