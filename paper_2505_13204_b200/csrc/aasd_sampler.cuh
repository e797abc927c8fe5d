// Keyed Gumbel-max sampling of a logits row (the row's own token of Eq. 1, and the
// alignment extras drawn from the prefill distribution, Sec. 2.3).
//
// Definition (shared with nothing: this is the CUDA path's own statement of it).
//   generator : Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11),
//               key = (seed low word, seed high word), counter = (index, row, step, domain)
//   variate   : 32-bit word r -> u = (r + 0.5) * 2^-32 in (0, 1), G = -ln(-ln u)
//   group stage  : the vocabulary is cut into groups of 32 consecutive ids; group g scores
//                  Lambda_g + G(word j of philox(g, row, step, domain_group)), where
//                  Lambda_g = ln sum_{i in g} e^{y_i}; best score wins, ties to the lower g
//   element stage: inside the winning group, id i scores y_i + G(word j of
//                  philox(i, row, step, domain_elem)); best wins, ties to the lower id
//   draw j (0..3) uses word j, so up to four draws share the generator calls.
// By max-stability of the Gumbel law the winner is distributed exactly as softmax(y).
//
// Fast path: argmax_g (Lambda_g + G_g) = argmax_g (s_g / E_g) with s_g = sum 2^(t_i) the
// group's share of the softmax denominator (already formed by the streaming pass) and
// E_g = -ln u_g an exponential variate, so the streaming pass compares fp32 ratios.  Their
// relative error is below 2e-5 (fma rounding of t up to |t| = 96, ex2.approx, 32-term sum,
// lg2.approx / series for E, rcp.approx); every group whose ratio lies within kSampleBand
// of the best one is re-scored in fp64 from the logits, and rows where more groups are that
// close than the pass keeps track of are sampled by the exhaustive fp64 routine.
#pragma once

#include "aasd_device.cuh"

namespace aasd {

constexpr int kGroup = 32;              // ids per sampling group
constexpr float kSampleBand = 1.0e-3f;  // relative band around the best fp32 ratio that is re-scored in fp64
constexpr int kSampleKeep = 3;          // best groups kept per draw

enum SampleDomain : unsigned int {
    kDomAlignGroup = 2,
    kDomAlignElem = 3,
    kDomVerifyGroup = 4,
    kDomVerifyElem = 5,
};

// What the kernels need to know to sample.
constexpr unsigned int kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;   // key increments per round

struct SampleJob {
    unsigned int key0, key1;   // seed
    unsigned int step;         // decoding step / stream tag
    unsigned int dom_group, dom_elem;
    float inv_t;               // inv_temperature
    // the generator's key schedule, key + round * increment, laid out by the host so that the
    // streaming pass reads its round keys as launch constants instead of adding them up
    unsigned int rk0[10], rk1[10];
};

inline void fill_round_keys(SampleJob& s) {
    for (int r = 0; r < 10; ++r) {
        s.rk0[r] = s.key0 + (unsigned int)r * kPhiloxW0;
        s.rk1[r] = s.key1 + (unsigned int)r * kPhiloxW1;
    }
}

__device__ __forceinline__ void philox4x32_10(unsigned int c0, unsigned int c1, unsigned int c2, unsigned int c3,
                                              unsigned int k0, unsigned int k1, unsigned int (&out)[4]) {
    constexpr unsigned int M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = kPhiloxW0, W1 = kPhiloxW1;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const u64 p0 = (u64)M0 * c0, p1 = (u64)M1 * c2;   // one wide multiply each
        const unsigned int hi0 = (unsigned int)(p0 >> 32), lo0 = (unsigned int)p0;
        const unsigned int hi1 = (unsigned int)(p1 >> 32), lo1 = (unsigned int)p1;
        const unsigned int n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0;
        c1 = lo1;
        c2 = n2;
        c3 = lo0;
        k0 += W0;
        k1 += W1;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

// The same generator with the round keys taken from the job (see SampleJob::rk0).
__device__ __forceinline__ void philox4x32_10_scheduled(unsigned int c0, unsigned int c1, unsigned int c2, unsigned int c3,
                                                        const SampleJob& sj, unsigned int (&out)[4]) {
    constexpr unsigned int M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const u64 p0 = (u64)M0 * c0, p1 = (u64)M1 * c2;
        const unsigned int hi0 = (unsigned int)(p0 >> 32), lo0 = (unsigned int)p0;
        const unsigned int hi1 = (unsigned int)(p1 >> 32), lo1 = (unsigned int)p1;
        const unsigned int n0 = hi1 ^ c1 ^ sj.rk0[round], n2 = hi0 ^ c3 ^ sj.rk1[round];
        c0 = n0;
        c1 = lo1;
        c2 = n2;
        c3 = lo0;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

__device__ __forceinline__ float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// E = -ln u for u = (r + 0.5) * 2^-32, fp32, relative error below 1e-5 over the whole range.
// Close to u = 1 the complement w = 1 - u = (~r + 0.5) * 2^-32 is formed exactly and
// -ln(1 - w) is summed as a series; elsewhere lg2.approx of u is accurate enough.
__device__ __forceinline__ float exponential_fast(unsigned int r) {
    const float two_m32 = 2.3283064365386963e-10f;
    const float w = fmaf((float)(~r), two_m32, 0.5f * two_m32);
    const float u = fmaf((float)r, two_m32, 0.5f * two_m32);
    // w + w^2/2 + w^3/3 + w^4/4: truncation below w^4/5 < 2e-7 relative for w < 2^-5
    float p = fmaf(w, 0.25f, 1.0f / 3.0f);
    p = fmaf(w, p, 0.5f);
    p = fmaf(w, p, 1.0f);
    const float near_one = w * p;
    const float general = -0.6931471805599453f * lg2_approx(u);
    return w < 0.03125f ? near_one : general;
}

// fp64 variate exactly as defined above
__device__ __forceinline__ double gumbel_exact(unsigned int r) {
    const double u = ((double)r + 0.5) * (1.0 / 4294967296.0);
    return -log(-log(u));
}

__device__ __forceinline__ double logit_f64(float x, float inv_t) { return (double)x * (double)inv_t; }

// Running state of one thread over the groups it meets, per draw: its best ratio with the
// group it belongs to, and the best ratio among all its other groups.
template <int ND>
struct GroupRace {
    float best[ND];
    float runner[ND];
    int best_g[ND];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int j = 0; j < ND; ++j) {
            best[j] = -1.f;
            runner[j] = -1.f;
            best_g[j] = -1;
        }
    }
    // 1 / E for the ND draws of group g: depends on the group's index only, not on its logits, so
    // a caller can have it computed while the logits are still on their way through the pipes
    static __device__ __forceinline__ void inverse_variates(int g, unsigned int row, const SampleJob& sj, float (&inv_e)[ND]) {
        unsigned int w[4];
        philox4x32_10_scheduled((unsigned int)g, row, sj.step, sj.dom_group, sj, w);
#pragma unroll
        for (int j = 0; j < ND; ++j) inv_e[j] = rcp_approx(exponential_fast(w[j]));
    }
    // group g with softmax share gsum (relative to the row's reference); valid = false: the group
    // does not take part (it is not wholly inside the row's vectors)
    __device__ __forceinline__ void take(float gsum, const float (&inv_e)[ND], int g, bool valid) {
#pragma unroll
        for (int j = 0; j < ND; ++j) {
            const float q = valid ? gsum * inv_e[j] : -1.f;
            // groups are met in ascending order: '>' keeps the lower g among equal ratios
            const bool up = q > best[j];
            runner[j] = fmaxf(runner[j], up ? best[j] : q);
            best_g[j] = up ? g : best_g[j];
            best[j] = up ? q : best[j];
        }
    }
};

// (ratio, group) as a sortable key: larger ratio first, equal ratios by lower group.
__device__ __forceinline__ u64 race_key(float q, int g) { return g < 0 ? 0ull : make_key(q, g); }

// Per draw: the kSampleKeep best (ratio, group) keys over threads' bests, and the largest
// runner-up ratio of any thread.
struct RaceSummary {
    u64 key[kSampleKeep];
    float runner;
};

// Merges sorted key lists held one per lane (heads in list[0]); every lane gets the result.
template <int N>
__device__ __forceinline__ void warp_merge_keys(u64 (&list)[N], u64 (&out)[N]) {
#pragma unroll
    for (int r = 0; r < N; ++r) {
        const u64 m = warp_max_u64(list[0]);
        out[r] = m;
        if (m != 0 && list[0] == m) {
#pragma unroll
            for (int j = 0; j + 1 < N; ++j) list[j] = list[j + 1];
            list[N - 1] = 0;
        }
    }
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

struct ScoreId {
    double score;
    int id;
};
// larger score first, equal scores by lower id; id < 0 = nothing
__device__ __forceinline__ ScoreId better(const ScoreId& a, const ScoreId& b) {
    if (b.id < 0) return a;
    if (a.id < 0) return b;
    if (a.score > b.score || (a.score == b.score && a.id < b.id)) return a;
    return b;
}
__device__ __forceinline__ ScoreId warp_best(ScoreId v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ScoreId w;
        w.score = __shfl_xor_sync(0xFFFFFFFFu, v.score, o);
        w.id = __shfl_xor_sync(0xFFFFFFFFu, v.id, o);
        v = better(v, w);
    }
    return v;
}

// fp64 score Lambda_g + G of group g for draw j, by a whole warp (one id per lane).
// Returns id < 0 when the group holds no token of positive probability.
template <int DT>
__device__ ScoreId warp_group_score(const char* rowp, int V, int g, unsigned int row, int draw, const SampleJob& sj) {
    const int lane = threadIdx.x & 31;
    const int i = g * kGroup + lane;
    double y = -CUDART_INF;
    if (i < V) y = logit_f64(Elt<DT>::load(rowp, i), sj.inv_t);
    double gm = y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gm = fmax(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, o));
    ScoreId r;
    r.id = -1;
    r.score = 0.0;
    if (gm == -CUDART_INF) return r;
    // index order of the sum: lanes are ids, so add them up one after the other
    const double e = (y == -CUDART_INF) ? 0.0 : exp(y - gm);
    double s = 0.0;
    for (int l = 0; l < kGroup; ++l) s += __shfl_sync(0xFFFFFFFFu, e, l);
    unsigned int w[4];
    philox4x32_10((unsigned int)g, row, sj.step, sj.dom_group, sj.key0, sj.key1, w);
    r.score = gm + log(s) + gumbel_exact(w[draw]);
    r.id = g;
    return r;
}

// Element stage inside group g for draw j, by a whole warp.  Returns the token or NONE.
template <int DT>
__device__ int warp_element_stage(const char* rowp, int V, int g, unsigned int row, int draw, const SampleJob& sj) {
    const int lane = threadIdx.x & 31;
    const int i = g * kGroup + lane;
    ScoreId v;
    v.id = -1;
    v.score = 0.0;
    if (i < V) {
        const double y = logit_f64(Elt<DT>::load(rowp, i), sj.inv_t);
        if (y != -CUDART_INF) {
            unsigned int w[4];
            philox4x32_10((unsigned int)i, row, sj.step, sj.dom_elem, sj.key0, sj.key1, w);
            v.score = y + gumbel_exact(w[draw]);
            v.id = i;
        }
    }
    v = warp_best(v);
    return v.id < 0 ? AASD_NONE : v.id;
}

// The whole definition in fp64 by one warp: every group is scored from the logits.
template <int DT>
__device__ int warp_sample_exhaustive(const char* rowp, int V, unsigned int row, int draw, const SampleJob& sj) {
    const int n_groups = (V + kGroup - 1) / kGroup;
    ScoreId best;
    best.id = -1;
    best.score = 0.0;
    for (int g = 0; g < n_groups; ++g) best = better(best, warp_group_score<DT>(rowp, V, g, row, draw, sj));
    if (best.id < 0) return AASD_NONE;
    return warp_element_stage<DT>(rowp, V, best.id, row, draw, sj);
}

// Decision of one draw from the streaming pass's summary, by a whole warp.
//   tail_group: index of the last, incomplete group that the pass did not score, or -1.
//   force_exhaustive: the pass's ratios cannot be trusted (row re-centred, sums out of range).
// `recheck` / `exhaustive` count what happened (lane 0's copy is the one that is flushed).
template <int DT>
__device__ int warp_sample_decide(const char* rowp, int V, unsigned int row, int draw, const SampleJob& sj,
                                  const RaceSummary& rs, int tail_group, bool force_exhaustive, unsigned int& recheck,
                                  unsigned int& exhaustive) {
    const float q1 = rs.key[0] ? key_value(rs.key[0]) : 0.f;
    const float band = q1 * (1.0f - kSampleBand);
    bool exact = force_exhaustive || !(q1 > 0.f) || !(q1 <= 3.0e38f);
    exact = exact || rs.runner >= band;                                           // two close groups met by one thread
    exact = exact || (rs.key[kSampleKeep - 1] && key_value(rs.key[kSampleKeep - 1]) >= band);   // more close groups than kept
    if (exact) {
        exhaustive += 1;
        return warp_sample_exhaustive<DT>(rowp, V, row, draw, sj);
    }
    int g = key_id(rs.key[0]);
    int n_close = 1;
#pragma unroll
    for (int r = 1; r + 1 < kSampleKeep; ++r)
        if (rs.key[r] && key_value(rs.key[r]) >= band) n_close = r + 1;
    if (n_close > 1 || tail_group >= 0) {
        recheck += 1;
        ScoreId best;
        best.id = -1;
        best.score = 0.0;
        for (int r = 0; r < n_close; ++r) best = better(best, warp_group_score<DT>(rowp, V, key_id(rs.key[r]), row, draw, sj));
        if (tail_group >= 0) best = better(best, warp_group_score<DT>(rowp, V, tail_group, row, draw, sj));
        g = best.id;
        if (g < 0) return AASD_NONE;
    }
    return warp_element_stage<DT>(rowp, V, g, row, draw, sj);
}

}  // namespace aasd
