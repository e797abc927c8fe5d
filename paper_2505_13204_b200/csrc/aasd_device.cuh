// Device-side building blocks shared by the AASD kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/aasd.h"

namespace aasd {

constexpr int kThreads = 256;             // threads per CTA of the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxK = AASD_MAX_EXTRA;     // widest ordered top-k list
constexpr int kMaxSplit = 32;             // most CTAs that share one logits row
constexpr int kPartialSlots = 8192;       // (row, chunk) records held by a workspace
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453;
// A row whose maximum sits more than this many binary orders above the provisional
// reference is streamed a second time with the maximum as reference.  The reference is one
// of the row's own entries, so the shift is never negative; 2^96 times the vocabulary stays
// inside fp32, and the entropy's error grows like shift * 2^-24 (6e-6 at the limit).
constexpr float kRedoShift = 96.0f;

using u64 = unsigned long long;

// Device block owned by a context: status word + running counters.
struct DeviceState {
    unsigned int status;
    unsigned int pad;
    u64 counters[8];
};
enum Counter { kCntRows = 0, kCntBad, kCntRedo, kCntNear, kCntAccepted, kCntRecheck, kCntExact };

// Checked build (-DAASD_BOUNDS_CHECK): the kernels range-check the indices they compute
// before they use them (shared-memory stages and slots, vectors and tokens of a row, rows,
// candidates, scratch records); a violation raises AASD_STATUS_INTERNAL and the access is
// skipped.  In the normal build the macro is the constant true and costs nothing.
#ifdef AASD_BOUNDS_CHECK
__device__ __forceinline__ bool checked_range(bool ok, DeviceState* state) {
    if (!ok) atomicOr(&state->status, AASD_STATUS_INTERNAL);
    return ok;
}
#define AASD_IN_RANGE(cond, state) (::aasd::checked_range((cond), (state)))
#else
#define AASD_IN_RANGE(cond, state) (true)
#endif

// Per (row, chunk) result of the streaming pass.
struct RowPartial {
    double S;          // sum 2^(x*c1 - refc)
    double A;          // sum 2^(x*c1 - refc) * (x*c1 - refc)
    u64 key[kMaxK];    // best tokens, descending; 0 = empty
    long long ahead;   // top-k verification: tokens counted ahead of the draft token so far
};

// ---- ordered keys: larger logit first, equal logits by lower id --------------------
__device__ __forceinline__ unsigned int ordered_bits(float f) {
    unsigned int u = __float_as_uint(f);
    return u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float unordered_bits(unsigned int o) {
    unsigned int u = (o & 0x80000000u) ? (o ^ 0x80000000u) : ~o;
    return __uint_as_float(u);
}
__device__ __forceinline__ u64 make_key(float v, int id) {
    return ((u64)ordered_bits(v) << 32) | (u64)(0xFFFFFFFFu - (unsigned int)id);
}
__device__ __forceinline__ float key_value(u64 k) { return unordered_bits((unsigned int)(k >> 32)); }
__device__ __forceinline__ int key_id(u64 k) { return (int)(0xFFFFFFFFu - (unsigned int)k); }

template <int K>
__device__ __forceinline__ void key_insert(u64 (&list)[K], u64 k) {
#pragma unroll
    for (int j = 0; j < K; ++j) {
        u64 hi = list[j] > k ? list[j] : k;
        k = list[j] > k ? k : list[j];
        list[j] = hi;
    }
}

__device__ __forceinline__ u64 warp_max_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        u64 w = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = w > v ? w : v;
    }
    return v;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum of the values held by lanes 0..7 (the other lanes' values are ignored), in every lane.
__device__ __forceinline__ double octet_sum_f64(double v) {
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return __shfl_sync(0xFFFFFFFFu, v, 0);
}

__device__ __forceinline__ long long warp_sum_i64(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Takes a ticket: adds 1 to a counter in global memory and returns its old value.  The
// addition releases what this thread wrote before it and acquires what earlier ticket holders
// released, in one instruction (instead of a fence, an atomic and another fence).
__device__ __forceinline__ unsigned int take_ticket(unsigned int* counter) {
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
    return old;
}

// ---- programmatic dependent launch -----------------------------------------------------
// Lets the next kernel of the stream be scheduled early; it still waits for this grid.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
// Blocks until the preceding kernel of the stream has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- element access ---------------------------------------------------------------------
template <int DT> struct Elt;
template <> struct Elt<AASD_F32> {
    static constexpr int kVec = 4;
    static constexpr int kSize = 4;
    static __device__ __forceinline__ float load(const void* row, int64_t i) {
        return __ldg(static_cast<const float*>(row) + i);
    }
    static __device__ __forceinline__ void unpack(const uint4& q, float (&x)[4]) {
        x[0] = __uint_as_float(q.x);
        x[1] = __uint_as_float(q.y);
        x[2] = __uint_as_float(q.z);
        x[3] = __uint_as_float(q.w);
    }
};
template <> struct Elt<AASD_BF16> {
    static constexpr int kVec = 8;
    static constexpr int kSize = 2;
    static __device__ __forceinline__ float load(const void* row, int64_t i) {
        unsigned short h = __ldg(static_cast<const unsigned short*>(row) + i);
        return __uint_as_float((unsigned int)h << 16);
    }
    static __device__ __forceinline__ void unpack(const uint4& q, float (&x)[8]) {
        x[0] = __uint_as_float(q.x << 16);
        x[1] = __uint_as_float(q.x & 0xFFFF0000u);
        x[2] = __uint_as_float(q.y << 16);
        x[3] = __uint_as_float(q.y & 0xFFFF0000u);
        x[4] = __uint_as_float(q.z << 16);
        x[5] = __uint_as_float(q.z & 0xFFFF0000u);
        x[6] = __uint_as_float(q.w << 16);
        x[7] = __uint_as_float(q.w & 0xFFFF0000u);
    }
};

// 16-byte streaming load: every logit is read exactly once.
__device__ __forceinline__ uint4 load_stream16(const void* p) {
    uint4 q;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w)
                 : "l"(p));
    return q;
}

// ---- the streaming pass over one chunk of one row -------------------------------------------
//
// Per thread: packed fp32 accumulators of S and A relative to a reference, and the K vectors
// with the largest maxima (value, vector index).
//   first pass (SAFE = false): t = fma(x, c1, r) with r = -(ref * c1): one FMA per pair;
//   second pass (SAFE = true): t = (x + r) * c1 with r = -max, exact at the maximum for any
//   magnitude, and -inf logits are clamped so that 0 * -inf never reaches A.
template <int DT, int K, bool SAFE>
struct RowAccumulator {
    static constexpr int kVec = Elt<DT>::kVec;
    static constexpr int kAcc = kVec / 2;
    float2 S2[kAcc];
    float2 A2[kAcc];
    float best[K > 0 ? K : 1];
    int best_vec[K > 0 ? K : 1];

    __device__ __forceinline__ void init() {
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            S2[i] = make_float2(0.f, 0.f);
            A2[i] = make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < (K > 0 ? K : 1); ++j) {
            best[j] = -CUDART_INF_F;
            best_vec[j] = -1;
        }
    }

    __device__ __forceinline__ void add_vector(const uint4& q, int vec_index, float c1, float neg_refc) {
        float x[kVec];
        Elt<DT>::unpack(q, x);
        const float2 cc = make_float2(c1, c1);
        const float2 rr = make_float2(neg_refc, neg_refc);
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            float2 t;
            if (SAFE) {
                t = __fmul2_rn(__fadd2_rn(make_float2(x[2 * i], x[2 * i + 1]), rr), cc);
                t.x = (t.x < -3.0e38f) ? -3.0e38f : t.x;
                t.y = (t.y < -3.0e38f) ? -3.0e38f : t.y;
            } else {
                t = __ffma2_rn(make_float2(x[2 * i], x[2 * i + 1]), cc, rr);
            }
            float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
            S2[i] = __fadd2_rn(S2[i], e);
            A2[i] = __ffma2_rn(e, t, A2[i]);
        }
        if (K > 0) {
            float vmax = x[0];
#pragma unroll
            for (int i = 1; i < kVec; ++i) vmax = fmaxf(vmax, x[i]);
            int vi = vec_index;
#pragma unroll
            bool up = false;
            for (int j = 0; j < K; ++j) {
                // A thread meets its vectors in ascending order, so a new one goes ahead of a kept
                // one only if it is larger ('>' keeps the lower id ahead among equals); what a
                // slot hands down was ranked above everything below it and stays so, whatever
                // the comparison of the values alone says (equal values: it is the earlier one).
                up = up || vmax > best[j];
                float hi = fmaxf(best[j], vmax);
                float lo = fminf(best[j], vmax);
                int hi_i = up ? vi : best_vec[j];
                int lo_i = up ? best_vec[j] : vi;
                best[j] = hi;
                best_vec[j] = hi_i;
                vmax = lo;
                vi = lo_i;
            }
        }
    }

    __device__ __forceinline__ void add_scalar(float xv, float c1, float neg_refc, float& S, float& A) {
        float t;
        if (SAFE) {
            t = (xv + neg_refc) * c1;
            t = (t < -3.0e38f) ? -3.0e38f : t;
        } else {
            t = fmaf(xv, c1, neg_refc);
        }
        float e = ex2_approx(t);
        S += e;
        A = fmaf(e, t, A);
    }

    __device__ __forceinline__ void totals(double& S, double& A) const {
        S = 0.0;
        A = 0.0;
#pragma unroll
        for (int i = 0; i < kAcc; ++i) {
            S += (double)S2[i].x + (double)S2[i].y;
            A += (double)A2[i].x + (double)A2[i].y;
        }
    }
};

}  // namespace aasd
