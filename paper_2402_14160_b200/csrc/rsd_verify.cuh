// Recursive rejection sampling along the draft tree (Eqs. 1-4, Algorithm 1; Section 3.2.2, Algorithm 6) and the
// stand-alone residual draw.  One thread block walks one sequence and reads only the rows of visited nodes.
//
// The chain of residuals is carried in closed form.  With p, q the node's draft and target distributions, x_0, x_1,
// ... the children in stored order, P_j the draft mass of the first j children and
//     A_0 = 0, Z_0 = 1,   A_{j+1} = A_j + Z_j / (1 - P_j),   Z_j = sum_y (q(y) - A_j p(y))+ ,
// Eq. 2's residual after j rejections is q_j = (q - A_j p)+ / Z_j and Eq. 1's draft is p without x_0..x_{j-1},
// divided by 1 - P_j.  (Induction on Eq. 2: subtracting Z_j p / (1 - P_j) from (q - A_j p)+ and clamping gives
// (q - A_{j+1} p)+; a rejected token has residual mass 0 from then on, so removed tokens need no mask.)
// Eq. 3's threshold becomes  theta_j = min(1, (q(x_j) - A_j p(x_j))+ (1 - P_j) / (Z_j p(x_j))).
// Every further sibling therefore costs one read-only pass over the two rows.
// A removed token keeps the residual mass it had when it was removed (its draft probability is 0 afterwards, so
// Eq. 2 no longer lowers it).  After a genuine rejection (theta < 1) that mass is 0 and the formula above is
// already right; for a caller-supplied list of removals it may be positive, so the passes patch those tokens.
//
// Numerics: exponentials in fp32 relative to a per-row reference m (any value near the row maximum), sums of 16
// in fp32, everything above that and all scalars of the chain in fp64.  The coefficient a = A S_q / S_p is applied
// as a two-float sum so that its rounding does not tilt the whole residual.
#pragma once
#include "rsd_device.cuh"
#include "rsd_scan.cuh"  // ex2_approx

namespace rsd {

constexpr int kMaxTiles = 512;        // tiles of 512 elements: V <= 262144
constexpr int kMaxCachedNodes = 384;  // trees up to this size are copied to shared memory
constexpr int kMaxRemoved = 32;      // removed tokens tracked per node (later ones carry no residual mass)
#ifndef RSD_PASS_UNROLL
#define RSD_PASS_UNROLL 4
#endif
constexpr int kPassUnroll = RSD_PASS_UNROLL;        // turns of a pass whose warp-wide sums are taken together
constexpr float kRefSlack = 60.0f;    // redo a pass if the row maximum exceeds its reference by more than this

struct RowsDev {
    const void* data;
    int64_t seq_stride, row_stride;
    float inv_temp;   // 1 / sampling temperature of these rows (1: none); values enter as value * inv_temp
};

struct VerifyArgs {
    RowsDev draft, target;
    int V, L, num_nodes, shared_topology;
    int rule;      // 0 recursive rejection sampling, 1 multi-round rejection sampling, 2 K-SEQ
    float gamma;   // K-SEQ's parameter
    int final_sampler;   // 0 inverse CDF with one uniform, 1 Gumbel-Top-1
    const int32_t* parent;
    const int32_t* token;
    uint32_t seed_lo, seed_hi, step, seq_base;
    int32_t* accepted_len;
    int32_t* accepted_node;
    int32_t* accepted_token;
    int32_t* last_token;
    int32_t* stop_reason;
    float* dbg_theta;
    int32_t* status;
};

struct ResampleArgs {
    RowsDev draft, target;
    int V, max_k;
    const int32_t* rejected;
    const int32_t* rng_node;
    uint32_t seed_lo, seed_hi, step, seq_base;
    int32_t* out_token;
    float* out_residual;
    int32_t* status;
};

__device__ __forceinline__ float residual_weight(float qh, float ph, float a_hi, float a_lo) {
    return fmaxf(fmaf(-a_lo, ph, fmaf(-a_hi, ph, qh)), 0.0f);
}

template <typename T>
__device__ __forceinline__ const char* row_ptr(const RowsDev& r, int b, int node) {
    return (const char*)r.data + ((int64_t)b * r.seq_stride + (int64_t)node * r.row_stride) * RowIO<T>::kBytes;
}

// Sum of 16 weights in a fixed order: four packed additions fold the eight (even, odd) pairs, the two halves last.
__device__ __forceinline__ float tree_sum16(const float (&w)[16]) {
    const unsigned long long x0 = add_f32x2(f32x2(w[0], w[1]), f32x2(w[2], w[3]));
    const unsigned long long x1 = add_f32x2(f32x2(w[4], w[5]), f32x2(w[6], w[7]));
    const unsigned long long x2 = add_f32x2(f32x2(w[8], w[9]), f32x2(w[10], w[11]));
    const unsigned long long x3 = add_f32x2(f32x2(w[12], w[13]), f32x2(w[14], w[15]));
    float lo, hi;
    split_f32x2(add_f32x2(add_f32x2(x0, x1), add_f32x2(x2, x3)), lo, hi);
    return lo + hi;
}

// exp2(v * k - c) of 16 values, two per fma
__device__ __forceinline__ void exp16(const float (&v)[16], float k, float c, float (&e)[16]) {
    const unsigned long long k2 = f32x2(k, k), c2 = f32x2(-c, -c);
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
        float a, b;
        split_f32x2(fma_f32x2(f32x2(v[j], v[j + 1]), k2, c2), a, b);
        e[j] = ex2_approx(a);
        e[j + 1] = ex2_approx(b);
    }
}

// (qh - a ph)+ for 16 pairs; a = a_hi + a_lo, applied as in residual_weight()
__device__ __forceinline__ void residual16(const float (&qh)[16], const float (&ph)[16], float a_hi, float a_lo,
                                           float (&w)[16]) {
    const unsigned long long nh = f32x2(-a_hi, -a_hi), nl = f32x2(-a_lo, -a_lo);
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
        const unsigned long long p2 = f32x2(ph[j], ph[j + 1]);
        float a, b;
        split_f32x2(fma_f32x2(p2, nl, fma_f32x2(p2, nh, f32x2(qh[j], qh[j + 1]))), a, b);
        w[j] = fmaxf(a, 0.0f);
        w[j + 1] = fmaxf(b, 0.0f);
    }
}

// raw load of group g; rows on 32-byte boundaries take 256-bit loads (a group is 32 or 64 bytes, so every group of
// such a row is aligned)
template <typename T, bool ALIGNED>
__device__ __forceinline__ void load_raw(Packed<T>& pk, const char* row, int g, int V) {
    pk.load(row, g, V, ALIGNED && (g + 1) * 16 <= V, ((uintptr_t)row & 31u) == 0);
}

// unpack a loaded group, turn NaN into -inf (reported), return the group's maximum
template <typename T>
__device__ __forceinline__ float clean(const Packed<T>& pk, float (&v)[16], bool& saw_nan) {
    float m = group_max_nan(pk);   // packed maxima for bf16; NaN if any element is NaN
    pk.unpack(v);
    if (m != m) {
        saw_nan = true;
        m = kNegInf;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (v[j] != v[j]) v[j] = kNegInf;
            m = fmaxf(m, v[j]);
        }
    }
    return m;
}

// Weight modes of a pass over the two rows (qh, ph = exponentials of the target and draft values):
//   kTargetOnly  qh                               plain target distribution
//   kResidual    (qh - a ph)+                     Eq. 2 in closed form, a = a_hi + a_lo
//   kSeqOverlap  min(a_hi ph, a_lo qh)            K-SEQ: min{p, q / gamma} in units of qh
//   kSeqResidual (qh - c min(a_hi ph, a_lo qh))+  K-SEQ: the all-rejected residual
enum { kTargetOnly = 0, kResidual = 1, kSeqOverlap = 2, kSeqResidual = 3 };

template <int MODE>
__device__ __forceinline__ float weight1(float qh, float ph, float a_hi, float a_lo, float c) {
    if (MODE == kResidual) return residual_weight(qh, ph, a_hi, a_lo);
    const float m = fminf(a_hi * ph, a_lo * qh);
    if (MODE == kSeqOverlap) return m;
    if (MODE == kSeqResidual) return fmaxf(fmaf(-c, m, qh), 0.0f);
    return qh;
}

template <int MODE>
__device__ __forceinline__ void weights16(const float (&qh)[16], const float (&ph)[16], float a_hi, float a_lo, float c,
                                          float (&w)[16]) {
    if (MODE == kResidual) {
        residual16(qh, ph, a_hi, a_lo, w);
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) w[j] = weight1<MODE>(qh[j], ph[j], a_hi, a_lo, c);
    }
}

// load a group, turn NaN into -inf (reported), return the group's maximum
template <typename T, bool ALIGNED>
__device__ __forceinline__ float load_clean(const char* row, int g, int V, float (&v)[16], bool& saw_nan) {
    Packed<T> pk;
    load_raw<T, ALIGNED>(pk, row, g, V);
    return clean<T>(pk, v, saw_nan);
}

// The walk itself is compiled twice (rsd_verify_walk.inc): for blocks of 256 threads, three (2-byte rows) or two
// (4-byte rows) per SM, and for blocks of 512 threads, one per SM with all its registers.  A launch with at most one
// sequence per SM has every SM to spare, and there the wider block shortens each pass of a walk's chain.
#define RSD_WALK_NS walk_narrow
#define RSD_WALK_THREADS 256
#define RSD_WALK_MIN_BLOCKS_2B 3
#define RSD_WALK_MIN_BLOCKS_4B 2
#define RSD_WALK_WITH_RESAMPLE
#include "rsd_verify_walk.inc"
#undef RSD_WALK_WITH_RESAMPLE
#undef RSD_WALK_NS
#undef RSD_WALK_THREADS
#undef RSD_WALK_MIN_BLOCKS_2B
#undef RSD_WALK_MIN_BLOCKS_4B

#define RSD_WALK_NS walk_wide
#define RSD_WALK_THREADS 512
#define RSD_WALK_MIN_BLOCKS_2B 1
#define RSD_WALK_MIN_BLOCKS_4B 1
#include "rsd_verify_walk.inc"
#undef RSD_WALK_NS
#undef RSD_WALK_THREADS
#undef RSD_WALK_MIN_BLOCKS_2B
#undef RSD_WALK_MIN_BLOCKS_4B

}  // namespace rsd
