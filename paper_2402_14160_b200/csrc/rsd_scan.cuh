// Row scan: exact sorted arg-top-k of (row + Gumbel noise) in one pass over the row (Eqs. 6-7, Algorithm 4), and
// the per-sequence epilogue of a Stochastic Beam Search level (Eqs. 10-12, Algorithm 9).
//
// The noise of a group of 16 consecutive elements is drawn through its order statistics (see rsd_device.cuh): one
// word of a Philox call gives the group's largest noise and the element that carries it, and one call serves the
// four groups a lane meets in a chunk of 128 groups.  The streaming loop
// therefore needs, per group, only the largest value of the group: value_max + noise_max bounds every perturbed
// value of the group from above, and value(a) + noise_max is the exact perturbed value of one element, i.e. a
// sample from below.  The k-th largest of those samples is a true lower bound tau of the k-th largest perturbed
// value; after the loop only the groups whose upper bound reaches tau are looked at element by element, with
// exact noise.  Nothing that could rank is skipped, so the result equals "perturb everything and sort" in fp32.
#pragma once
#include <cuda_fp16.h>

#include "rsd_device.cuh"

namespace rsd {

constexpr int kScanThreads = 128;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kMaxRows = 256;
constexpr int kIdxNone = 0x7FFFFFFF;
// Queue sizes of the per-row stages.  Overflow of any of them is handled (general path, raised bound), so a build
// with tiny sizes (-DRSD_SCAN_SMALL_QUEUES) gives the same results; the tests use one to exercise those paths.
#ifdef RSD_SCAN_SMALL_QUEUES
constexpr int kCandCap = 4, kTaskCap = 4, kFinCap = 2, kSurvCap = 40;
#else
constexpr int kCandCap = 512;           // candidate groups queued per row (more are handled in place)
constexpr int kTaskCap = 512;           // elements of candidate groups that may reach the bound
constexpr int kFinCap = 256;            // elements that pass the cheap noise test
constexpr int kSurvCap = 256;           // elements whose exact perturbed value reaches the bound (>= RSD_MAX_K)
#endif

struct ScanArgs {
    const void* data;
    int64_t seq_stride, row_stride;  // elements
    int R, V, max_k;
    uint32_t seed_lo, seed_hi, step, seq_base;
    int subtract_lse;     // 1: outputs in log-probability units (value - LSE)
    float inv_temp, temp; // every value is multiplied by inv_temp = 1 / temperature before anything else (1: none)
    int raw_values;       // 1: out_value receives the rows' own values as stored (the beam search epilogue scales them
                          // in double); 0: value * inv_temp - shift
    int32_t* out_token;   // [B][R][max_k]
    float* out_perturbed; // [B][R][max_k] or null
    float* out_value;     // [B][R][max_k] or null: the row's own value at each pick
    float* out_lse;       // [B][R] or null
    int32_t* status;      // [B], OR-ed into
    int32_t* row_status;  // [B][R] or null; when set, the row's NaN flag is stored here instead (beam search level:
                          // the epilogue assembles status[b], and a row with fewer than k picks is not an event)
    int32_t* node_token;  // [B][node_stride] or null: pick j of row r also goes to node child_base[r] + j
    int node_stride;
    uint32_t rk0[10], rk1[10];  // Philox round keys: seed_lo + r * 0x9E3779B9, seed_hi + r * 0xBB67AE85
    uint8_t k_row[kMaxRows];
    int32_t node_row[kMaxRows];
    int32_t child_base[kMaxRows];
};

// Packed pairs of fp32 (sm_100 executes fma/add on two floats per instruction).
__device__ __forceinline__ unsigned long long f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ void split_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

// Coarse Gumbel stream of one row: counter words 1..3 and the key are fixed, only word 0 (the group index)
// varies, so the parts of the first two rounds that do not depend on it are computed once per block.
struct PhiloxRow {
    uint32_t c3k1;  // c3 ^ k1[0]
    uint32_t b0;    // lo(M1 * c2) ^ k0[1]
    uint32_t b2;    // hi(M0 * a0) ^ k1[1],  a0 = hi(M1 * c2) ^ c1 ^ k0[0]
    uint32_t b3;    // lo(M0 * a0)
};

__device__ __forceinline__ PhiloxRow philox_row_setup(const ScanArgs& a, uint32_t c1, uint32_t c2, uint32_t c3) {
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t a0 = (uint32_t)(p1 >> 32) ^ c1 ^ a.rk0[0];
    const uint64_t p0 = (uint64_t)0xD2511F53u * a0;
    PhiloxRow r;
    r.c3k1 = c3 ^ a.rk1[0];
    r.b0 = (uint32_t)p1 ^ a.rk0[1];
    r.b2 = (uint32_t)(p0 >> 32) ^ a.rk1[1];
    r.b3 = (uint32_t)p0;
    return r;
}

// Philox4x32-10 of counter (c0, c1, c2, c3) with the row's constants folded in; equals philox4x32_10().
__device__ __forceinline__ uint4 philox_row(const ScanArgs& a, const PhiloxRow& r, uint32_t c0) {
    // round 1: only the c0 half varies
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint32_t x2 = (uint32_t)(p0 >> 32) ^ r.c3k1;
    uint32_t x3 = (uint32_t)p0;
    // round 2: inputs (a0, lo(M1 c2), x2, x3)
    uint64_t p1 = (uint64_t)0xCD9E8D57u * x2;
    uint32_t y0 = (uint32_t)(p1 >> 32) ^ r.b0;
    uint32_t y1 = (uint32_t)p1;
    uint32_t y2 = x3 ^ r.b2;
    uint32_t y3 = r.b3;
#pragma unroll
    for (int i = 2; i < 10; ++i) {
        p0 = (uint64_t)0xD2511F53u * y0;
        p1 = (uint64_t)0xCD9E8D57u * y2;
        y0 = (uint32_t)(p1 >> 32) ^ y1 ^ a.rk0[i];
        y2 = (uint32_t)(p0 >> 32) ^ y3 ^ a.rk1[i];
        y1 = (uint32_t)p1;
        y3 = (uint32_t)p0;
    }
    return make_uint4(y0, y1, y2, y3);
}

// Fine Gumbel stream word of element e, with the round keys taken from the kernel arguments.
__device__ __forceinline__ uint32_t fine_word_rk(const ScanArgs& a, const RngKey& k, uint32_t node, uint32_t e) {
    uint32_t c0 = e >> 2, c1 = (node & 0x0FFFFFFFu) | (kTagGumbelFine << 28), c2 = k.seq, c3 = k.step;
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ a.rk0[i];
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ a.rk1[i];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
    }
    const uint32_t sel = e & 3u;
    return sel < 2 ? (sel == 0 ? c0 : c1) : (sel == 2 ? c2 : c3);
}

__device__ __forceinline__ bool better(float v1, int i1, float v2, int i2) {
    return v1 > v2 || (v1 == v2 && i1 < i2);
}

__device__ __forceinline__ float ex2_approx(float x) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// The 16 elements of a group as loaded (fp32: four 16-byte words, bf16: two), kept packed while they wait.
template <typename T>
struct Packed;
template <>
struct Packed<float> {
    uint4 w[4];
    __device__ __forceinline__ void unpack(float (&v)[16]) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[4 * i + 0] = __uint_as_float(w[i].x);
            v[4 * i + 1] = __uint_as_float(w[i].y);
            v[4 * i + 2] = __uint_as_float(w[i].z);
            v[4 * i + 3] = __uint_as_float(w[i].w);
        }
    }
    __device__ __forceinline__ void fill_neg_inf() {
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
    }
    static __device__ __forceinline__ uint32_t clean_word(uint32_t q) {
        return (q & 0x7FFFFFFFu) > 0x7F800000u ? 0xFF800000u : q;
    }
    __device__ __forceinline__ void clean_nan() {   // NaN elements become -inf
#pragma unroll
        for (int i = 0; i < 4; ++i)
            w[i] = make_uint4(clean_word(w[i].x), clean_word(w[i].y), clean_word(w[i].z), clean_word(w[i].w));
    }
    // f(pair) for the 8 pairs of neighbouring values, as packed fp32, in order
    template <typename F>
    __device__ __forceinline__ void for_each_pair(F f) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f(f32x2(__uint_as_float(w[i].x), __uint_as_float(w[i].y)));
            f(f32x2(__uint_as_float(w[i].z), __uint_as_float(w[i].w)));
        }
    }
    __device__ __forceinline__ void load_aligned(const void* group, bool wide) {  // 64 bytes, 16- or 32-byte aligned
        if (wide) {
            ld_stream_256(group, w[0], w[1]);
            ld_stream_256((const char*)group + 32, w[2], w[3]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = ld_stream((const uint4*)group + i);
        }
    }
    __device__ __forceinline__ void load(const void* row, int g, int V, bool aligned_full, bool wide = false) {
        if (aligned_full) {
            load_aligned((const float*)row + (size_t)g * 16, wide);
        } else {
            uint32_t u[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int x = g * 16 + i;
                u[i] = x < V ? __float_as_uint(((const float*)row)[x]) : 0xFF800000u;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = make_uint4(u[4 * i], u[4 * i + 1], u[4 * i + 2], u[4 * i + 3]);
        }
    }
};
template <>
struct Packed<__nv_bfloat16> {
    uint4 w[2];
    __device__ __forceinline__ void unpack(float (&v)[16]) const {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t q[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[8 * i + 2 * j + 0] = __uint_as_float(q[j] << 16);
                v[8 * i + 2 * j + 1] = __uint_as_float(q[j] & 0xFFFF0000u);
            }
        }
    }
    __device__ __forceinline__ void fill_neg_inf() {
        w[0] = w[1] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
    }
    static __device__ __forceinline__ uint32_t clean_word(uint32_t q) {
        if ((q & 0x7FFFu) > 0x7F80u) q = (q & 0xFFFF0000u) | 0xFF80u;
        if ((q & 0x7FFF0000u) > 0x7F800000u) q = (q & 0xFFFFu) | 0xFF800000u;
        return q;
    }
    __device__ __forceinline__ void clean_nan() {   // NaN elements become -inf
#pragma unroll
        for (int i = 0; i < 2; ++i)
            w[i] = make_uint4(clean_word(w[i].x), clean_word(w[i].y), clean_word(w[i].z), clean_word(w[i].w));
    }
    // f(pair) for the 8 pairs of neighbouring values, as packed fp32, in order
    template <typename F>
    __device__ __forceinline__ void for_each_pair(F f) const {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t q[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) f(f32x2(__uint_as_float(q[j] << 16), __uint_as_float(q[j] & 0xFFFF0000u)));
        }
    }
    __device__ __forceinline__ void load_aligned(const void* group, bool wide) {  // 32 bytes, 16- or 32-byte aligned
        if (wide) {
            ld_stream_256(group, w[0], w[1]);
        } else {
            w[0] = ld_stream((const uint4*)group);
            w[1] = ld_stream((const uint4*)group + 1);
        }
    }
    __device__ __forceinline__ void load(const void* row, int g, int V, bool aligned_full, bool wide = false) {
        if (aligned_full) {
            load_aligned((const uint16_t*)row + (size_t)g * 16, wide);
        } else {
            uint32_t u[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int x = g * 16 + 2 * i;
                const uint32_t lo = x < V ? ((const uint16_t*)row)[x] : 0xFF80u;
                const uint32_t hi = x + 1 < V ? ((const uint16_t*)row)[x + 1] : 0xFF80u;
                u[i] = lo | (hi << 16);
            }
            w[0] = make_uint4(u[0], u[1], u[2], u[3]);
            w[1] = make_uint4(u[4], u[5], u[6], u[7]);
        }
    }
};

// largest of the 16 values, NaN if any is NaN
__device__ __forceinline__ float group_max_nan(const Packed<float>& p) {
    float m = max_nan(max_nan(__uint_as_float(p.w[0].x), __uint_as_float(p.w[0].y)),
                      max_nan(__uint_as_float(p.w[0].z), __uint_as_float(p.w[0].w)));
#pragma unroll
    for (int i = 1; i < 4; ++i)
        m = max_nan(m, max_nan(max_nan(__uint_as_float(p.w[i].x), __uint_as_float(p.w[i].y)),
                               max_nan(__uint_as_float(p.w[i].z), __uint_as_float(p.w[i].w))));
    return m;
}
__device__ __forceinline__ uint32_t bf162_max_nan(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ float group_max_nan(const Packed<__nv_bfloat16>& p) {
    const uint32_t a = bf162_max_nan(bf162_max_nan(p.w[0].x, p.w[0].y), bf162_max_nan(p.w[0].z, p.w[0].w));
    const uint32_t b = bf162_max_nan(bf162_max_nan(p.w[1].x, p.w[1].y), bf162_max_nan(p.w[1].z, p.w[1].w));
    const uint32_t m = bf162_max_nan(a, b);
    return max_nan(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
}
// element `pos` (0..15) of the group, by a select tree (no dynamic register indexing)
__device__ __forceinline__ uint32_t pick_word(const uint4& q, int i) {
    const uint32_t lo = (i & 1) ? q.y : q.x, hi = (i & 1) ? q.w : q.z;
    return (i & 2) ? hi : lo;
}
__device__ __forceinline__ float group_element(const Packed<float>& p, int pos) {
    const uint32_t a = pick_word(p.w[0], pos), b = pick_word(p.w[1], pos), c = pick_word(p.w[2], pos),
                   d = pick_word(p.w[3], pos);
    const uint32_t lo = (pos & 4) ? b : a, hi = (pos & 4) ? d : c;
    return __uint_as_float((pos & 8) ? hi : lo);
}
__device__ __forceinline__ float group_element(const Packed<__nv_bfloat16>& p, int pos) {
    const int wi = pos >> 1;
    const uint32_t a = pick_word(p.w[0], wi), b = pick_word(p.w[1], wi);
    const uint32_t w = (wi & 4) ? b : a;
    return __uint_as_float((pos & 1) ? (w & 0xFFFF0000u) : (w << 16));
}

// bit j set when element j of the group is >= need (need finite; NaN and -inf elements never pass)
__device__ __forceinline__ uint32_t group_mask_ge(const Packed<float>& p, float need) {
    float v[16];
    p.unpack(v);
    uint32_t m = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j)
        if (v[j] >= need) m |= 1u << j;
    return m;
}
__device__ __forceinline__ uint32_t group_mask_ge(const Packed<__nv_bfloat16>& p, float need) {
    // the values lie on the bf16 grid, so v >= need exactly when v >= need rounded up to that grid
    uint16_t nb;
    asm("cvt.rp.bf16.f32 %0, %1;" : "=h"(nb) : "f"(need));
    const uint32_t need2 = (uint32_t)nb * 0x00010001u;
    const uint32_t q[8] = {p.w[0].x, p.w[0].y, p.w[0].z, p.w[0].w, p.w[1].x, p.w[1].y, p.w[1].z, p.w[1].w};
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t ge;   // 0xFFFF per half that passes
        asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(ge) : "r"(q[i]), "r"(need2));
        acc |= ge & ((1u << (2 * i)) | (1u << (2 * i + 17)));
    }
    return (acc | (acc >> 16)) & 0xFFFFu;
}

// Bounds of the group's largest noise G_max = -ln(t / 16), t = -ln((bits + 1/2) / 2^28), from two fast logarithms:
// lo <= G_max <= hi.  With t_hat the fast value of t, |t_hat - t| <= 2.7e-7 + 3e-7 t (conversion, fma and lg2.approx
// at 2^-22), so for t >= 2^-12 the relative error of t_hat / 16 is below 1.2e-3; the outer lg2.approx and the final
// fma add less than 1e-5.  Below 2^-12 (one group in 4096) the bounds are -huge and +huge.
constexpr float kNoiseMargin = 1.5e-3f;
__device__ __forceinline__ float lg2_approx(float x) {
    float r;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void group_noise_bounds(uint32_t bits, float& lo, float& hi) {
    const float u = fmaf((float)bits, 3.725290298461914e-09f, 1.862645149230957e-09f);  // (bits + 1/2) / 2^28
    const float ts = fmaf(lg2_approx(u), -0.04332169878499658f, 1e-30f);                // t / 16 (> 0), -ln2 / 16
    const float margin = ts >= 1.52587890625e-05f ? kNoiseMargin : 1e30f;               // t / 16 >= 2^-16
    const float l2 = lg2_approx(ts);
    hi = fmaf(l2, -0.6931471805599453f, margin);
    lo = fmaf(l2, -0.6931471805599453f, -margin);
}

// Shared-memory slot of one thread for the group it is working on: the 16 values as loaded, so that the one at a
// position known only at run time can be read back with one load instead of a select tree.  The stride of 16 bytes
// more than the data keeps the 16-byte stores of a quarter warp on distinct banks.
template <typename T>
struct GroupSlot {
    static constexpr int kStride = (int)sizeof(Packed<T>) + 16;
};
__device__ __forceinline__ void slot_store(uint32_t addr, const Packed<float>& p) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr + 16u * i), "r"(p.w[i].x), "r"(p.w[i].y),
                     "r"(p.w[i].z), "r"(p.w[i].w));
}
__device__ __forceinline__ void slot_store(uint32_t addr, const Packed<__nv_bfloat16>& p) {
#pragma unroll
    for (int i = 0; i < 2; ++i)
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr + 16u * i), "r"(p.w[i].x), "r"(p.w[i].y),
                     "r"(p.w[i].z), "r"(p.w[i].w));
}
template <typename T>
__device__ __forceinline__ float slot_element(uint32_t addr, uint32_t pos);
template <>
__device__ __forceinline__ float slot_element<float>(uint32_t addr, uint32_t pos) {
    float r;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(r) : "r"(addr + 4u * pos));
    return r;
}
template <>
__device__ __forceinline__ float slot_element<__nv_bfloat16>(uint32_t addr, uint32_t pos) {
    uint32_t r;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(r) : "r"(addr + 2u * pos));
    return __uint_as_float(r << 16);
}

// One block per row.
// ALIGNED: rows start on 16-byte boundaries and V is a multiple of 16 (vector loads); WIDE: 32-byte boundaries as well.
// TEMP: a sampling temperature other than 1 applies (otherwise the scale factors are compile-time constants).
// Nine blocks per SM for 2-byte rows (56 registers: a group in flight is 8 registers), eight for 4-byte rows.
template <typename T, bool ALIGNED, bool WIDE, bool NEED_LSE, bool TEMP>
__global__ void __launch_bounds__(kScanThreads, sizeof(T) == 2 ? 9 : 8) scan_topk_kernel(const ScanArgs a) {
    extern __shared__ float ub[];                    // [n_groups] upper bound of each group's perturbed values
    // One buffer, two uses: the threads' group slots during the streaming loop, the queues of the stages after it.
    constexpr int kQueueBytes = 4 * (kCandCap + 3 * kTaskCap + 4 * kFinCap);
    constexpr int kSlotBytes = kScanThreads * GroupSlot<T>::kStride;
    __shared__ __align__(16) unsigned char shared_buf[kQueueBytes > kSlotBytes ? kQueueBytes : kSlotBytes];
    int* const cand = (int*)shared_buf;                              // groups whose bound reaches tau
    uint32_t* const tk_x = (uint32_t*)(cand + kCandCap);             // element index | (it carries the group's largest noise) << 31
    float* const tk_base = (float*)(tk_x + kTaskCap);                // lower bound of t(U_M) / 16 of the element's group
    uint32_t* const tk_word = (uint32_t*)(tk_base + kTaskCap);       // coarse-stream word of its group
    uint32_t* const fin_x = tk_word + kTaskCap;                      // element (same encoding as tk_x) ...
    uint32_t* const fin_w = fin_x + kFinCap;                         // ... its fine-stream word,
    float* const fin_raw = (float*)(fin_w + kFinCap);                // value
    uint32_t* const fin_word = (uint32_t*)(fin_raw + kFinCap);       // and coarse-stream word
    __shared__ int n_task, n_fin;
    __shared__ float sv_val[kSurvCap], sv_raw[kSurvCap];
    __shared__ int sv_idx[kSurvCap];
    __shared__ uint32_t bin_max[32];                 // per lane index: largest sample over the warps (ordered encoding)
    __shared__ float red_f[kScanWarps];
    __shared__ float red_s[kScanWarps];
    __shared__ int n_cand, n_surv, nan_flag;
    __shared__ float lse_sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / a.R, r = blockIdx.x % a.R;
    const int k = a.k_row[r];
    const uint32_t node = (uint32_t)a.node_row[r];
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    const char* row = (const char*)a.data + ((int64_t)b * a.seq_stride + (int64_t)r * a.row_stride) * RowIO<T>::kBytes;
    const int V = a.V, n_groups = (V + 15) >> 4;
    const int n_iter = (n_groups + kScanThreads - 1) / kScanThreads;
    const PhiloxRow pr = philox_row_setup(a, (node & 0x0FFFFFFFu) | (kTagGumbelCoarse << 28), key.seq, key.step);

    if (tid == 0) { n_cand = 0; n_surv = 0; nan_flag = 0; n_task = 0; n_fin = 0; }
    if (tid < 32) bin_max[tid] = float_to_ordered(kNegInf);
    if (tid < 4 && n_groups + tid < ((n_groups + 3) & ~3)) ub[n_groups + tid] = kNegInf;   // padding of the bounds
    __syncthreads();

    // ---- streaming loop ----------------------------------------------------------------------------------------------
    // A warp takes chunks of 128 consecutive groups; lane l meets groups l, l + 32, l + 64, l + 96 of the chunk, whose
    // coarse-stream words are the four words of one Philox call.
    float best = kNegInf;                  // largest exact sample of this thread (value(a) + lower bound of G_max)
    // Running log-sum-exp of this thread's elements: sum of 2^(value * log2(e) - c) with an integer c, fixed at the
    // first finite group maximum and moved up only when a group maximum exceeds it by more than 40.
    const float inv_temp = TEMP ? a.inv_temp : 1.0f, temp = TEMP ? a.temp : 1.0f;   // values enter as value * inv_temp
    const float log2e_t = kLog2e * inv_temp;
    float lse_thr = kNegInf;               // group maxima above this move the reference (-inf: nothing finite yet)
    float lse_negc = 0.0f;                 // -c
    unsigned long long acc0 = f32x2(0.0f, 0.0f), acc1 = acc0;
    const uint32_t slot = (uint32_t)__cvta_generic_to_shared(shared_buf) + (uint32_t)tid * GroupSlot<T>::kStride;
    // work on one group whose 16 values are in `cur`; `word` is the group's coarse-stream word, `ub_g` = &ub[group]
    auto body = [&](Packed<T>& cur, float* ub_g, uint32_t word) {   // may rewrite cur
        slot_store(slot, cur);
        float g_lo, g_hi;
        group_noise_bounds(word >> 4, g_lo, g_hi);
        float gmax = group_max_nan(cur);
        *ub_g = fmaf(gmax, inv_temp, g_hi);                    // NaN if the group holds a NaN: looked at later
        best = fmaxf(best, fmaf(slot_element<T>(slot, word & 15u), inv_temp, g_lo));  // fmaxf drops NaN
        if (NEED_LSE) {
            // The sums are taken straight from the packed words, a pair at a time, so that no more than a few unpacked
            // values are alive at once; the rare cases below rewrite the group in place first.
            if (!(gmax <= lse_thr)) {  // rare: a NaN in the group, the first finite group, or a jump of more than 40
                if (gmax != gmax) {    // NaN counts as -inf
                    cur.clean_nan();
                    gmax = group_max_nan(cur);
                }
                if (gmax > lse_thr) {
                    const float c_new = ceilf(gmax * log2e_t);
                    const float sc = lse_thr > kNegInf ? ex2_approx(-(lse_negc + c_new)) : 0.0f;  // 2^(c_old - c_new) <= 1
                    float s0, s1, s2, s3;
                    split_f32x2(acc0, s0, s1);
                    split_f32x2(acc1, s2, s3);
                    acc0 = f32x2(s0 * sc, s1 * sc);
                    acc1 = f32x2(s2 * sc, s3 * sc);
                    lse_negc = -c_new;
                    lse_thr = fmaf(40.0f, temp, gmax);   // 40 in scaled units
                }
            }
            const unsigned long long l2 = f32x2(log2e_t, log2e_t), c2 = f32x2(lse_negc, lse_negc);
            int turn = 0;
            cur.for_each_pair([&](unsigned long long p) {   // two elements per fma / add, two accumulators in turn
                float e0, e1;
                split_f32x2(fma_f32x2(p, l2, c2), e0, e1);
                const unsigned long long x = f32x2(ex2_approx(e0), ex2_approx(e1));
                if (turn & 1) acc1 = add_f32x2(acc1, x);
                else acc0 = add_f32x2(acc0, x);
                ++turn;
            });
        }
    };
    // Two buffers: the group two turns ahead is requested as soon as a buffer has been consumed.  Chunks that lie
    // wholly inside the row run without bounds checks; the row's last, partial chunk runs the same steps guarded.
    {
        const int n_full = n_groups >> 7;                    // whole chunks
        auto fetch = [&](Packed<T>& q, int g) {              // guarded
            if (g < n_groups) q.load(row, g, V, ALIGNED, WIDE);
        };
        Packed<T> q0, q1;
        int c = warp;
        fetch(q0, c * 128 + lane);
        fetch(q1, c * 128 + 32 + lane);
        for (; c < n_full; c += kScanWarps) {
            const int g0 = c * 128 + lane;
            float* ub_g = ub + g0;
            const uint4 cw = philox_row(a, pr, (uint32_t)(c * 32 + lane));
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {   // two turns of two groups: keeps the loop's code small
                const int g_next = h ? g0 + kScanWarps * 128 : g0 + 64;   // first turn: inside this chunk
                body(q0, ub_g + 64 * h, h ? cw.z : cw.x);
                fetch(q0, g_next);
                body(q1, ub_g + 64 * h + 32, h ? cw.w : cw.y);
                fetch(q1, g_next + 32);
            }
        }
        if (c == n_full && (n_groups & 127)) {   // this warp owns the partial chunk; q0 and q1 are on their way
            const int g0 = c * 128 + lane;
            float* ub_g = ub + g0;
            const uint4 cw = philox_row(a, pr, (uint32_t)(c * 32 + lane));
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                const int g = g0 + 64 * h;
                if (g < n_groups) body(q0, ub_g + 64 * h, h ? cw.z : cw.x);
                if (h == 0) fetch(q0, g0 + 64);
                if (g + 32 < n_groups) body(q1, ub_g + 64 * h + 32, h ? cw.w : cw.y);
                if (h == 0) fetch(q1, g0 + 96);
            }
        }
    }

    // ---- tau: a lower bound of the k-th largest perturbed value from the threads' samples -------------------------
    // The samples belong to distinct elements.  They are folded into 32 bins (one per lane index, maximum over the
    // warps); the k-th largest bin maximum is at most the k-th largest sample, hence at most the k-th largest
    // perturbed value of the row.  Every warp finds it from the 32 bin maxima itself, so one barrier is enough.
    if (best > kNegInf) atomicMax(&bin_max[lane], float_to_ordered(best));
    if (NEED_LSE) {
        // the warp's share of the log-sum-exp: largest reference exponent C_w and sum of s_t * 2^(c_t - C_w) (exact
        // scaling); the last thread combines the warps' shares after the barrier.  All in fp32: the threads' sums
        // already are, and double-precision instructions are slow enough to show on every row's critical path.
        const float lse_c = lse_thr > kNegInf ? -lse_negc : kNegInf;  // this thread's reference exponent
        const float cw_max = warp_max(lse_c);
        float s0, s1, s2, s3;
        split_f32x2(acc0, s0, s1);
        split_f32x2(acc1, s2, s3);
        const float d = lse_c - cw_max;   // <= 0, an integer (NaN or -inf when there is nothing to add)
        float term = 0.0f;
        if (lse_c > kNegInf && d > -120.0f) term = ((s0 + s1) + (s2 + s3)) * exp2f(d);
        if (cw_max == -kNegInf) term = cw_max - cw_max;  // a +inf value: the sum is not a number
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) term += __shfl_xor_sync(0xFFFFFFFFu, term, o);
        if (lane == 0) { red_f[warp] = cw_max; red_s[warp] = term; }
    }
    __syncthreads();   // also: every thread is done with its group slot, the queues may take the buffer over
    if (NEED_LSE && tid == kScanThreads - 1) {
        float C = red_f[0];
#pragma unroll
        for (int w = 1; w < kScanWarps; ++w) C = fmaxf(C, red_f[w]);
        float S = 0.0f;
#pragma unroll
        for (int w = 0; w < kScanWarps; ++w) {
            const float d = red_f[w] - C;
            if (red_f[w] > kNegInf && d > -120.0f) S += red_s[w] * exp2f(d);
            else if (d != d) S = d;
        }
        // C ln 2 + ln S with ln 2 split so that C * hi is exact (C is a small integer)
        lse_sh = (C > kNegInf && (S > 0.0f || S != S)) ? fmaf(C, 0.693145751953125f, fmaf(C, 1.4286068203094172e-06f, logf(S))) : kNegInf;
    }
    float tau;
    {
        // k-th largest of the 32 bin maxima: take the maximum k times, dropping it (and its equals, which can only
        // lower the result: still a lower bound) after each turn
        uint32_t v = bin_max[lane], top = 0;
        for (int i = 0; i < k; ++i) {
            top = __reduce_max_sync(0xFFFFFFFFu, v);
            if (v == top) v = 0;
        }
        tau = top ? ordered_to_float(top) : kNegInf;
    }

    // ---- candidate groups ---------------------------------------------------------------------------------------------
    // (a NaN bound compares false: the group is kept; the bounds are padded with -inf to a multiple of four)
    const int n_quads = (n_groups + 3) >> 2;
    if (n_quads <= 8 * kScanThreads) {
        // four bounds per load, one bit per group, then one queue reservation per warp
        const float4* ub4 = (const float4*)ub;
        uint32_t mine = 0;
        for (int sw = 0, q = tid; q < n_quads; ++sw, q += kScanThreads) {
            const float4 u = ub4[q];
            const uint32_t m = (!(u.x < tau) ? 1u : 0u) | (!(u.y < tau) ? 2u : 0u) | (!(u.z < tau) ? 4u : 0u) |
                               (!(u.w < tau) ? 8u : 0u);
            mine |= m << (4 * sw);
        }
        const int cnt = __popc(mine);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        int base = 0;
        if (lane == 31) base = atomicAdd(&n_cand, incl);
        base = __shfl_sync(0xFFFFFFFFu, base, 31);
        int slot_c = base + incl - cnt;
        while (mine) {
            const int bit = __ffs(mine) - 1;
            mine &= mine - 1;
            if (slot_c < kCandCap) cand[slot_c] = (((bit >> 2) * kScanThreads + tid) << 2) + (bit & 3);
            ++slot_c;
        }
    } else {
        for (int it = 0; it < n_iter; ++it) {
            const int g = it * kScanThreads + tid;
            if (g < n_groups && !(ub[g] < tau)) {
                const int slot_c = atomicAdd(&n_cand, 1);
                if (slot_c < kCandCap) cand[slot_c] = g;
            }
        }
    }
    __syncthreads();
    const int n_queued = n_cand;

    // exact perturbed values of the elements of group g that can reach tau
    auto process_group = [&](int g) {
        Packed<T> grp;
        grp.load(row, g, V, ALIGNED && (g + 1) * 16 <= V, WIDE);
        const uint32_t word = coarse_select(philox_row(a, pr, coarse_index((uint32_t)g)), (uint32_t)g);
        const float base = neg_log_group_uniform_f32(word) * 0.0625f;   // t(U_M) / 16
        const float g_max = -logf(base);
        const int apos = (int)(word & 15u);
        // elements whose value plus the group's largest noise reaches tau (NaN compares false both ways: flagged)
        uint32_t todo = 0;
        {
            float v[16];
            grp.unpack(v);
            const float need = (tau - g_max - 1e-5f) * temp - 1e-6f * fabsf((tau - g_max) * temp);   // in raw units
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (v[j] != v[j]) nan_flag = 1;
                else if (v[j] > kNegInf && v[j] >= need) todo |= 1u << j;
            }
        }
        while (todo) {
            const int j = __ffs(todo) - 1;
            todo &= todo - 1;
            const int x = g * 16 + j;
            const float raw_u = group_element(grp, j);
            const float raw = raw_u * inv_temp;
            float pert = raw + g_max;
            if (j != apos) pert = raw - logf(base + neg_log_uniform_f32(fine_word_rk(a, key, node, (uint32_t)x)));
            if (pert >= tau) {
                const int sidx = atomicAdd(&n_surv, 1);
                if (sidx < kSurvCap) { sv_val[sidx] = pert; sv_idx[sidx] = x; sv_raw[sidx] = raw_u; }
            }
        }
    };

    // ---- short path: three stages of independent items, one item per thread ------------------------------------------
    // A: per candidate group, the elements whose value plus the group's largest noise can reach tau;
    // B: per such element, its fine-stream word and a cheap test of  t(U_M)/16 + t(U_x) <= exp(value - tau);
    // C: exact perturbed value of what is left.  Any overflow falls through to the general path below.
    bool general = n_queued > kCandCap;
    if (!general) {
        for (int i = tid; i < n_queued; i += kScanThreads) {
            const int g = cand[i];
            Packed<T> grp;
            grp.load(row, g, V, ALIGNED && (g + 1) * 16 <= V, WIDE);
            const uint32_t word = coarse_select(philox_row(a, pr, coarse_index((uint32_t)g)), (uint32_t)g);
            const float u = fmaf((float)(word >> 4), 3.725290298461914e-09f, 1.862645149230957e-09f);
            const float t_hat = -__logf(u);
            const float base_lo = fmaxf(t_hat - fmaf(t_hat, 1e-6f, 2.5e-7f), 0.0f) * 0.0625f;
            const float need = tau + __logf(fmaxf(base_lo, 1e-37f)) - 2e-4f;   // tau - (upper bound of G_max)
            const uint32_t apos = word & 15u;
            if (ub[g] != ub[g]) nan_flag = 1;                  // the bound is NaN exactly when the group holds one
            // the same bound for the raw values (value * inv_temp >= need), rounded down; finite: -inf, NaN never pass
            const float need_f = fmaxf(need * temp - 2e-6f * fabsf(need * temp), -3.4028234663852886e38f);
            uint32_t todo = group_mask_ge(grp, need_f);
            if (todo) {
                int slot_t = atomicAdd(&n_task, __popc(todo));
                while (todo) {
                    const uint32_t j = (uint32_t)__ffs(todo) - 1u;
                    todo &= todo - 1;
                    if (slot_t < kTaskCap) {
                        tk_x[slot_t] = (uint32_t)(g * 16) + j + (j == apos ? 0x80000000u : 0u);
                        tk_base[slot_t] = base_lo;
                        tk_word[slot_t] = word;
                    }
                    ++slot_t;
                }
            }
        }
        __syncthreads();
        const int nt = n_task;
        general = nt > kTaskCap;
        if (!general) {
            for (int i = tid; i < nt; i += kScanThreads) {
                const uint32_t xe = tk_x[i];
                const uint32_t x = xe & 0x7FFFFFFFu;
                uint32_t w = 0;
                bool keep = true;
                const float raw_u = RowIO<T>::scalar(row, (int)x);   // an L2 hit, in flight during the Philox rounds
                const float raw = raw_u * inv_temp;
                if (!(xe & 0x80000000u)) {
                    w = fine_word_rk(a, key, node, x);
                    const float uu = fmaf((float)w, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
                    const float t_hat = -__logf(uu);
                    const float t_lo = fmaxf(t_hat - fmaf(t_hat, 1e-6f, 2.5e-7f), 0.0f);
                    const float y_hi = __expf(raw - tau) * 1.0002f;   // upper bound of exp(value - tau)
                    keep = tk_base[i] + t_lo <= y_hi;
                }
                if (keep) {
                    const int slot = atomicAdd(&n_fin, 1);
                    if (slot < kFinCap) { fin_x[slot] = xe; fin_w[slot] = w; fin_raw[slot] = raw_u; fin_word[slot] = tk_word[i]; }
                }
            }
            __syncthreads();
            const int nf = n_fin;
            general = nf > kFinCap;
            if (!general) {
                for (int i = tid; i < nf; i += kScanThreads) {
                    const uint32_t xe = fin_x[i];
                    const int x = (int)(xe & 0x7FFFFFFFu);
                    const float base = neg_log_group_uniform_f32(fin_word[i]) * 0.0625f;
                    const float raw_u = fin_raw[i];
                    const float raw = raw_u * inv_temp;
                    const float t_x = (xe & 0x80000000u) ? 0.0f : neg_log_uniform_f32(fin_w[i]);
                    const float pert = raw - logf(base + t_x);
                    if (pert >= tau) {
                        const int sidx = atomicAdd(&n_surv, 1);
                        if (sidx < kSurvCap) { sv_val[sidx] = pert; sv_idx[sidx] = x; sv_raw[sidx] = raw_u; }
                    }
                }
                __syncthreads();
                general = n_surv > kSurvCap;
            }
        }
        if (general) {  // start over in the general path
            __syncthreads();
            if (tid == 0) n_surv = 0;
            __syncthreads();
        }
    }

    int ns = n_surv;
    for (int attempt = 0; general && attempt < 16; ++attempt) {
        // the queued candidate groups, or (when they did not fit the queue) every group whose bound reaches tau
        const bool queued = n_queued <= kCandCap;
        const int n_items = queued ? n_queued : n_groups;
        for (int i = tid; i < n_items; i += kScanThreads) {
            int g = i;
            if (queued) g = cand[i];
            else if (ub[i] < tau) continue;
            process_group(g);
        }
        __syncthreads();
        ns = n_surv;
        if (ns <= kSurvCap) break;
        // more elements reach tau than fit: raise tau to the k-th largest of those kept (still a lower bound)
        float my = kNegInf;
        for (int e = tid; e < kSurvCap; e += kScanThreads) {
            const float mv = sv_val[e];
            const int mi = sv_idx[e];
            int rnk = 0;
            for (int f = 0; f < kSurvCap; ++f) rnk += better(sv_val[f], sv_idx[f], mv, mi) ? 1 : 0;
            if (rnk == k - 1) my = mv;
        }
        const float raised = block_max<kScanThreads>(my, red_f);
        __syncthreads();
        tau = fmaxf(tau, raised);
        if (tid == 0) n_surv = 0;
        __syncthreads();
        ns = 0;
    }
    if (ns > kSurvCap) ns = kSurvCap;

    const float lse = NEED_LSE ? lse_sh : 0.0f;   // written before the barriers that end the stages above

    // ---- rank the survivors, write the picks ----------------------------------------------------------------------------
    const int total = ns < k ? ns : k;
    const int64_t o = ((int64_t)b * a.R + r) * a.max_k;
    const float shift = (a.subtract_lse && NEED_LSE) ? lse : 0.0f;
    for (int e = tid; e < ns; e += kScanThreads) {
        const float mv = sv_val[e];
        const int mi = sv_idx[e];
        int rnk = 0;
        for (int f = 0; f < ns; ++f) rnk += better(sv_val[f], sv_idx[f], mv, mi) ? 1 : 0;
        if (rnk < k) {
            a.out_token[o + rnk] = mi;
            if (a.node_token) a.node_token[(int64_t)b * a.node_stride + a.child_base[r] + rnk] = mi;
            if (a.out_perturbed) a.out_perturbed[o + rnk] = mv - shift;
            if (a.out_value) a.out_value[o + rnk] = a.raw_values ? sv_raw[e] : fmaf(sv_raw[e], inv_temp, -shift);
        }
    }
    if (tid >= total && tid < a.max_k) {
        a.out_token[o + tid] = -1;
        if (a.node_token && tid < k) a.node_token[(int64_t)b * a.node_stride + a.child_base[r] + tid] = -1;
        if (a.out_perturbed) a.out_perturbed[o + tid] = kNegInf;
        if (a.out_value) a.out_value[o + tid] = kNegInf;
    }
    if (tid == 0) {
        if (a.out_lse) a.out_lse[(int64_t)b * a.R + r] = NEED_LSE ? lse : 0.0f;
        int st = 0;
        if (nan_flag) st |= 1;       // RSD_ST_NAN_INPUT
        if (total < k) st |= 2;      // RSD_ST_FEWER_THAN_K
        if (a.row_status) a.row_status[(int64_t)b * a.R + r] = st & 1;
        else if (st) atomicOr(&a.status[b], st);
    }
}

// ---------------------------------------------------------------------------------------------------------
// Stochastic Beam Search level, per-sequence epilogue.
// For a fixed parent psi is increasing in phi~ (Theorem 3.2's argument), so the W best pairs over all parents are
// among each parent's own W best by phi~.  The scan above leaves those n_par * W finalists in scratch; this kernel
// recomputes their noise in double, applies the truncation T of Eq. 11 in the stable form
//   w = log1p(-exp(phi~ - Z)),  v = Gamma - phi~ + w,  psi = Gamma - max(v, 0) - log1p(exp(-|v|)),
// and keeps the W best by (psi desc, parent asc, token asc).
// ---------------------------------------------------------------------------------------------------------
struct SbsEpilogueArgs {
    int n_par, W, is_logprob;
    int64_t fin_seq_stride;    // elements between sequences in fin_token / fin_value / fin_pert (n_par * W for one level)
    int64_t row_seq_stride;    // elements between sequences in fin_lse / row_status (n_par for one level)
    int64_t state_stride;      // elements between sequences in sum_in / gamma_in (n_par for one level)
    int64_t out_state_stride;  // elements between sequences in sum_out / gamma_out (W; 0 when they hold one sequence)
    double inv_temp;           // 1 / temperature of the parents' rows (1: none)
    int32_t first_parent_node;
    uint32_t seed_lo, seed_hi, step, seq_base;
    const int32_t* fin_token;  // [B][n_par][W]
    const float* fin_value;    // [B][n_par][W] the row's own value at the finalist
    const float* fin_pert;     // [B][n_par][W] value + noise in fp32 (decreasing within a parent)
    const float* fin_lse;      // [B][n_par]
    const int32_t* row_status; // [B][n_par] status bits of the row scans
    const float* sum_in;       // [B][n_par] or null
    const float* gamma_in;     // [B][n_par] or null
    int32_t* out_token;   // [B][out_stride]
    int32_t* out_parent;  // [B][out_stride], parent_base added
    int64_t out_stride;
    int32_t parent_base;
    float* sum_out;
    float* gamma_out;
    int32_t* out_count;
    int32_t* status;
};

constexpr int kEpilogueThreads = 128;

// bytes of shared memory one level needs in sbs_epilogue_body, rounded up to 16
__host__ __device__ inline size_t sbs_level_scratch_bytes(int n_par, int W) {
    return (((size_t)n_par * W * 32 + (size_t)n_par * 12) + 15) & ~(size_t)15;
}

// order-preserving map of a double to an unsigned integer (for an atomic maximum), and back; 0 stands for "none"
__device__ __forceinline__ unsigned long long double_to_ordered(double v) {
    const unsigned long long u = (unsigned long long)__double_as_longlong(v);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
__device__ __forceinline__ double ordered_to_double(unsigned long long k) {
    if (k == 0) return -__longlong_as_double(0x7FF0000000000000LL);
    return __longlong_as_double((long long)((k >> 63) ? (k & 0x7FFFFFFFFFFFFFFFull) : ~k));
}

// One level for sequence b, by a block of kEpilogueThreads threads; sm_d: sbs_level_scratch_bytes(n_par, W) bytes.
__device__ __forceinline__ void sbs_epilogue_body(const SbsEpilogueArgs& a, const int b, double* sm_d) {
    const int F = a.n_par * a.W;
    // the finalists that pass the first test are gathered in a list; entry i of the arrays below belongs to list[i]
    double* s_pert = sm_d;                   // [F] phi~
    double* s_phi = sm_d + F;                // [F] phi
    double* s_psi = sm_d + 2 * F;            // [F] psi
    unsigned long long* s_z = (unsigned long long*)(sm_d + 3 * F);   // [n_par] largest phi~ of the parent, ordered
    int* s_list = (int*)(s_z + a.n_par);     // [F] finalist index f = parent * W + place
    int* s_tok = s_list + F;                 // [F] its token
    float* s_gam = (float*)(s_tok + F);      // [n_par]
    const int tid = threadIdx.x;
    const int64_t fin_off = (int64_t)b * a.fin_seq_stride, row_off = (int64_t)b * a.row_seq_stride,
                  state_off = (int64_t)b * a.state_stride;
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};

    // A child enters the beam only if its psi reaches the W-th best psi of the level.  The best child of parent j has
    // psi = Gamma_j exactly, so that bound is at least L = the W-th largest Gamma among the parents that deliver a
    // child (valid parent, at least one finalist); L = -inf when fewer than W do.  Finalists that a cheap fp32 test
    // shows to lie clearly below L are dropped before the double-precision work; a parent's best finalist is
    // always kept.
    __shared__ float s_L;
    __shared__ int s_row_bits, s_n;
    if (tid == 0) { s_L = kNegInf; s_row_bits = 0; s_n = 0; }
    for (int kp = tid; kp < a.n_par; kp += kEpilogueThreads) {
        const float sg = a.sum_in ? a.sum_in[state_off + kp] : 0.0f;
        const float gm = a.gamma_in ? a.gamma_in[state_off + kp] : 0.0f;
        // a parent slot that the level above left empty (its sum or truncated Gumbel is -inf) has no children
        const bool delivers = a.fin_token[fin_off + (int64_t)kp * a.W] >= 0 && sg > kNegInf && gm > kNegInf;
        s_gam[kp] = delivers ? gm : kNegInf;
        s_z[kp] = 0;
    }
    __syncthreads();
    for (int kp = tid; kp < a.n_par; kp += kEpilogueThreads) {
        if (const int bits = a.row_status[row_off + kp]) atomicOr(&s_row_bits, bits);
        const float g = s_gam[kp];
        int rank = 0;
        for (int j = 0; j < a.n_par; ++j) {
            const float o = s_gam[j];
            rank += (o > g || (o == g && j < kp)) ? 1 : 0;
        }
        if (rank == a.W - 1 && g > kNegInf) s_L = g;
    }
    __syncthreads();
    const float L = s_L;

    for (int f = tid; f < F; f += kEpilogueThreads) {
        const int kpar = f / a.W;
        int x = a.fin_token[fin_off + f];
        if (s_gam[kpar] == kNegInf) x = -1;   // s_gam is -inf exactly for the slots that deliver nothing
        if (x >= 0 && L > kNegInf && f != kpar * a.W) {
            // psi_f < L  <=>  exp(-phi~_f) - exp(-Z) > exp(-L) - exp(-Gamma_k), with Z - phi~_f = the gap d between
            // the parent's best and this finalist's fp32 perturbed values; margins cover the fp32 arithmetic
            const float sg = a.sum_in ? a.sum_in[state_off + kpar] : 0.0f;
            const float gm = a.gamma_in ? a.gamma_in[state_off + kpar] : 0.0f;
            const float lse = a.is_logprob ? 0.0f : a.fin_lse[row_off + kpar];
            const float u0 = a.fin_pert[fin_off + (int64_t)kpar * a.W];
            const float d_lo = (u0 - a.fin_pert[fin_off + f]) - 1e-4f;
            if (d_lo > 0.0f) {
                const float z = sg - lse + u0;
                const float rhs = expf(-L + 1e-3f) - expf(-gm);
                if (rhs <= 0.0f || -z + logf(expm1f(d_lo)) > logf(rhs) + 1e-2f) x = -1;   // cannot reach the beam
            }
        }
        if (x >= 0) s_list[atomicAdd(&s_n, 1)] = f;   // the order of the list does not matter below
    }
    __syncthreads();
    const int n = s_n;

    // phi and phi~ of the listed finalists, with the noise recomputed in double; Z = the parent's largest phi~
    for (int i = tid; i < n; i += kEpilogueThreads) {
        const int f = s_list[i], kpar = f / a.W;
        const int x = a.fin_token[fin_off + f];
        const double sigma = a.sum_in ? (double)a.sum_in[state_off + kpar] : 0.0;
        const double lse = a.is_logprob ? 0.0 : (double)a.fin_lse[row_off + kpar];
        const uint32_t node = (uint32_t)(a.first_parent_node + kpar);
        const uint32_t word = coarse_word(key, node, (uint32_t)x >> 4);
        const double t_elem = (((uint32_t)x & 15u) != (word & 15u))
                                  ? neg_log_uniform_f64(fine_word(key, node, (uint32_t)x)) : 0.0;
        const double phi = sigma + ((double)a.fin_value[fin_off + f] * a.inv_temp - lse);
        const double pert = phi - log(neg_log_group_uniform_f64(word) * 0.0625 + t_elem);
        s_tok[i] = x;
        s_phi[i] = phi;
        s_pert[i] = pert;
        atomicMax(&s_z[kpar], double_to_ordered(pert));
    }
    __syncthreads();
    for (int i = tid; i < n; i += kEpilogueThreads) {
        const int kpar = s_list[i] / a.W;
        const double z = ordered_to_double(s_z[kpar]);
        const double gamma = a.gamma_in ? (double)a.gamma_in[state_off + kpar] : 0.0;
        const double pert = s_pert[i];
        const double d = pert - z;
        double psi = gamma;
        if (!(d >= 0.0)) {
            const double w = log1p(-exp(d));
            const double v = gamma - pert + w;
            psi = gamma - fmax(v, 0.0) - log1p(exp(-fabs(v)));
        }
        s_psi[i] = psi;
    }
    __syncthreads();
    // Rank by (psi desc, parent asc, token asc); the finalists of a parent are neighbours in f, so f orders the
    // parents, and within a parent the token decides.
    for (int i = tid; i < n; i += kEpilogueThreads) {
        const double psi = s_psi[i];
        const int f = s_list[i], x = s_tok[i], kpar = f / a.W;
        const int own = kpar * a.W;   // first finalist of f's parent
        int rank = 0;
#pragma unroll 4
        for (int e = 0; e < n; ++e) {
            const double pe = s_psi[e];
            const int fe = s_list[e];
            const bool tie_first = fe < own || (fe < own + a.W && s_tok[e] < x);   // earlier parent, or same parent and smaller token
            rank += (pe > psi || (pe == psi && tie_first)) ? 1 : 0;
        }
        if (rank < a.W) {
            const int64_t o = (int64_t)b * a.out_state_stride + rank;
            a.out_token[(int64_t)b * a.out_stride + rank] = x;
            a.out_parent[(int64_t)b * a.out_stride + rank] = a.parent_base + kpar;
            a.sum_out[o] = (float)s_phi[i];
            a.gamma_out[o] = (float)psi;
        }
    }
    const int cnt = n < a.W ? n : a.W;
    if (tid >= cnt && tid < a.W) {
        const int64_t o = (int64_t)b * a.out_state_stride + tid;
        a.out_token[(int64_t)b * a.out_stride + tid] = -1;
        a.out_parent[(int64_t)b * a.out_stride + tid] = -1;
        a.sum_out[o] = kNegInf;
        a.gamma_out[o] = kNegInf;
    }
    if (tid == 0) {
        a.status[b] = (s_row_bits & 1) | (cnt < a.W ? 2 : 0);  // RSD_ST_NAN_INPUT, RSD_ST_FEWER_THAN_K
        a.out_count[b] = cnt;
    }
}


static __global__ void __launch_bounds__(kEpilogueThreads) sbs_epilogue_kernel(const SbsEpilogueArgs a) {
    extern __shared__ double sm_d[];
    sbs_epilogue_body(a, blockIdx.x, sm_d);
}

// All L levels of one Stochastic Beam Search tree (Algorithm 8's level loop around Algorithm 9) for rows that exist
// before drafting starts: the parent rows of every level were scanned in one launch (row r of a sequence is flat node
// r: the root, then W slots per level), and this kernel runs the levels' epilogues in order, one block per sequence.
// The sequence log-probabilities and truncated Gumbels (Eqs. 10-12) travel from level to level through two pairs of
// W-element arrays in shared memory used in turn; level l writes the tokens and parents of flat nodes
// 1 + l W .. (l + 1) W.  When `staged` is set the sequence's finalists (P W tokens, values and perturbed values, P
// log-sum-exps and row flags) are copied to shared memory once, so that no level waits for global memory.
struct SbsChainArgs {
    SbsEpilogueArgs lvl;        // level-independent fields; the per-level ones are filled in by the kernel
    int L, P;                   // levels; parent rows per sequence, 1 + (L - 1) W
    int B;
    int staged;                 // 1: the dynamic shared memory also holds the finalists' copies
    int32_t* node_token;        // [B][node_stride]
    int32_t* node_parent;
    int64_t node_stride;
    int32_t* level_count;       // [L][B]
    int32_t* level_status;      // [L][B]
    int32_t* status;            // [B]: OR over the levels
    float* sum_out;             // [B][W] of the last level, or null
    float* gamma_out;
};

// dynamic shared memory of sbs_chain_kernel
__host__ __device__ inline size_t sbs_chain_smem_bytes(int W, int P, bool staged) {
    return sbs_level_scratch_bytes(W, W) + (size_t)4 * W * 4 + (staged ? (size_t)P * W * 12 + (size_t)P * 8 : 0);
}

static __global__ void __launch_bounds__(kEpilogueThreads) sbs_chain_kernel(const SbsChainArgs c) {
    extern __shared__ double sm_d[];
    const int b = blockIdx.x, W = c.lvl.W, tid = threadIdx.x, F = c.P * W;
    float* const state = (float*)((unsigned char*)sm_d + sbs_level_scratch_bytes(W, W));   // sum[2][W], gamma[2][W]
    int32_t* const s_tok = (int32_t*)(state + 4 * W);
    float* const s_val = (float*)(s_tok + F);
    float* const s_pert = s_val + F;
    float* const s_lse = s_pert + F;
    int32_t* const s_rs = (int32_t*)(s_lse + c.P);
    if (c.staged) {
        const int64_t f0 = (int64_t)b * F, r0 = (int64_t)b * c.P;
        for (int i = tid; i < F; i += kEpilogueThreads) {
            s_tok[i] = c.lvl.fin_token[f0 + i];
            s_val[i] = c.lvl.fin_value[f0 + i];
            s_pert[i] = c.lvl.fin_pert[f0 + i];
        }
        for (int i = tid; i < c.P; i += kEpilogueThreads) {
            s_lse[i] = c.lvl.fin_lse[r0 + i];
            s_rs[i] = c.lvl.row_status[r0 + i];
        }
        __syncthreads();
    }
    int st = 0;
    for (int l = 0; l < c.L; ++l) {
        SbsEpilogueArgs a = c.lvl;
        const int first = l == 0 ? 0 : 1 + (l - 1) * W;     // flat node of the level's parent slot 0
        a.n_par = l == 0 ? 1 : W;
        a.first_parent_node = first;
        if (c.staged) {
            a.fin_seq_stride = 0;
            a.row_seq_stride = 0;
            a.fin_token = s_tok + first * W;
            a.fin_value = s_val + first * W;
            a.fin_pert = s_pert + first * W;
            a.fin_lse = s_lse + first;
            a.row_status = s_rs + first;
        } else {
            a.fin_token = c.lvl.fin_token + (int64_t)first * W;
            a.fin_value = c.lvl.fin_value + (int64_t)first * W;
            a.fin_pert = c.lvl.fin_pert + (int64_t)first * W;
            a.fin_lse = c.lvl.fin_lse + first;
            a.row_status = c.lvl.row_status + first;
        }
        a.state_stride = 0;
        a.sum_in = l == 0 ? nullptr : state + ((l + 1) & 1) * W;
        a.gamma_in = l == 0 ? nullptr : state + (2 + ((l + 1) & 1)) * W;
        const bool last = l == c.L - 1;
        a.out_state_stride = 0;
        a.sum_out = state + (l & 1) * W;
        a.gamma_out = state + (2 + (l & 1)) * W;
        a.out_token = c.node_token + 1 + (int64_t)l * W;
        a.out_parent = c.node_parent + 1 + (int64_t)l * W;
        a.out_stride = c.node_stride;
        a.parent_base = first;
        a.out_count = c.level_count + (int64_t)l * c.B;
        a.status = c.level_status + (int64_t)l * c.B;
        sbs_epilogue_body(a, b, sm_d);
        __syncthreads();   // the level's outputs are the next level's inputs
        if (tid == 0) st |= a.status[b];
        if (last && tid < W) {
            if (c.sum_out) c.sum_out[(int64_t)b * W + tid] = a.sum_out[tid];
            if (c.gamma_out) c.gamma_out[(int64_t)b * W + tid] = a.gamma_out[tid];
        }
    }
    if (tid == 0) c.status[b] = st;
}

}  // namespace rsd
