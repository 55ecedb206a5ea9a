// Device-side building blocks shared by the RSD kernels: the counter-based random streams, 16-element row
// loads for fp32 and bf16 storage, and warp/block reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rsd {

constexpr uint32_t kTagGumbelCoarse = 0u, kTagGumbelFine = 1u, kTagAccept = 2u, kTagResample = 3u;
constexpr uint32_t kTagFinalGumbelCoarse = 4u, kTagFinalGumbelFine = 5u;   // Gumbel-Top-1 draw of the last token
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInf = -__builtin_huge_valf();

struct RngKey {
    uint32_t seed_lo, seed_hi, step, seq;  // seq = global sequence index
};

// ---------------------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of
//   (c0,c1,c2,c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0)),  key += Weyl constants.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// counter = (index, node | tag << 28, sequence, step); key = seed
__device__ __forceinline__ uint4 rng_draw(const RngKey& k, uint32_t node, uint32_t tag, uint32_t index) {
    return philox4x32_10(index, (node & 0x0FFFFFFFu) | (tag << 28), k.seq, k.step, k.seed_lo, k.seed_hi);
}

// Gumbel noise, RNG layout 3: the 16 noises of a group of consecutive elements are drawn through the order
// statistics of 16 i.i.d. uniforms.  With t(U) = -ln U,
//     coarse stream: one 32-bit word per group; its upper 28 bits -> U_M = (bits + 1/2) / 2^28, its low 4 bits ->
//         position a of the group's largest noise.  Group g reads word (g >> 5) & 3 of the call with index
//         (g >> 7) * 32 + (g & 31): one call serves groups g, g + 32, g + 64, g + 96 of a block of 128 groups,
//         i.e. the four groups a lane of a warp meets while the warp sweeps 2048 consecutive elements.
//     fine stream (index = x >> 2, word x & 3) -> U_x = (bits + 1/2) / 2^32
//     G_x = -ln( t(U_M) / 16 + [x mod 16 != a] t(U_x) ),
// so the element at position a has the largest noise of its group, -ln(t(U_M) / 16), known from the coarse stream.
__device__ __forceinline__ uint32_t coarse_index(uint32_t g) { return ((g >> 7) << 5) | (g & 31u); }
__device__ __forceinline__ uint32_t coarse_select(const uint4& w, uint32_t g) {
    const uint32_t sel = (g >> 5) & 3u;
    return sel < 2 ? (sel == 0 ? w.x : w.y) : (sel == 2 ? w.z : w.w);
}
__device__ __forceinline__ uint32_t coarse_word(const RngKey& k, uint32_t node, uint32_t g) {
    return coarse_select(rng_draw(k, node, kTagGumbelCoarse, coarse_index(g)), g);
}
__device__ __forceinline__ uint32_t fine_word(const RngKey& k, uint32_t node, uint32_t e) {
    const uint4 w = rng_draw(k, node, kTagGumbelFine, e >> 2);
    const uint32_t sel = e & 3u;
    return sel < 2 ? (sel == 0 ? w.x : w.y) : (sel == 2 ? w.z : w.w);
}

// t = -ln U, U = (bits + 1/2) / 2^32, in fp32 with ~1e-7 relative error (for U >= 1/2 through 1 - U, which is
// exact in fp32 when it is small).
__device__ __forceinline__ float neg_log_uniform_f32(uint32_t bits) {
    if (bits < 0x80000000u) return -logf(((float)bits + 0.5f) * 2.3283064365386963e-10f);
    return -log1pf(-(((float)(~bits) + 0.5f) * 2.3283064365386963e-10f));  // 1 - U = (2^32 - 1 - bits + 1/2) / 2^32
}
__device__ __forceinline__ double neg_log_uniform_f64(uint32_t bits) {
    return -log(((double)bits + 0.5) * (1.0 / 4294967296.0));
}
// the same for the group uniform: U_M = ((word >> 4) + 1/2) / 2^28
__device__ __forceinline__ float neg_log_group_uniform_f32(uint32_t word) {
    const uint32_t bits = word >> 4;
    if (bits < 0x08000000u) return -logf(((float)bits + 0.5f) * 3.725290298461914e-09f);
    return -log1pf(-(((float)(0x0FFFFFFFu - bits) + 0.5f) * 3.725290298461914e-09f));
}
__device__ __forceinline__ double neg_log_group_uniform_f64(uint32_t word) {
    return -log(((double)(word >> 4) + 0.5) * (1.0 / 268435456.0));
}

// ---------------------------------------------------------------------------------------------------------
// 16 consecutive elements of a row as fp32 registers
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float max_nan(float a, float b) {  // NaN if either is NaN
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 32 bytes at a 32-byte aligned address in one request (sm_100: 256-bit global loads)
__device__ __forceinline__ void ld_stream_256(const void* p, uint4& lo, uint4& hi) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
                 : "l"(p));
}

// ---------------------------------------------------------------------------------------------------------
// mbarrier and bulk copy (global -> this block's shared memory; this GPU's own memory, no cluster, no multicast)
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// `bytes` a multiple of 16, both addresses 16-byte aligned; completion counts on `bar`
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
constexpr long long kCopyWaitCycles = 1ll << 31;   // about a second: a copy that has not landed by then never will
// Wait for phase `parity` of `bar`, at most about a second.  A wait that runs out sets *gave_up and returns: the caller
// goes on with whatever the memory holds and reports RSD_ST_TIMEOUT at its next decision point.
__device__ __forceinline__ void wait_bar(unsigned long long* bar, uint32_t parity, int* gave_up) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kCopyWaitCycles) {
            *gave_up = 1;
            return;
        }
    }
}

template <typename T>
struct RowIO;

template <>
struct RowIO<float> {
    static constexpr int kBytes = 4;
    __device__ static __forceinline__ float scalar(const void* row, int x) { return ((const float*)row)[x]; }
    // full, 16-byte aligned group g
    __device__ static __forceinline__ void load16(const void* row, int g, float (&v)[16]) {
        const uint4* p = (const uint4*)((const float*)row + (size_t)g * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 q = ld_stream(p + i);
            v[4 * i + 0] = __uint_as_float(q.x);
            v[4 * i + 1] = __uint_as_float(q.y);
            v[4 * i + 2] = __uint_as_float(q.z);
            v[4 * i + 3] = __uint_as_float(q.w);
        }
    }
};

template <>
struct RowIO<__nv_bfloat16> {
    static constexpr int kBytes = 2;
    __device__ static __forceinline__ float scalar(const void* row, int x) {
        return __uint_as_float((uint32_t)((const uint16_t*)row)[x] << 16);
    }
    __device__ static __forceinline__ void load16(const void* row, int g, float (&v)[16]) {
        const uint4* p = (const uint4*)((const uint16_t*)row + (size_t)g * 16);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint4 q = ld_stream(p + i);
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[8 * i + 2 * j + 0] = __uint_as_float(w[j] << 16);
                v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
            }
        }
    }
};

// Group g of a row of V elements: vector loads when the row is aligned and the group is full, else guarded scalar
// loads padded with -inf.
template <typename T, bool ALIGNED>
__device__ __forceinline__ void load_group(const void* row, int g, int V, float (&v)[16]) {
    if (ALIGNED && (g + 1) * 16 <= V) {
        RowIO<T>::load16(row, g, v);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int x = g * 16 + i;
            v[i] = x < V ? RowIO<T>::scalar(row, x) : kNegInf;
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// reductions
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// Block-wide sum of doubles / max of floats; `scratch` holds one slot per warp; all threads get the result.
template <int NT>
__device__ __forceinline__ double block_sum(double v, double* scratch) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t += scratch[w];  // fixed order: the same on every thread
    return t;
}
template <int NT>
__device__ __forceinline__ float block_max(float v, float* scratch) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = scratch[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) t = fmaxf(t, scratch[w]);
    return t;
}

// order-preserving map float -> uint32 so that atomicMax works on floats of either sign
__device__ __forceinline__ uint32_t float_to_ordered(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_float(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

}  // namespace rsd
