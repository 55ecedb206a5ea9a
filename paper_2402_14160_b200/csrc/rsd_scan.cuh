// Row scan: exact sorted arg-top-k of (row + Gumbel noise) in one pass over the row (Eqs. 6-7, Algorithm 4), and
// the per-sequence epilogue of a Stochastic Beam Search level (Eqs. 10-12, Algorithm 9).
//
// The noise of a group of 16 consecutive elements is drawn through its order statistics (see rsd_device.cuh): one
// Philox call per group gives the group's largest noise and the element that carries it.  The streaming loop
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
constexpr int kQueueCap = 64;  // per-warp candidate queue (a push adds at most 32 to at most 31 pending)
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
    int32_t* out_token;   // [B][R][max_k]
    float* out_perturbed; // [B][R][max_k] or null
    float* out_value;     // [B][R][max_k] or null: the row's own value at each pick
    float* out_lse;       // [B][R] or null
    int32_t* status;      // [B], OR-ed into
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
    __device__ __forceinline__ void load(const void* row, int g, int V, bool aligned_full) {
        if (aligned_full) {
            const uint4* p = (const uint4*)((const float*)row + (size_t)g * 16);
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = ld_stream(p + i);
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
    __device__ __forceinline__ void load(const void* row, int g, int V, bool aligned_full) {
        if (aligned_full) {
            const uint4* p = (const uint4*)((const uint16_t*)row + (size_t)g * 16);
            w[0] = ld_stream(p);
            w[1] = ld_stream(p + 1);
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

// Bounds of the group's largest noise G_max = -ln(t / 16), t = -ln((bits + 1/2) / 2^32), from fast logarithms:
// lo <= G_max <= hi.  (|t_hat - t| <= 2.5e-7 + 1e-6 t covers the conversion and lg2.approx; the outer logarithm
// adds at most 2e-6; hi is +huge when t_hat is too small to bound.)
__device__ __forceinline__ void group_noise_bounds(uint32_t bits, float& lo, float& hi) {
    const float u = fmaf((float)bits, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
    const float t_hat = -__logf(u);
    const float dt = fmaf(t_hat, 1e-6f, 2.5e-7f);
    hi = -__logf(fmaxf(t_hat - dt, 1e-37f) * 0.0625f) + 2e-4f;
    lo = -__logf((t_hat + dt) * 0.0625f) - 2e-4f;
}

// One block per row.
template <typename T, bool ALIGNED, bool NEED_LSE>
__global__ void __launch_bounds__(kScanThreads, 8) scan_topk_kernel(const ScanArgs a) {
    extern __shared__ float ub[];                    // [n_groups] upper bound of each group's perturbed values
    __shared__ int cand[kCandCap];                   // groups whose bound reaches tau
    __shared__ uint32_t tk_x[kTaskCap];              // element index | (it carries the group's largest noise) << 31
    __shared__ float tk_base[kTaskCap];              // lower bound of t(U_M) / 16 of the element's group
    __shared__ uint32_t fin_x[kFinCap], fin_w[kFinCap];  // element (same encoding) and its fine-stream word
    __shared__ int n_task, n_fin;
    __shared__ float sv_val[kSurvCap], sv_raw[kSurvCap];
    __shared__ int sv_idx[kSurvCap];
    __shared__ uint32_t bin_max[32];                 // per lane index: largest sample over the warps (ordered encoding)
    __shared__ float red_f[kScanWarps];
    __shared__ double red_d[kScanWarps];
    __shared__ int n_cand, n_surv, nan_flag;

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
    __syncthreads();

    // ---- streaming loop: one group per thread per sweep ------------------------------------------------------------
    float best = kNegInf;                  // largest exact sample of this thread (value(a) + lower bound of G_max)
    float lse_m = kNegInf, lse_s = 0.0f;   // running log-sum-exp of this thread's elements
    bool saw_nan = false;
    // work on one group whose 16 values are in `cur`
    auto body = [&](const Packed<T>& cur, int g) {
        const uint4 cw = philox_row(a, pr, (uint32_t)g);
        float g_lo, g_hi;
        group_noise_bounds(cw.x, g_lo, g_hi);
        float gmax = group_max_nan(cur);
        ub[g] = gmax + g_hi;                                   // NaN if the group holds a NaN: looked at later
        best = fmaxf(best, group_element(cur, (int)(cw.y & 15u)) + g_lo);  // fmaxf drops NaN
        if (NEED_LSE) {
            float v[16];
            cur.unpack(v);
            if (gmax != gmax) {  // NaN counts as -inf
                gmax = kNegInf;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (v[j] != v[j]) v[j] = kNegInf;
                    gmax = fmaxf(gmax, v[j]);
                }
            }
            // branch-free online softmax: rescale by exp(old max - new max) (1 when the max does not grow; the
            // running sum is 0 while the max is -inf), then add this group's exponentials
            const float new_m = fmaxf(lse_m, gmax);
            const float scale = (new_m > lse_m && lse_m > kNegInf) ? ex2_approx((lse_m - new_m) * kLog2e) : 1.0f;
            lse_m = new_m;
            {
                const float c = (lse_m > kNegInf) ? lse_m * kLog2e : 0.0f;   // all -inf so far: terms are exp2(-inf) = 0
                const unsigned long long l2 = f32x2(kLog2e, kLog2e), c2 = f32x2(-c, -c);
                unsigned long long acc = f32x2(0.0f, 0.0f);
#pragma unroll
                for (int j = 0; j < 16; j += 2) {  // two elements per fma / add
                    float e0, e1;
                    split_f32x2(fma_f32x2(f32x2(v[j], v[j + 1]), l2, c2), e0, e1);
                    acc = add_f32x2(acc, f32x2(ex2_approx(e0), ex2_approx(e1)));
                }
                float s0, s1;
                split_f32x2(acc, s0, s1);
                lse_s = fmaf(lse_s, scale, s0 + s1);
            }
        }
    };
    // Sweeps in which every thread has a group run without bounds checks, two per turn on alternating buffers
    // (loads are issued one sweep ahead); the ragged last sweep is fetched first and handled last.
    const int n_full = n_groups / kScanThreads;
    const int g_last = n_full * kScanThreads + tid;
    Packed<T> last, buf_a, buf_b;
    if (g_last < n_groups) last.load(row, g_last, V, ALIGNED && (g_last + 1) * 16 <= V);
    if (n_full > 0) buf_a.load(row, tid, V, ALIGNED);
    int it = 0;
    for (; it + 1 < n_full; it += 2) {
        buf_b.load(row, (it + 1) * kScanThreads + tid, V, ALIGNED);
        body(buf_a, it * kScanThreads + tid);
        if (it + 2 < n_full) buf_a.load(row, (it + 2) * kScanThreads + tid, V, ALIGNED);
        body(buf_b, (it + 1) * kScanThreads + tid);
    }
    if (it < n_full) body(buf_a, it * kScanThreads + tid);
    if (g_last < n_groups) body(last, g_last);

    // ---- tau: a lower bound of the k-th largest perturbed value from the threads' samples -------------------------
    // The samples belong to distinct elements.  They are folded into 32 bins (one per lane index, maximum over the
    // warps); the k-th largest bin maximum is at most the k-th largest sample, hence at most the k-th largest
    // perturbed value of the row.  Every warp sorts the 32 bin maxima itself, so one barrier is enough.
    if (best > kNegInf) atomicMax(&bin_max[lane], float_to_ordered(best));
    if (NEED_LSE) {
        const float wm = warp_max(lse_m);
        if (lane == 0) red_f[warp] = wm;
    }
    __syncthreads();
    float lse_M = kNegInf;
    if (NEED_LSE) {
#pragma unroll
        for (int w = 0; w < kScanWarps; ++w) lse_M = fmaxf(lse_M, red_f[w]);
    }
    float tau;
    {
        float v = ordered_to_float(bin_max[lane]);  // bitonic sort across the warp, ascending
#pragma unroll
        for (int k2 = 2; k2 <= 32; k2 <<= 1) {
#pragma unroll
            for (int j = k2 >> 1; j > 0; j >>= 1) {
                const float other = __shfl_xor_sync(0xFFFFFFFFu, v, j);
                const bool up = (lane & k2) == 0, lower = (lane & j) == 0;
                v = (lower == up) ? fminf(v, other) : fmaxf(v, other);
            }
        }
        tau = __shfl_sync(0xFFFFFFFFu, v, 32 - k);  // k-th largest (k <= 32)
    }

    // ---- candidate groups ---------------------------------------------------------------------------------------------
    for (int it = 0; it < n_iter; ++it) {
        const int g = it * kScanThreads + tid;
        if (g < n_groups) {
            const float u = ub[g];
            if (u >= tau || u != u) {
                const int slot = atomicAdd(&n_cand, 1);
                if (slot < kCandCap) cand[slot] = g;
            }
        }
    }
    __syncthreads();
    const int n_queued = n_cand;

    // exact perturbed values of the elements of group g that can reach tau
    auto process_group = [&](int g) {
        Packed<T> grp;
        grp.load(row, g, V, ALIGNED && (g + 1) * 16 <= V);
        const uint4 cw = philox_row(a, pr, (uint32_t)g);
        const float base = neg_log_uniform_f32(cw.x) * 0.0625f;   // t(U_M) / 16
        const float g_max = -logf(base);
        const int apos = (int)(cw.y & 15u);
        // elements whose value plus the group's largest noise reaches tau (NaN compares false both ways: flagged)
        uint32_t todo = 0;
        {
            float v[16];
            grp.unpack(v);
            const float need = tau - g_max - 1e-5f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (v[j] != v[j]) saw_nan = true;
                else if (v[j] > kNegInf && v[j] >= need) todo |= 1u << j;
            }
        }
        while (todo) {
            const int j = __ffs(todo) - 1;
            todo &= todo - 1;
            const int x = g * 16 + j;
            const float raw = group_element(grp, j);
            float pert = raw + g_max;
            if (j != apos) pert = raw - logf(base + neg_log_uniform_f32(fine_word(key, node, (uint32_t)x)));
            if (pert >= tau) {
                const int sidx = atomicAdd(&n_surv, 1);
                if (sidx < kSurvCap) { sv_val[sidx] = pert; sv_idx[sidx] = x; sv_raw[sidx] = raw; }
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
            grp.load(row, g, V, ALIGNED && (g + 1) * 16 <= V);
            const uint4 cw = philox_row(a, pr, (uint32_t)g);
            const float u = fmaf((float)cw.x, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
            const float t_hat = -__logf(u);
            const float base_lo = fmaxf(t_hat - fmaf(t_hat, 1e-6f, 2.5e-7f), 0.0f) * 0.0625f;
            const float need = tau + __logf(fmaxf(base_lo, 1e-37f)) - 2e-4f;   // tau - (upper bound of G_max)
            const uint32_t apos = cw.y & 15u;
            float v[16];
            grp.unpack(v);
            uint32_t todo = 0;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (v[j] != v[j]) saw_nan = true;
                else if (v[j] > kNegInf && v[j] >= need) todo |= 1u << j;
            }
            while (todo) {
                const uint32_t j = (uint32_t)__ffs(todo) - 1u;
                todo &= todo - 1;
                const int slot = atomicAdd(&n_task, 1);
                if (slot < kTaskCap) {
                    tk_x[slot] = (uint32_t)(g * 16) + j + (j == apos ? 0x80000000u : 0u);
                    tk_base[slot] = base_lo;
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
                if (!(xe & 0x80000000u)) {
                    w = fine_word(key, node, x);
                    const float raw = RowIO<T>::scalar(row, (int)x);
                    const float uu = fmaf((float)w, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
                    const float t_hat = -__logf(uu);
                    const float t_lo = fmaxf(t_hat - fmaf(t_hat, 1e-6f, 2.5e-7f), 0.0f);
                    const float y_hi = __expf(raw - tau) * 1.0002f;   // upper bound of exp(value - tau)
                    keep = tk_base[i] + t_lo <= y_hi;
                }
                if (keep) {
                    const int slot = atomicAdd(&n_fin, 1);
                    if (slot < kFinCap) { fin_x[slot] = xe; fin_w[slot] = w; }
                }
            }
            __syncthreads();
            const int nf = n_fin;
            general = nf > kFinCap;
            if (!general) {
                for (int i = tid; i < nf; i += kScanThreads) {
                    const uint32_t xe = fin_x[i];
                    const int x = (int)(xe & 0x7FFFFFFFu);
                    const uint4 cw = philox_row(a, pr, (uint32_t)x >> 4);
                    const float base = neg_log_uniform_f32(cw.x) * 0.0625f;
                    const float raw = RowIO<T>::scalar(row, x);
                    const float t_x = (xe & 0x80000000u) ? 0.0f : neg_log_uniform_f32(fin_w[i]);
                    const float pert = raw - logf(base + t_x);
                    if (pert >= tau) {
                        const int sidx = atomicAdd(&n_surv, 1);
                        if (sidx < kSurvCap) { sv_val[sidx] = pert; sv_idx[sidx] = x; sv_raw[sidx] = raw; }
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
        if (n_queued <= kCandCap) {
            for (int i = tid; i < n_queued; i += kScanThreads) process_group(cand[i]);
        } else {  // too many candidate groups for the queue: each thread handles its own
            for (int it = 0; it < n_iter; ++it) {
                const int g = it * kScanThreads + tid;
                if (g < n_groups) {
                    const float u = ub[g];
                    if (u >= tau || u != u) process_group(g);
                }
            }
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

    float lse = 0.0f;
    if (NEED_LSE) {
        const float M = lse_M;
        const float scaled = (lse_m > kNegInf) ? lse_s * ex2_approx((lse_m - M) * kLog2e) : 0.0f;
        const double S = block_sum<kScanThreads>((double)scaled, red_d);
        lse = (M > kNegInf && S > 0.0) ? (float)((double)M + log(S)) : kNegInf;
    }
    if (saw_nan) nan_flag = 1;
    __syncthreads();

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
            if (a.out_value) a.out_value[o + rnk] = sv_raw[e] - shift;
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
        if (st) atomicOr(&a.status[b], st);
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
    int32_t first_parent_node;
    uint32_t seed_lo, seed_hi, step, seq_base;
    const int32_t* fin_token;  // [B][n_par][W]
    const float* fin_value;    // [B][n_par][W] the row's own value at the finalist
    const float* fin_lse;      // [B][n_par]
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

__global__ void __launch_bounds__(kEpilogueThreads) sbs_epilogue_kernel(const SbsEpilogueArgs a) {
    extern __shared__ double sm_d[];  // [F] phi~ then psi, [F] phi
    const int F = a.n_par * a.W;
    double* s_val = sm_d;
    double* s_phi = sm_d + F;
    int* s_tok = (int*)(sm_d + 2 * F);
    const int b = blockIdx.x, tid = threadIdx.x;
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    const double ninf = -__longlong_as_double(0x7FF0000000000000LL);

    for (int f = tid; f < F; f += kEpilogueThreads) {
        const int kpar = f / a.W;
        const int x = a.fin_token[(int64_t)b * F + f];
        double phi = ninf, pert = ninf;
        if (x >= 0) {
            const double sigma = a.sum_in ? (double)a.sum_in[(int64_t)b * a.n_par + kpar] : 0.0;
            const double lse = a.is_logprob ? 0.0 : (double)a.fin_lse[(int64_t)b * a.n_par + kpar];
            const uint32_t node = (uint32_t)(a.first_parent_node + kpar);
            const uint4 cw = rng_draw(key, node, kTagGumbelCoarse, (uint32_t)x >> 4);
            const double t_elem = (((uint32_t)x & 15u) != (cw.y & 15u))
                                      ? neg_log_uniform_f64(fine_word(key, node, (uint32_t)x)) : 0.0;
            phi = sigma + ((double)a.fin_value[(int64_t)b * F + f] - lse);
            pert = phi - log(neg_log_uniform_f64(cw.x) * 0.0625 + t_elem);
        }
        s_tok[f] = x;
        s_phi[f] = phi;
        s_val[f] = pert;
    }
    __syncthreads();
    // psi of every finalist (Z = the parent's largest phi~)
    double my_psi[8];  // up to 8 finalists per thread: F <= 1024
    int n_mine = 0;
    for (int f = tid; f < F; f += kEpilogueThreads, ++n_mine) {
        const int kpar = f / a.W;
        double z = ninf;
        for (int i = 0; i < a.W; ++i) z = fmax(z, s_val[kpar * a.W + i]);
        const double gamma = a.gamma_in ? (double)a.gamma_in[(int64_t)b * a.n_par + kpar] : 0.0;
        const double pert = s_val[f];
        double psi = ninf;
        if (s_tok[f] >= 0) {
            const double d = pert - z;
            if (d >= 0.0) psi = gamma;
            else {
                const double w = log1p(-exp(d));
                const double v = gamma - pert + w;
                psi = gamma - fmax(v, 0.0) - log1p(exp(-fabs(v)));
            }
        }
        my_psi[n_mine] = psi;
    }
    __syncthreads();
    n_mine = 0;
    for (int f = tid; f < F; f += kEpilogueThreads, ++n_mine) s_val[f] = my_psi[n_mine];
    __syncthreads();
    int valid_here = 0;
    for (int f = tid; f < F; f += kEpilogueThreads) {
        const int x = s_tok[f];
        if (x < 0) continue;
        ++valid_here;
        const double psi = s_val[f];
        int rank = 0;
        for (int e = 0; e < F; ++e) {
            if (s_tok[e] < 0) continue;
            const double pe = s_val[e];
            // order: psi desc, then parent asc, then token asc; e's parent <= f's parent iff e / W <= f / W
            const bool e_first = pe > psi || (pe == psi && (e / a.W < f / a.W || (e / a.W == f / a.W && s_tok[e] < x)));
            rank += e_first ? 1 : 0;
        }
        if (rank < a.W) {
            const int64_t o = (int64_t)b * a.W + rank;
            a.out_token[(int64_t)b * a.out_stride + rank] = x;
            a.out_parent[(int64_t)b * a.out_stride + rank] = a.parent_base + f / a.W;
            a.sum_out[o] = (float)s_phi[f];
            a.gamma_out[o] = (float)psi;
        }
    }
    __shared__ int s_cnt;
    if (tid == 0) s_cnt = 0;
    __syncthreads();
    if (valid_here) atomicAdd(&s_cnt, valid_here);
    __syncthreads();
    const int cnt = s_cnt < a.W ? s_cnt : a.W;
    if (tid >= cnt && tid < a.W) {
        const int64_t o = (int64_t)b * a.W + tid;
        a.out_token[(int64_t)b * a.out_stride + tid] = -1;
        a.out_parent[(int64_t)b * a.out_stride + tid] = -1;
        a.sum_out[o] = kNegInf;
        a.gamma_out[o] = kNegInf;
    }
    if (tid == 0 && cnt < a.W) atomicOr(&a.status[b], 2);  // RSD_ST_FEWER_THAN_K
    if (tid == 0) a.out_count[b] = cnt;
}

}  // namespace rsd
