// Row scan: exact sorted arg-top-k of (row + Gumbel noise) in one pass over the row (Eqs. 6-7, Algorithm 4), and
// the per-sequence epilogue of a Stochastic Beam Search level (Eqs. 10-12, Algorithm 9).
//
// The noise of an element is 32 random bits: a coarse byte (16 elements per Philox call) on top of 24 fine bits
// (4 elements per call).  G is increasing in those bits, so the byte alone bounds G from above.  Every element is
// tested against "value + bound >= tau", where tau is a running lower bound of the k-th largest perturbed value;
// only the few that pass get their fine bits and an exact G.  Nothing that could be among the k largest is ever
// skipped, so the result equals the plain definition (perturb everything, sort) in fp32.
#pragma once
#include <cuda_fp16.h>

#include "rsd_device.cuh"

namespace rsd {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kQueueCap = 64;  // per-warp candidate queue (a push adds at most 32 to at most 31 pending)
constexpr int kMaxRows = 256;
constexpr int kIdxNone = 0x7FFFFFFF;
constexpr int kCandCap = 2048;          // block-level candidate queue of the guessed-threshold pass
constexpr int kSurvCap = 128;           // candidates whose exact value reaches the guessed threshold
constexpr float kSumScale = 4096.0f;    // fixed-point scale of the running sum behind the guess

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

// Sorted list of the 32 best (value, index) pairs seen by a warp: lane i holds the i-th best.
struct WarpTop {
    float v;
    int idx;
    float raw;
    __device__ __forceinline__ void init() { v = kNegInf; idx = kIdxNone; raw = kNegInf; }
    // all lanes call with the same candidate
    __device__ __forceinline__ void insert(float cv, int ci, float craw, int lane) {
        const int pos = __popc(__ballot_sync(0xFFFFFFFFu, better(v, idx, cv, ci)));
        const float uv = __shfl_up_sync(0xFFFFFFFFu, v, 1);
        const int ui = __shfl_up_sync(0xFFFFFFFFu, idx, 1);
        const float ur = __shfl_up_sync(0xFFFFFFFFu, raw, 1);
        if (lane > pos) { v = uv; idx = ui; raw = ur; }
        else if (lane == pos) { v = cv; idx = ci; raw = craw; }
    }
};

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

__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Expected number of elements above the guessed threshold, chosen so that fewer than k is a 1e-5 event.
__device__ __forceinline__ float guess_mean_count(int k) { return (float)k + 4.0f * sqrtf((float)k) + 8.0f; }

// One block per row.  Two ways through the row, with the same result:
//
//  guessed threshold (tried first).  With q(x) = exp(value(x) - ref) and S the sum of q over the elements read so
//    far, tau = ref + ln(S / mu) is exceeded by about mu of those elements' perturbed values (a Poisson count), so
//    it is very likely at most the k-th largest.  An element can reach tau only if its uniform U exceeds
//    exp(-q mu / S) >= 1 - q mu / S; with h the top byte of U that needs 255 - h <= 256 mu q / S, an integer
//    compare per element.  Elements that pass are queued, get their exact noise, and enter the warp's sorted
//    list.  At the end the guess is CHECKED: if the k-th value found is at least the largest tau used, nothing
//    that was skipped could have ranked, and the result is exact.  Otherwise the row is redone the other way.
//
//  running bound.  tau is the k-th largest perturbed value found so far (a true lower bound from the start, so
//    there is nothing to check); the test per element uses the bound of G given its byte.  Slower at the start of
//    a row, used only when the check above fails (fewer than k finite entries, overflow of q, bad luck).
template <typename T, bool ALIGNED, bool NEED_LSE>
__global__ void __launch_bounds__(kScanThreads) scan_topk_kernel(const ScanArgs a) {
    __shared__ uint32_t q_idxh[kScanWarps][kQueueCap];
    __shared__ uint32_t tau_blk;  // order-preserving encoding of the block's best lower bound (running-bound mode)
    __shared__ float m_v[kScanWarps * 32], m_raw[kScanWarps * 32];
    __shared__ int m_idx[kScanWarps * 32];
    __shared__ float red_f[kScanWarps];
    __shared__ double red_d[kScanWarps];
    __shared__ uint32_t cand[kCandCap];       // guessed-threshold pass: queued (index | byte << 24)
    __shared__ float sv_val[kSurvCap], sv_raw[kSurvCap];
    __shared__ int sv_idx[kSurvCap];
    __shared__ uint32_t s_fixed;              // running sum of exp(value - ref), fixed point
    __shared__ int n_cand, n_surv;
    __shared__ float kth_val;
    __shared__ int nan_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / a.R, r = blockIdx.x % a.R;
    const int k = a.k_row[r];
    const uint32_t node = (uint32_t)a.node_row[r];
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    const char* row = (const char*)a.data + ((int64_t)b * a.seq_stride + (int64_t)r * a.row_stride) * RowIO<T>::kBytes;
    const int V = a.V, n_groups = (V + 15) >> 4;
    const int n_iter = (n_groups + kScanThreads - 1) / kScanThreads;

    if (tid == 0) { tau_blk = float_to_ordered(kNegInf); nan_flag = 0; kth_val = kNegInf; s_fixed = 0u; n_cand = 0; n_surv = 0; }

    WarpTop top;
    top.init();
    int q_head = 0, q_count = 0;  // warp-uniform
    bool saw_nan = false;

    // Take up to 32 queued candidates: (bound test with the exact byte,) exact noise, insertion.
    auto drain = [&](int n, bool use_bound) {
        const bool have = lane < n;
        uint32_t idxh = 0;
        if (have) idxh = q_idxh[warp][(q_head + lane) & (kQueueCap - 1)];
        const int idx = (int)(idxh & 0x00FFFFFFu);
        const uint32_t h = idxh >> 24;
        float raw = kNegInf;
        if (have && idx < V) {  // padding of the last group is never read
            raw = RowIO<T>::scalar(row, idx);
            if (raw != raw) { saw_nan = true; raw = kNegInf; }
        }
        bool pass = have && raw > kNegInf;
        if (use_bound) {
            const float tau = fmaxf(__shfl_sync(0xFFFFFFFFu, top.v, k - 1), ordered_to_float(*(volatile uint32_t*)&tau_blk));
            pass = pass && (raw + gumbel_upper_bound(h) >= tau);
        }
        float pert = kNegInf;
        if (pass) pert = raw + gumbel_f32((h << 24) | fine_bits(key, node, (uint32_t)idx));
        unsigned m = __ballot_sync(0xFFFFFFFFu, pass);
        while (m) {
            const int src = __ffs(m) - 1;
            m &= m - 1;
            const float cv = __shfl_sync(0xFFFFFFFFu, pert, src);
            const int ci = __shfl_sync(0xFFFFFFFFu, idx, src);
            const float cr = __shfl_sync(0xFFFFFFFFu, raw, src);
            const float kv = __shfl_sync(0xFFFFFFFFu, top.v, k - 1);
            const int ki = __shfl_sync(0xFFFFFFFFu, top.idx, k - 1);
            if (better(cv, ci, kv, ki)) top.insert(cv, ci, cr, lane);
        }
        q_head = (q_head + n) & (kQueueCap - 1);
        q_count -= n;
        if (use_bound) {
            const float tw = __shfl_sync(0xFFFFFFFFu, top.v, k - 1);
            if (lane == 0 && tw > kNegInf) atomicMax(&tau_blk, float_to_ordered(tw));
        }
        __syncwarp();
    };

    // Merge the warps' lists: every entry learns its rank among all entries; returns the number of picks found.
    int rank = 0;
    bool mine = false;
    auto merge_lists = [&]() -> int {
        __syncthreads();
        m_v[tid] = top.v;
        m_idx[tid] = top.idx;
        m_raw[tid] = top.raw;
        if (tid == 0) kth_val = kNegInf;
        __syncthreads();
        mine = lane < k && top.idx != kIdxNone;
        rank = 0;
        if (mine) {
            for (int w = 0; w < kScanWarps; ++w)
                for (int i = 0; i < k; ++i) {
                    const int e = w * 32 + i;
                    rank += (m_idx[e] != kIdxNone && better(m_v[e], m_idx[e], top.v, top.idx)) ? 1 : 0;
                }
            if (rank == k - 1) kth_val = top.v;
        }
        const int cnt = __syncthreads_count(mine);
        return cnt < k ? cnt : k;
    };

    // ---- reference for the exponentials: the largest value of the first sweep -------------------------------
    Packed<T> first;
    if (tid < n_groups) first.load(row, tid, V, ALIGNED && (tid + 1) * 16 <= V);
    else first.fill_neg_inf();
    float ref;
    {
        float v[16];
        first.unpack(v);
        float vm = kNegInf;
#pragma unroll
        for (int j = 0; j < 16; ++j) vm = fmaxf(vm, v[j]);  // ignores NaN
        ref = block_max<kScanThreads>(vm, red_f);
        if (!(ref > kNegInf) || !(ref < -kNegInf)) ref = 0.0f;
    }

    // ---- attempt 1: guessed threshold ---------------------------------------------------------------------------
    float lse = 0.0f;
    int total = 0;
    bool ok;
    {
        const float mu = guess_mean_count(k);
        const float c_ref = ref * kLog2e;
        const PhiloxRow pr = philox_row_setup(a, (node & 0x0FFFFFFFu) | (kTagGumbelCoarse << 28), key.seq, key.step);
        float lse_acc = 0.0f;  // this lane's share of sum_x exp(value - ref)

        // candidates of one group: bit (j >> 1) + 16 (j & 1) of `pass` <-> element j
        auto push = [&](uint32_t pass, const uint4& cw, int g) {
            while (pass) {
                const int bit = __ffs(pass) - 1;
                pass &= pass - 1;
                const int j = ((bit & 15) << 1) | (bit >> 4);
                const uint32_t word = j < 8 ? (j < 4 ? cw.x : cw.y) : (j < 12 ? cw.z : cw.w);
                const uint32_t h = (word >> (8 * (j & 3))) & 0xFFu;
                const int slot = atomicAdd(&n_cand, 1);
                if (slot < kCandCap) cand[slot] = (uint32_t)(g * 16 + j) | (h << 24);
            }
        };
        // 255 - h_j <= round(x_j) for the 16 scaled values x = K q of a group, two at a time in half precision:
        // (1024 + x_j) >= (1024 + 255 - h_j), where 1024 + c has the bit pattern 0x6400 | c.
        auto byte_test = [&](const float (&x)[16], const uint4& cw) -> uint32_t {
            const uint32_t inv[4] = {~cw.x, ~cw.y, ~cw.z, ~cw.w};
            const __half2 bias = __floats2half2_rn(1024.0f, 1024.0f);
            uint32_t pass = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const __half2 y = __hadd2(__floats2half2_rn(x[2 * i], x[2 * i + 1]), bias);
                const uint32_t b0 = (uint32_t)((2 * i) & 3);
                const uint32_t cbits = __byte_perm(inv[i >> 1], 0x64646464u, 0x4040u | ((b0 + 1u) << 8) | b0);
                const uint32_t m = __hgeu2_mask(y, *reinterpret_cast<const __half2*>(&cbits));
                pass |= m & ((1u << i) | (1u << (16 + i)));
            }
            return pass;
        };
        // one capped term per group: the 32-bit total cannot overflow
        const float lane_cap = 2147483648.0f / (float)n_groups;
        auto add_to_sum = [&](float lane_sum) {
            const uint32_t u = (uint32_t)fminf(lane_sum * kSumScale, lane_cap);  // NaN becomes the cap
            const uint32_t wu = __reduce_add_sync(0xFFFFFFFFu, u);
            if (lane == 0) atomicAdd(&s_fixed, wu);
        };
        auto tree16 = [](const float (&q)[16]) {
            return (((q[0] + q[1]) + (q[2] + q[3])) + ((q[4] + q[5]) + (q[6] + q[7]))) +
                   (((q[8] + q[9]) + (q[10] + q[11])) + ((q[12] + q[13]) + (q[14] + q[15])));
        };

        // first sweep: block-wide sum, then the byte test with K from it
        Packed<T> nxt;
        {
            if (n_iter > 1) {
                const int g2 = tid + kScanThreads;
                if (g2 < n_groups) nxt.load(row, g2, V, ALIGNED && (g2 + 1) * 16 <= V);
                else nxt.fill_neg_inf();
            }
            const bool valid = tid < n_groups;
            uint4 cw = make_uint4(0, 0, 0, 0);
            if (valid) cw = philox_row(a, pr, (uint32_t)tid);
            float q[16];
            first.unpack(q);
#pragma unroll
            for (int j = 0; j < 16; ++j) q[j] = ex2_approx(fmaf(q[j], kLog2e, -c_ref));
            const float lane_sum = tree16(q);
            lse_acc = lane_sum;
            add_to_sum(lane_sum);
            __syncthreads();
            float K = __fdividef(256.0f * mu * kSumScale, (float)*(volatile uint32_t*)&s_fixed);
            if (!(K < 1.0e30f)) K = 1.0e30f;
#pragma unroll
            for (int j = 0; j < 16; ++j) q[j] *= K;
            if (valid) push(byte_test(q, cw), cw, tid);
        }
        for (int it = 1; it < n_iter; ++it) {
            const int g = it * kScanThreads + tid;
            const bool valid = g < n_groups;
            const Packed<T> cur = nxt;
            if (it + 1 < n_iter) {
                const int g2 = g + kScanThreads;
                if (g2 < n_groups) nxt.load(row, g2, V, ALIGNED && (g2 + 1) * 16 <= V);
                else nxt.fill_neg_inf();
            }
            uint4 cw = make_uint4(0, 0, 0, 0);
            if (valid) cw = philox_row(a, pr, (uint32_t)g);
            // K from the sum so far (any earlier value is valid: the threshold only rises)
            const float S = (float)*(volatile uint32_t*)&s_fixed;
            float K = __fdividef(256.0f * mu * kSumScale, S);
            if (!(K < 1.0e30f)) K = 1.0e30f;
            const float e_off = __log2f(K) - c_ref;
            const float inv_K = __fdividef(1.0f, K);
            float q[16];
            cur.unpack(q);
#pragma unroll
            for (int j = 0; j < 16; ++j) q[j] = ex2_approx(fmaf(q[j], kLog2e, e_off));  // K exp(value - ref)
            const float lane_sum = tree16(q) * inv_K;
            lse_acc += lane_sum;
            add_to_sum(lane_sum);
            if (valid) push(byte_test(q, cw), cw, g);
        }

        // end of row: exact values of the queued candidates, keep those that reach the final threshold
        const double S_exact = block_sum<kScanThreads>((double)lse_acc, red_d);  // also a barrier after the pushes
        const int n_queued = n_cand;
        const float S_fixed = (float)s_fixed * (1.0f / kSumScale);
        const float tau_keep = ref + logf(S_fixed / mu) + 1e-4f;  // every threshold used is below this
        const int n_eval = n_queued < kCandCap ? n_queued : kCandCap;
        for (int i = tid; i < n_eval; i += kScanThreads) {
            const uint32_t idxh = cand[i];
            const int idx = (int)(idxh & 0x00FFFFFFu);
            if (idx >= V) continue;  // padding of the last group
            float raw = RowIO<T>::scalar(row, idx);
            if (raw != raw) { saw_nan = true; continue; }
            if (!(raw > kNegInf)) continue;
            const float pert = raw + gumbel_f32((idxh & 0xFF000000u) | fine_bits(key, node, (uint32_t)idx));
            if (pert >= tau_keep) {
                const int sidx = atomicAdd(&n_surv, 1);
                if (sidx < kSurvCap) { sv_val[sidx] = pert; sv_idx[sidx] = idx; sv_raw[sidx] = raw; }
            }
        }
        __syncthreads();
        const int ns = n_surv;
        ok = (n_queued <= kCandCap) && (ns >= k) && (ns <= kSurvCap) && (S_exact > 0.0) && (S_exact < 1.0e300) &&
             (s_fixed > 0u);
        if (ok) {
            lse = (float)((double)ref + log(S_exact));
            const float shift = (a.subtract_lse && NEED_LSE) ? lse : 0.0f;
            const int64_t o = ((int64_t)b * a.R + r) * a.max_k;
            if (tid < ns) {
                const float mv = sv_val[tid];
                const int mi = sv_idx[tid];
                int rnk = 0;
                for (int e = 0; e < ns; ++e) rnk += better(sv_val[e], sv_idx[e], mv, mi) ? 1 : 0;
                if (rnk < k) {
                    a.out_token[o + rnk] = mi;
                    if (a.node_token) a.node_token[(int64_t)b * a.node_stride + a.child_base[r] + rnk] = mi;
                    if (a.out_perturbed) a.out_perturbed[o + rnk] = mv - shift;
                    if (a.out_value) a.out_value[o + rnk] = sv_raw[tid] - shift;
                }
            }
            if (tid >= k && tid < a.max_k) {
                a.out_token[o + tid] = -1;
                if (a.out_perturbed) a.out_perturbed[o + tid] = kNegInf;
                if (a.out_value) a.out_value[o + tid] = kNegInf;
            }
            if (tid == 0 && a.out_lse) a.out_lse[(int64_t)b * a.R + r] = NEED_LSE ? lse : 0.0f;
            // a NaN makes S_exact NaN, so this path never ends with one: no status bit to set
            return;
        }
    }

    // ---- attempt 2: running bound (only when the check failed) ----------------------------------------------------
    {
        __syncthreads();
        top.init();
        q_head = 0;
        q_count = 0;
        float lse_m = kNegInf, lse_s = 0.0f;
        for (int it = 0; it < n_iter; ++it) {
            const int g = it * kScanThreads + tid;
            const bool valid = g < n_groups;
            float v[16];
            uint4 cw = make_uint4(0, 0, 0, 0);
            float vmax = kNegInf;
            if (valid) {
                load_group<T, ALIGNED>(row, g, V, v);
                cw = rng_draw(key, node, kTagGumbelCoarse, (uint32_t)g);
#pragma unroll
                for (int j = 0; j < 16; ++j) vmax = max_nan(vmax, v[j]);
                if (vmax != vmax) {  // a NaN in this group: treat as -inf
                    saw_nan = true;
                    vmax = kNegInf;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (v[j] != v[j]) v[j] = kNegInf;
                        vmax = fmaxf(vmax, v[j]);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = kNegInf;
            }
            if (NEED_LSE) {
                if (vmax > lse_m) {  // rescale the running sum to the new reference
                    lse_s *= ex2_approx((lse_m - vmax) * kLog2e);  // lse_m = -inf gives 0
                    lse_m = vmax;
                }
                if (lse_m > kNegInf) {
                    const float c = lse_m * kLog2e;
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        s0 += ex2_approx(fmaf(v[j], kLog2e, -c));
                        s1 += ex2_approx(fmaf(v[j + 1], kLog2e, -c));
                    }
                    lse_s += s0 + s1;
                }
            }
            // bytes below 255 bound G by kGumbelBoundBelow255; byte 255 always goes on
            float thr = fmaxf(__shfl_sync(0xFFFFFFFFu, top.v, k - 1), ordered_to_float(*(volatile uint32_t*)&tau_blk)) -
                        kGumbelBoundBelow255;
            const uint32_t inv0 = ~cw.x, inv1 = ~cw.y, inv2 = ~cw.z, inv3 = ~cw.w;  // a 0xFF byte is a zero byte here
            const uint32_t any255 = ((inv0 - 0x01010101u) & ~inv0 & 0x80808080u) | ((inv1 - 0x01010101u) & ~inv1 & 0x80808080u) |
                                    ((inv2 - 0x01010101u) & ~inv2 & 0x80808080u) | ((inv3 - 0x01010101u) & ~inv3 & 0x80808080u);
            const bool cand = valid && vmax > kNegInf && (vmax >= thr || any255 != 0u);
            if (__any_sync(0xFFFFFFFFu, cand)) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const uint32_t word = j < 8 ? (j < 4 ? cw.x : cw.y) : (j < 12 ? cw.z : cw.w);
                    const uint32_t h = (word >> (8 * (j & 3))) & 0xFFu;
                    const bool p = cand && v[j] > kNegInf && (v[j] >= thr || h == 255u);
                    const unsigned bal = __ballot_sync(0xFFFFFFFFu, p);
                    if (bal) {
                        if (p) {
                            const int slot = (q_head + q_count + __popc(bal & ((1u << lane) - 1u))) & (kQueueCap - 1);
                            q_idxh[warp][slot] = (uint32_t)(g * 16 + j) | (h << 24);
                        }
                        q_count += __popc(bal);
                        __syncwarp();
                        if (q_count >= 32) {
                            drain(32, true);
                            thr = fmaxf(__shfl_sync(0xFFFFFFFFu, top.v, k - 1),
                                        ordered_to_float(*(volatile uint32_t*)&tau_blk)) - kGumbelBoundBelow255;
                        }
                    }
                }
            }
        }
        while (q_count > 0) drain(q_count < 32 ? q_count : 32, true);
        total = merge_lists();
        if (NEED_LSE) {
            const float M = block_max<kScanThreads>(lse_m, red_f);
            const float scaled = (lse_m > kNegInf) ? lse_s * ex2_approx((lse_m - M) * kLog2e) : 0.0f;
            const double S = block_sum<kScanThreads>((double)scaled, red_d);
            lse = (M > kNegInf && S > 0.0) ? (float)((double)M + log(S)) : kNegInf;
        }
    }

    if (saw_nan) nan_flag = 1;
    __syncthreads();
    const int64_t o = ((int64_t)b * a.R + r) * a.max_k;
    const float shift = (a.subtract_lse && NEED_LSE) ? lse : 0.0f;
    if (mine && rank < k) {
        a.out_token[o + rank] = top.idx;
        if (a.node_token) a.node_token[(int64_t)b * a.node_stride + a.child_base[r] + rank] = top.idx;
        if (a.out_perturbed) a.out_perturbed[o + rank] = top.v - shift;
        if (a.out_value) a.out_value[o + rank] = top.raw - shift;
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
            const uint32_t bits = (coarse_byte(cw, (uint32_t)x & 15u) << 24) | fine_bits(key, node, (uint32_t)x);
            phi = sigma + ((double)a.fin_value[(int64_t)b * F + f] - lse);
            pert = phi + gumbel_f64(bits);
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
