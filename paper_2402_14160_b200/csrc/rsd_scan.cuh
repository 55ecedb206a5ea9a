// Row scan: exact sorted arg-top-k of (row + Gumbel noise) in one pass over the row (Eqs. 6-7, Algorithm 4), and
// the per-sequence epilogue of a Stochastic Beam Search level (Eqs. 10-12, Algorithm 9).
//
// The noise of an element is 32 random bits: a coarse byte (16 elements per Philox call) on top of 24 fine bits
// (4 elements per call).  G is increasing in those bits, so the byte alone bounds G from above.  Every element is
// tested against "value + bound >= tau", where tau is a running lower bound of the k-th largest perturbed value;
// only the few that pass get their fine bits and an exact G.  Nothing that could be among the k largest is ever
// skipped, so the result equals the plain definition (perturb everything, sort) in fp32.
#pragma once
#include "rsd_device.cuh"

namespace rsd {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kQueueCap = 64;  // per-warp candidate queue (a push adds at most 32 to at most 31 pending)
constexpr int kMaxRows = 256;
constexpr int kIdxNone = 0x7FFFFFFF;

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
    uint8_t k_row[kMaxRows];
    int32_t node_row[kMaxRows];
    int32_t child_base[kMaxRows];
};

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

template <typename T, bool ALIGNED, bool NEED_LSE>
__global__ void __launch_bounds__(kScanThreads) scan_topk_kernel(const ScanArgs a) {
    __shared__ uint32_t q_idxh[kScanWarps][kQueueCap];
    __shared__ float q_val[kScanWarps][kQueueCap];
    __shared__ uint32_t tau_blk;  // order-preserving encoding of the block's best lower bound
    __shared__ float m_v[kScanWarps * 32], m_raw[kScanWarps * 32];
    __shared__ int m_idx[kScanWarps * 32];
    __shared__ float red_f[kScanWarps];
    __shared__ double red_d[kScanWarps];
    __shared__ int nan_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / a.R, r = blockIdx.x % a.R;
    const int k = a.k_row[r];
    const uint32_t node = (uint32_t)a.node_row[r];
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    const char* row = (const char*)a.data + ((int64_t)b * a.seq_stride + (int64_t)r * a.row_stride) * RowIO<T>::kBytes;
    const int V = a.V, n_groups = (V + 15) >> 4;

    if (tid == 0) { tau_blk = float_to_ordered(kNegInf); nan_flag = 0; }
    __syncthreads();

    WarpTop top;
    top.init();
    int q_head = 0, q_count = 0;   // warp-uniform
    float lse_m = kNegInf, lse_s = 0.0f;
    bool saw_nan = false;

    // Take up to 32 queued candidates: bound test with the exact byte, then exact noise, then insertion.
    auto drain = [&](int n) {
        const bool have = lane < n;
        uint32_t idxh = 0;
        float raw = kNegInf;
        if (have) {
            const int slot = (q_head + lane) & (kQueueCap - 1);
            idxh = q_idxh[warp][slot];
            raw = q_val[warp][slot];
        }
        const int idx = (int)(idxh & 0x00FFFFFFu);
        const uint32_t h = idxh >> 24;
        const float tau = fmaxf(__shfl_sync(0xFFFFFFFFu, top.v, k - 1), ordered_to_float(*(volatile uint32_t*)&tau_blk));
        float pert = kNegInf;
        const bool pass = have && (raw + gumbel_upper_bound(h) >= tau);
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
        const float tw = __shfl_sync(0xFFFFFFFFu, top.v, k - 1);
        if (lane == 0 && tw > kNegInf) atomicMax(&tau_blk, float_to_ordered(tw));
        __syncwarp();
    };

    const int n_iter = (n_groups + kScanThreads - 1) / kScanThreads;
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

        // Stage 1: bytes below 255 bound G by kGumbelBoundBelow255; byte 255 always goes on.
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
                        q_val[warp][slot] = v[j];
                    }
                    q_count += __popc(bal);
                    __syncwarp();
                    if (q_count >= 32) {
                        drain(32);
                        thr = fmaxf(__shfl_sync(0xFFFFFFFFu, top.v, k - 1),
                                    ordered_to_float(*(volatile uint32_t*)&tau_blk)) - kGumbelBoundBelow255;
                    }
                }
            }
        }
    }
    while (q_count > 0) drain(q_count < 32 ? q_count : 32);

    // merge the warps' lists: rank every entry among all entries
    m_v[tid] = top.v;
    m_idx[tid] = top.idx;
    m_raw[tid] = top.raw;
    if (saw_nan) nan_flag = 1;

    float lse = 0.0f;
    if (NEED_LSE) {
        const float M = block_max<kScanThreads>(lse_m, red_f);
        const float scaled = (lse_m > kNegInf) ? lse_s * ex2_approx((lse_m - M) * kLog2e) : 0.0f;
        const double S = block_sum<kScanThreads>((double)scaled, red_d);
        lse = (M > kNegInf && S > 0.0) ? (float)((double)M + log(S)) : kNegInf;
    }
    __syncthreads();

    const bool mine = lane < k && top.idx != kIdxNone;
    int rank = 0;
    if (mine) {
        for (int w = 0; w < kScanWarps; ++w)
            for (int i = 0; i < k; ++i) {
                const int e = w * 32 + i;
                rank += (m_idx[e] != kIdxNone && better(m_v[e], m_idx[e], top.v, top.idx)) ? 1 : 0;
            }
    }
    // number of distinct picks available to this row
    int total = 0;
    {
        // every finite element seen by some warp is in that warp's list if it ranks in its top k, so the union's
        // size, capped at k, is the number of finite picks
        const int cnt = __syncthreads_count(mine);
        total = cnt < k ? cnt : k;
    }
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
