// Logit warping of vocabulary rows: top-k and nucleus (top-p) filtering after the temperature (Section 4's sampling
// settings: temperature 0.3 / 1.0, nucleus 0.95).  A filtered token counts as log-probability -inf from then on, which
// is how the drafting and verification kernels already treat masked entries (Algorithms 4 and 9 drop them).
//
//   top-k   keep the k largest values (equal values: the smaller token first)
//   top-p   of what is left, in order of decreasing probability (equal values: the smaller token first), the
//           shortest prefix whose share of the mass reaches top_p (at least one token)
//
// One block per row.  The row is copied to shared memory once; both cuts are then found without sorting: the value
// of the last kept token by a 16-ary search over the ordered bit patterns of the values (each pass sorts the tokens
// of the current interval into 16 equal sub-intervals and counts them, or sums their weights exp(value / T), in bins
// private to each thread; four passes settle a 16-bit pattern, eight a 32-bit one), and the last kept token among
// equal values by a prefix count in token order.  Sums are taken in a fixed order (per thread, over the threads of a
// bin, over the bins), so the result does not depend on timing.
#pragma once
#include "rsd_device.cuh"
#include "rsd_scan.cuh"   // ex2_approx, better()

namespace rsd {

constexpr int kFilterThreads = 256;
constexpr int kFilterWarps = kFilterThreads / 32;
constexpr int kTrials = 2;                       // trial values a tally can take at once
constexpr int kBins = 16;                        // sub-intervals per search pass

struct FilterArgs {
    const void* data;
    void* out;                                   // [B][R][V], the rows' element type
    int64_t seq_stride, row_stride;              // elements
    int R, V;
    int top_k;                                   // 0: none
    float top_p;                                 // >= 1: none
    float log2e_over_t;                          // log2(e) / temperature
    int32_t* kept;                               // [B][R] or null
    int32_t* status;                             // [B], OR-ed into
};

struct FilterSmem {
    float bins[kBins][kFilterThreads];           // per-thread bins of a search pass (counts are stored as floats' bits)
    double bin_total[kBins];
    double red_d[kFilterWarps][kTrials];
    int red_i[kFilterWarps][kTrials];
    float red_f[kFilterWarps];
    int scan_i[kFilterWarps];
    int found;
    int nan_flag;
};

// ordered code of element i of the row in shared memory: larger value <=> larger code; NaN counts as -inf.
// 2-byte rows: the 16-bit pattern (all that distinguishes two bf16 values); 4-byte rows: all 32 bits.
template <typename T>
struct RowCodes;
template <>
struct RowCodes<__nv_bfloat16> {
    static constexpr int kBits = 16;
    __device__ static __forceinline__ uint32_t code_of_bits(uint32_t h) {       // h: the 16-bit pattern
        if ((h & 0x7FFFu) > 0x7F80u) h = 0xFF80u;                                  // NaN -> -inf
        return (h & 0x8000u) ? (~h & 0xFFFFu) : (h | 0x8000u);
    }
    __device__ static __forceinline__ uint32_t code(const unsigned char* row, int i) { return code_of_bits(((const uint16_t*)row)[i]); }
    __device__ static __forceinline__ float value_of_code(uint32_t c) {
        const uint32_t h = (c & 0x8000u) ? (c & 0x7FFFu) : (~c & 0xFFFFu);
        return __uint_as_float(h << 16);
    }
    __device__ static __forceinline__ bool is_nan(const unsigned char* row, int i) { return (((const uint16_t*)row)[i] & 0x7FFFu) > 0x7F80u; }
    static constexpr uint32_t kNegInfCode = 0x007Fu;                               // code of -inf (0xFF80)
    static constexpr uint32_t kNegInfBits = 0xFF80u;
};
template <>
struct RowCodes<float> {
    static constexpr int kBits = 32;
    __device__ static __forceinline__ uint32_t code_of_bits(uint32_t u) {
        if ((u & 0x7FFFFFFFu) > 0x7F800000u) u = 0xFF800000u;
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static __forceinline__ uint32_t code(const unsigned char* row, int i) { return code_of_bits(((const uint32_t*)row)[i]); }
    __device__ static __forceinline__ float value_of_code(uint32_t c) {
        return __uint_as_float((c & 0x80000000u) ? (c & 0x7FFFFFFFu) : ~c);
    }
    __device__ static __forceinline__ bool is_nan(const unsigned char* row, int i) { return (((const uint32_t*)row)[i] & 0x7FFFFFFFu) > 0x7F800000u; }
    static constexpr uint32_t kNegInfCode = 0x007FFFFFu;
    static constexpr uint32_t kNegInfBits = 0xFF800000u;
};

// A cut in the order (value descending, token ascending): a token is at or before the cut iff its code is larger,
// or equal with a token index not beyond `tok`.
struct Cut {
    uint32_t code;
    int tok;
};
__device__ __forceinline__ bool within(const Cut& c, uint32_t code, int i) { return code > c.code || (code == c.code && i <= c.tok); }

template <typename T>
struct RowFilter {
    FilterSmem& sm;
    const unsigned char* row;   // shared memory
    int V;
    float k, neg_c;             // weight of a value: 2^(value * k + neg_c)

    __device__ __forceinline__ float weight(uint32_t code) const { return ex2_approx(fmaf(RowCodes<T>::value_of_code(code), k, neg_c)); }

    // For each of the trial codes t[0] < ... < t[n-1]: over the tokens within `inside` whose code is >= t[j], their number
    // (WEIGH = false) or the sum of their weights (WEIGH = true).  Identical on all threads.
    template <bool WEIGH>
    __device__ __forceinline__ void tally(const uint32_t (&t)[kTrials], int n, const Cut& inside, double (&out)[kTrials]) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        float acc[kTrials];
        int cnt[kTrials];
#pragma unroll
        for (int j = 0; j < kTrials; ++j) { acc[j] = 0.0f; cnt[j] = 0; }
        for (int i = tid; i < V; i += kFilterThreads) {
            const uint32_t code = RowCodes<T>::code(row, i);
            if (!within(inside, code, i) || code <= RowCodes<T>::kNegInfCode) continue;
            const float w = WEIGH ? weight(code) : 0.0f;
#pragma unroll
            for (int j = 0; j < kTrials; ++j) {
                if (j < n && code >= t[j]) {
                    if (WEIGH) acc[j] += w;
                    else ++cnt[j];
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kTrials; ++j) {
            if (WEIGH) {
                float v = acc[j];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                if (lane == 0) sm.red_d[warp][j] = (double)v;
            } else {
                const int v = __reduce_add_sync(0xFFFFFFFFu, cnt[j]);
                if (lane == 0) sm.red_i[warp][j] = v;
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < kTrials; ++j) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < kFilterWarps; ++w) s += WEIGH ? sm.red_d[w][j] : (double)sm.red_i[w][j];   // fixed order
            out[j] = s;
        }
        __syncthreads();
    }

    // The largest code t in [lo, hi] with F(t) >= need, where F(t) is the number (WEIGH = false) or the weight
    // (WEIGH = true) of the tokens within `inside` whose code is >= t.  F is non-increasing; the caller guarantees
    // F(lo) >= need and that nothing within `inside` lies above hi.  Also returns F(t + 1), the tally strictly above t.
    template <bool WEIGH>
    __device__ __forceinline__ uint32_t search(uint32_t lo, uint32_t hi, double need, const Cut& inside, double& above) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        above = 0.0;
        while (lo < hi) {
            const uint32_t span = hi - lo;                                   // >= 1
            const int shift = max(0, 32 - __clz(span) - 4);                  // (span >> shift) < 16
#pragma unroll
            for (int q = 0; q < kBins; ++q) sm.bins[q][tid] = 0.0f;
            for (int i = tid; i < V; i += kFilterThreads) {
                const uint32_t code = RowCodes<T>::code(row, i);
                if (code < lo || code > hi || !within(inside, code, i) || code <= RowCodes<T>::kNegInfCode) continue;
                const int q = (int)((code - lo) >> shift);
                if (WEIGH) sm.bins[q][tid] += weight(code);
                else sm.bins[q][tid] = __int_as_float(__float_as_int(sm.bins[q][tid]) + 1);
            }
            __syncthreads();
            // totals of the bins: warp w adds up bins 2 w and 2 w + 1, every lane eight threads' entries in order, then a
            // fixed tree over the lanes
#pragma unroll
            for (int h = 0; h < kBins / kFilterWarps; ++h) {
                const int q = warp * (kBins / kFilterWarps) + h;
                double v = 0.0;
#pragma unroll
                for (int e = 0; e < kFilterThreads / 32; ++e) {
                    const float x = sm.bins[q][lane * (kFilterThreads / 32) + e];
                    v += WEIGH ? (double)x : (double)__float_as_int(x);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                if (lane == 0) sm.bin_total[q] = v;
            }
            __syncthreads();
            // from the top bin down: the first bin that brings the tally to `need` holds t
            double run = above;
            int pick = 0;
            for (int q = kBins - 1; q >= 0; --q) {
                const double with_q = run + sm.bin_total[q];
                if (with_q >= need) { pick = q; break; }
                run = with_q;
            }
            above = run;
            const uint32_t new_lo = lo + ((uint32_t)pick << shift);
            const uint32_t width = shift >= 32 ? 0xFFFFFFFFu : ((1u << shift) - 1u);
            hi = (new_lo + width < new_lo || new_lo + width > hi) ? hi : new_lo + width;
            lo = new_lo;
            __syncthreads();
        }
        return lo;
    }

    // Index of the j-th (1-based) token, in token order, that has code `code` and lies within `inside`; -1 if there are
    // fewer.  Threads own consecutive runs of tokens; one prefix count over the block.
    __device__ __forceinline__ int nth_with_code(uint32_t code, int j, const Cut& inside) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        const int per = (V + kFilterThreads - 1) / kFilterThreads;
        const int i0 = tid * per, i1 = min(V, i0 + per);
        int mine = 0;
        for (int i = i0; i < i1; ++i) mine += (RowCodes<T>::code(row, i) == code && within(inside, code, i)) ? 1 : 0;
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sm.scan_i[warp] = incl;
        if (tid == 0) sm.found = -1;
        __syncthreads();
        int before = incl - mine;
        for (int w = 0; w < warp; ++w) before += sm.scan_i[w];
        if (mine > 0 && before < j && j <= before + mine) {
            int seen = before;
            for (int i = i0; i < i1; ++i) {
                if (RowCodes<T>::code(row, i) == code && within(inside, code, i) && ++seen == j) { sm.found = i; break; }
            }
        }
        __syncthreads();
        const int r = sm.found;
        __syncthreads();
        return r;
    }
};

template <typename T>
__global__ void __launch_bounds__(kFilterThreads) filter_rows_kernel(const FilterArgs a) {
    extern __shared__ __align__(16) unsigned char row_sm[];
    __shared__ FilterSmem sm;
    constexpr int kElem = (int)sizeof(T);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / a.R, r = blockIdx.x % a.R, V = a.V;
    const unsigned char* src = (const unsigned char*)a.data + ((int64_t)b * a.seq_stride + (int64_t)r * a.row_stride) * kElem;
    unsigned char* dst = (unsigned char*)a.out + ((int64_t)b * a.R + r) * (int64_t)V * kElem;

    // ---- the row into shared memory (16 bytes at a time where the source allows it) ---------------------------------------
    if (tid == 0) sm.nan_flag = 0;
    {
        const int n16 = ((uintptr_t)src & 15u) == 0 ? (V * kElem) / 16 : 0;
        for (int i = tid; i < n16; i += kFilterThreads) ((uint4*)row_sm)[i] = ld_stream((const uint4*)src + i);
        for (int i = n16 * (16 / kElem) + tid; i < V; i += kFilterThreads) {
            if (kElem == 2) ((uint16_t*)row_sm)[i] = ((const uint16_t*)src)[i];
            else ((uint32_t*)row_sm)[i] = ((const uint32_t*)src)[i];
        }
    }
    __syncthreads();

    // ---- the largest value and the number of finite entries ------------------------------------------------------------------
    uint32_t top = RowCodes<T>::kNegInfCode;
    int finite = 0;
    bool saw_nan = false;
    for (int i = tid; i < V; i += kFilterThreads) {
        saw_nan |= RowCodes<T>::is_nan(row_sm, i);
        const uint32_t c = RowCodes<T>::code(row_sm, i);
        top = c > top ? c : top;
        finite += c > RowCodes<T>::kNegInfCode ? 1 : 0;
    }
    top = __reduce_max_sync(0xFFFFFFFFu, top);
    finite = __reduce_add_sync(0xFFFFFFFFu, finite);
    if (lane == 0) { sm.red_i[warp][0] = (int)top; sm.red_i[warp][1] = finite; }
    if (saw_nan) sm.nan_flag = 1;
    __syncthreads();
    top = 0u;
    finite = 0;
    for (int w = 0; w < kFilterWarps; ++w) {
        top = (uint32_t)sm.red_i[w][0] > top ? (uint32_t)sm.red_i[w][0] : top;
        finite += sm.red_i[w][1];
    }
    __syncthreads();

    const float vmax = RowCodes<T>::value_of_code(top);
    const bool plus_inf = vmax == -kNegInf;                       // a +inf entry: it alone carries the mass
    RowFilter<T> f = {sm, row_sm, V, a.log2e_over_t, (finite > 0 && !plus_inf) ? -vmax * a.log2e_over_t : 0.0f};
    Cut cut = {RowCodes<T>::kNegInfCode, V};                      // everything finite
    int kept = finite;

    // ---- top-k: the value of the k-th largest entry, then the last kept token among its equals -------------------------
    if (a.top_k > 0 && a.top_k < V && finite > a.top_k) {
        double above;
        const uint32_t t = f.template search<false>(RowCodes<T>::kNegInfCode + 1u, top, (double)a.top_k, cut, above);
        const int j = a.top_k - (int)above;                      // that many of the entries equal to t are kept
        const int tok = f.nth_with_code(t, j, cut);
        cut.code = t;
        cut.tok = tok >= 0 ? tok : V;
        kept = a.top_k;
    }
    // ---- top-p: of what is left, the shortest prefix (value descending, token ascending) whose mass reaches top_p -------
    if (a.top_p > 0.0f && a.top_p < 1.0f && kept > 0 && !plus_inf) {
        uint32_t t1[kTrials];
        double tot[kTrials];
        t1[0] = cut.code;                                         // (every entry within the cut has a code >= cut.code)
        f.template tally<true>(t1, 1, cut, tot);
        const double need = (double)a.top_p * tot[0];
        double above;
        const uint32_t t = f.template search<true>(cut.code, top, need, cut, above);
        // entries equal to t within the cut: each weighs w; the first j of them (token order) complete the prefix
        double ties_d[kTrials];
        uint32_t tt[kTrials];
        tt[0] = t;
        tt[1] = t + 1u;
        f.template tally<false>(tt, t == 0xFFFFFFFFu ? 1 : 2, cut, ties_d);
        const int ties = (int)(ties_d[0] - (t == 0xFFFFFFFFu ? 0.0 : ties_d[1]));
        const double w = (double)f.weight(t);
        int j = ties;
        if (w > 0.0) {
            const double want = ceil((need - above) / w);
            j = want < 1.0 ? 1 : (want > (double)ties ? ties : (int)want);
            while (j > 1 && above + (double)(j - 1) * w >= need) --j;
            while (j < ties && above + (double)j * w < need) ++j;
        }
        const int tok = f.nth_with_code(t, j, cut);
        const int n_above = t == 0xFFFFFFFFu ? 0 : (int)ties_d[1];
        cut.code = t;
        cut.tok = tok >= 0 ? tok : V;
        kept = n_above + j;
    }

    // ---- the row with -inf at the filtered entries ------------------------------------------------------------------------------
    for (int i = tid; i < V; i += kFilterThreads) {
        const uint32_t c = RowCodes<T>::code(row_sm, i);
        const bool keep = c > RowCodes<T>::kNegInfCode && within(cut, c, i);
        if (kElem == 2) ((uint16_t*)dst)[i] = keep ? ((const uint16_t*)row_sm)[i] : (uint16_t)RowCodes<T>::kNegInfBits;
        else ((uint32_t*)dst)[i] = keep ? ((const uint32_t*)row_sm)[i] : RowCodes<T>::kNegInfBits;
    }
    if (tid == 0) {
        if (a.kept) a.kept[(int64_t)b * a.R + r] = kept;
        if (sm.nan_flag) atomicOr(&a.status[b], 1);               // RSD_ST_NAN_INPUT
    }
}

}  // namespace rsd
