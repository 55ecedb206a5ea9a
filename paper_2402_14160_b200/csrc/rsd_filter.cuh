// Logit warping of vocabulary rows: top-k and nucleus (top-p) filtering after the temperature (Section 4's sampling
// settings: temperature 0.3 / 1.0, nucleus 0.95).  A filtered token counts as log-probability -inf from then on, which
// is how the drafting and verification kernels already treat masked entries (Algorithms 4 and 9 drop them).
//
//   top-k   keep the k largest values (equal values: the smaller token first)
//   top-p   of what is left, in order of decreasing probability (equal values: the smaller token first), the
//           shortest prefix whose share of the mass reaches top_p (at least one token)
//
// One block per row.  The row is copied to shared memory once; both cuts are then found without sorting: the value
// of the last kept token by a 16-ary search over the ordered bit patterns of the values.  Each pass sorts the tokens
// of the current interval into 16 sub-intervals (equal steps in value while the interval is wide, which is where the
// tokens spread evenly; equal steps in bit pattern once it is narrow) and counts them and sums their weights
// exp(value / T) in bins private to each thread.  The first pass also gives the row's total mass.  As soon as the
// interval holds few enough tokens their indices are gathered, in token order, and every later pass runs over that
// short list instead of the row.  The last kept token among equal values comes from a prefix count in token order.
// Sums are taken in a fixed order (per thread, over the threads of a bin, over the bins), so the result does not
// depend on timing.
#pragma once
#include "rsd_device.cuh"
#include "rsd_scan.cuh"   // ex2_approx, better()

namespace rsd {

constexpr int kFilterThreads = 256;
constexpr int kFilterWarps = kFilterThreads / 32;
constexpr int kBins = 16;                        // sub-intervals per search pass
constexpr int kListCap = 8192;                   // tokens gathered into a list (indices as 16 bits: rows up to 65,536)
constexpr float kValueRange = 24.0f;             // value-linear bins cover this many nats of value / T below the interval's top

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
    float mass[kBins][kFilterThreads];           // per-thread bins of a search pass
    uint16_t count[kBins][kFilterThreads];
    uint32_t bound[kBins + 1];                   // bin q holds the codes bound[q] .. bound[q + 1] - 1 (the last: .. hi)
    double mass_total[kBins];
    int count_total[kBins];
    uint16_t list[kListCap];                     // indices of the tokens still in play, in token order
    int red_i[kFilterWarps][2];
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
    __device__ static __forceinline__ uint32_t code_of_float(float v) { return code_of_bits(__float_as_uint(v) >> 16); }   // (truncated)
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
    __device__ static __forceinline__ uint32_t code_of_float(float v) { return code_of_bits(__float_as_uint(v)); }
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
    int n_list;                 // >= 0: the tokens still in play are sm.list[0 .. n_list); -1: the whole row

    __device__ __forceinline__ float weight(uint32_t code) const { return ex2_approx(fmaf(RowCodes<T>::value_of_code(code), k, neg_c)); }
    __device__ __forceinline__ int items() const { return n_list >= 0 ? n_list : V; }
    __device__ __forceinline__ int index(int m) const { return n_list >= 0 ? (int)sm.list[m] : m; }

    // What the search found: the code t of the last kept value, the mass and the number of the tokens strictly above it,
    // and the total mass of the tokens the search started from.
    struct Found {
        uint32_t t;
        double above_mass;
        int above_count;
        double total_mass;
    };

    // The largest code t in [lo, hi] with F(t) >= need, F(t) = the number (BY_MASS = false) or the weight (BY_MASS = true)
    // of the tokens within `inside` whose code is >= t.  need = need_abs, or, when need_abs < 0, need_frac times the
    // total weight of the tokens within `inside` (they all lie in [lo, hi]: the first pass measures it).  F is
    // non-increasing, F(lo) >= need, nothing within `inside` lies above hi.
    template <bool BY_MASS>
    __device__ __forceinline__ Found search(uint32_t lo, uint32_t hi, double need_abs, double need_frac, const Cut& inside) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        Found r = {lo, 0.0, 0, 0.0};
        double need = need_abs;
        int level = 0;
        for (;; ++level) {
            // ---- the 16 sub-intervals ------------------------------------------------------------------------------------------
            const uint32_t span = hi - lo;
            const bool by_value = level < 2 && span > 4096u;
            if (tid <= kBins) {
                uint32_t bd;
                if (tid == 0) bd = lo;
                else if (tid == kBins) bd = hi;          // (unused as a lower bound; bin 15 ends at hi)
                else if (by_value) {
                    const float v_hi = RowCodes<T>::value_of_code(hi);
                    const float v_lo = fmaxf(RowCodes<T>::value_of_code(lo), v_hi - kValueRange * kLog2e / k);
                    const uint32_t c = RowCodes<T>::code_of_float(v_lo + (v_hi - v_lo) * (float)tid * (1.0f / kBins));
                    bd = c <= lo ? lo + 1u : (c > hi ? hi : c);
                } else {
                    const int shift = max(0, 32 - __clz(span | 1u) - 4);      // (span >> shift) < 16
                    const uint32_t c = lo + ((uint32_t)tid << shift);
                    bd = (c < lo || c > hi) ? hi : c;                        // bins past the interval's end are empty ...
                    if (c > hi || c < lo) bd = hi;                           // ... they all start at hi, and only the last holds it
                }
                sm.bound[tid] = bd;
            }
#pragma unroll
            for (int q = 0; q < kBins; ++q) { sm.mass[q][tid] = 0.0f; sm.count[q][tid] = 0; }
            __syncthreads();
            // bins that start at the same code: only the last of them is used (the search below takes the largest q)
            const int n_items = items();
            for (int m = tid; m < n_items; m += kFilterThreads) {
                const int i = index(m);
                const uint32_t code = RowCodes<T>::code(row, i);
                if (code < lo || code > hi || !within(inside, code, i) || code <= RowCodes<T>::kNegInfCode) continue;
                int q = code >= sm.bound[8] ? 8 : 0;
                q += code >= sm.bound[q + 4] ? 4 : 0;
                q += code >= sm.bound[q + 2] ? 2 : 0;
                q += code >= sm.bound[q + 1] ? 1 : 0;
                if (q == kBins) q = kBins - 1;                               // code == hi == bound[16]
                sm.mass[q][tid] += weight(code);
                sm.count[q][tid] += 1;
            }
            __syncthreads();
            // ---- totals of the bins: warp w adds up bins 2 w and 2 w + 1, every lane eight threads' entries in order,
            // then a fixed tree over the lanes ----------------------------------------------------------------------------------
#pragma unroll
            for (int h = 0; h < kBins / kFilterWarps; ++h) {
                const int q = warp * (kBins / kFilterWarps) + h;
                double v = 0.0;
                int c = 0;
#pragma unroll
                for (int e = 0; e < kFilterThreads / 32; ++e) {
                    v += (double)sm.mass[q][lane * (kFilterThreads / 32) + e];
                    c += (int)sm.count[q][lane * (kFilterThreads / 32) + e];
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                c = __reduce_add_sync(0xFFFFFFFFu, c);
                if (lane == 0) { sm.mass_total[q] = v; sm.count_total[q] = c; }
            }
            __syncthreads();
            if (level == 0) {
                double tot = 0.0;
                for (int q = 0; q < kBins; ++q) tot += sm.mass_total[q];
                r.total_mass = tot;
                if (need_abs < 0.0) need = need_frac * tot;
            }
            // ---- from the top bin down: the first bin that brings the tally to `need` holds t ------------------------------
            double run_m = r.above_mass;
            int run_c = r.above_count;
            int pick = 0;
            for (int q = kBins - 1; q >= 0; --q) {
                const double f = BY_MASS ? run_m + sm.mass_total[q] : (double)(run_c + sm.count_total[q]);
                if (f >= need) { pick = q; break; }
                run_m += sm.mass_total[q];
                run_c += sm.count_total[q];
            }
            r.above_mass = run_m;
            r.above_count = run_c;
            const uint32_t new_lo = sm.bound[pick];
            uint32_t new_hi = hi;
            if (pick < kBins - 1) {
                const uint32_t nb = sm.bound[pick + 1];
                new_hi = nb > new_lo ? nb - 1u : new_lo;          // (an empty bin cannot be picked unless need <= what lies above)
                if (nb <= new_lo) new_hi = new_lo;
            }
            const int population = sm.count_total[pick];
            __syncthreads();
            lo = new_lo;
            hi = new_hi;
            if (lo >= hi) break;
            // few enough tokens left: gather them, in token order, and go on over the list
            if (n_list < 0 && population <= kListCap && V <= 65536) gather(lo, hi, inside);
        }
        r.t = lo;
        return r;
    }

    // The indices of the tokens within `inside` with a code in [lo, hi], in token order, into sm.list.
    __device__ __forceinline__ void gather(uint32_t lo, uint32_t hi, const Cut& inside) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        const int per = (V + kFilterThreads - 1) / kFilterThreads;
        const int i0 = tid * per, i1 = min(V, i0 + per);
        int mine = 0;
        for (int i = i0; i < i1; ++i) {
            const uint32_t code = RowCodes<T>::code(row, i);
            mine += (code >= lo && code <= hi && within(inside, code, i) && code > RowCodes<T>::kNegInfCode) ? 1 : 0;
        }
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sm.scan_i[warp] = incl;
        __syncthreads();
        int at = incl - mine, total = 0;
        for (int w = 0; w < kFilterWarps; ++w) {
            if (w < warp) at += sm.scan_i[w];
            total += sm.scan_i[w];
        }
        if (total <= kListCap) {
            for (int i = i0; i < i1; ++i) {
                const uint32_t code = RowCodes<T>::code(row, i);
                if (code >= lo && code <= hi && within(inside, code, i) && code > RowCodes<T>::kNegInfCode) sm.list[at++] = (uint16_t)i;
            }
        }
        __syncthreads();
        if (total <= kListCap) n_list = total;
    }

    // Number of the tokens in play that have code `code` and lie within `inside`, and the index of the j-th (1-based) of
    // them in token order (-1 if there are fewer).  Threads own consecutive runs; one prefix count over the block.
    __device__ __forceinline__ int nth_with_code(uint32_t code, int j, const Cut& inside, int& how_many) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        const int n_items = items();
        const int per = (n_items + kFilterThreads - 1) / kFilterThreads;
        const int m0 = tid * per, m1 = min(n_items, m0 + per);
        int mine = 0;
        for (int m = m0; m < m1; ++m) {
            const int i = index(m);
            mine += (RowCodes<T>::code(row, i) == code && within(inside, code, i)) ? 1 : 0;
        }
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sm.scan_i[warp] = incl;
        if (tid == 0) sm.found = -1;
        __syncthreads();
        int before = incl - mine, total = 0;
        for (int w = 0; w < kFilterWarps; ++w) {
            if (w < warp) before += sm.scan_i[w];
            total += sm.scan_i[w];
        }
        how_many = total;
        if (mine > 0 && before < j && j <= before + mine) {
            int seen = before;
            for (int m = m0; m < m1; ++m) {
                const int i = index(m);
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
    RowFilter<T> f = {sm, row_sm, V, a.log2e_over_t, (finite > 0 && !plus_inf) ? -vmax * a.log2e_over_t : 0.0f, -1};
    Cut cut = {RowCodes<T>::kNegInfCode, V};                      // everything finite
    int kept = finite;

    // ---- top-k: the value of the k-th largest entry, then the last kept token among its equals -------------------------
    if (a.top_k > 0 && a.top_k < V && finite > a.top_k) {
        const typename RowFilter<T>::Found r = f.template search<false>(RowCodes<T>::kNegInfCode + 1u, top, (double)a.top_k, 0.0, cut);
        int ties;
        const int tok = f.nth_with_code(r.t, a.top_k - r.above_count, cut, ties);   // that many of the entries equal to t stay
        cut.code = r.t;
        cut.tok = tok >= 0 ? tok : V;
        kept = a.top_k;
        f.n_list = -1;                                            // (the list was gathered for the old cut)
    }
    // ---- top-p: of what is left, the shortest prefix (value descending, token ascending) whose mass reaches top_p -------
    if (a.top_p > 0.0f && a.top_p < 1.0f && kept > 0 && !plus_inf) {
        const typename RowFilter<T>::Found r = f.template search<true>(cut.code, top, -1.0, (double)a.top_p, cut);
        const double need = (double)a.top_p * r.total_mass;
        // entries equal to t within the cut: each weighs w; the first j of them (token order) complete the prefix
        int ties;
        f.nth_with_code(r.t, 1, cut, ties);
        const double w = (double)f.weight(r.t);
        int j = ties;
        if (w > 0.0) {
            const double want = ceil((need - r.above_mass) / w);
            j = want < 1.0 ? 1 : (want > (double)ties ? ties : (int)want);
            while (j > 1 && r.above_mass + (double)(j - 1) * w >= need) --j;
            while (j < ties && r.above_mass + (double)j * w < need) ++j;
        }
        const int tok = f.nth_with_code(r.t, j, cut, ties);
        cut.code = r.t;
        cut.tok = tok >= 0 ? tok : V;
        kept = r.above_count + j;
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
