// Logit warping of vocabulary rows: top-k and nucleus (top-p) filtering after the temperature (Section 4's sampling
// settings: temperature 0.3 / 1.0, nucleus 0.95).  A filtered token counts as log-probability -inf from then on, which
// is how the drafting and verification kernels already treat masked entries (Algorithms 4 and 9 drop them).
//
//   top-k   keep the k largest values (equal values: the smaller token first)
//   top-p   of what is left, in order of decreasing probability (equal values: the smaller token first), the
//           shortest prefix whose share of the mass reaches top_p (at least one token)
//
// One block per row.  The row is copied to shared memory once (NaN turned into -inf on the way); both cuts are then
// found without sorting, by a search for the value of the last kept token over the ordered bit patterns of the
// values.  The first step of a search sweeps the row once, 16 bytes at a time, into a histogram of 2048 bins of equal
// width in value (where the tokens spread evenly): one 64-bit shared-memory addition per token carries both its
// count and its weight exp(value / T) as a fixed-point number, so the sums are integers and do not depend on the
// order of the additions.  The bin that brings the tally to what is needed holds a few hundred tokens at most; they
// are gathered, in token order, and the rest of the search runs over that short list, 16 sub-intervals at a time with
// bins private to each thread (summed in a fixed order).  The last kept token among equal values comes from a prefix
// count in token order.
#pragma once
#include "rsd_device.cuh"
#include "rsd_scan.cuh"   // ex2_approx, better()

namespace rsd {

constexpr int kFilterThreads = 512;
constexpr int kFilterWarps = kFilterThreads / 32;
constexpr int kFineThreads = 256;                // threads that keep private bins in a search pass over the list
constexpr int kBins = 16;                        // sub-intervals per search pass over the list
constexpr int kCoarseBins = 2048;                // bins of the sweep over the row
constexpr int kCountShift = 47;                  // a histogram entry: count << 47 | weight as fixed point, kept as two 32-bit halves
constexpr int kListCap = 2048;                   // tokens gathered into a list (indices as 16 bits: rows up to 65,536); sized so
                                                 // that a 4-byte row of 50,272 entries still fits beside this kernel's other data
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
    union {
        struct {
            float mass[kBins][kFineThreads];     // per-thread bins of a search pass over the list
            uint16_t count[kBins][kFineThreads];
        } fine;
        struct {
            uint32_t lo[kCoarseBins];            // the sweep's histogram: low halves (weights),
            uint32_t hi[kCoarseBins];            // high halves (count << 15 | the weights' carries)
        } hist;
    };
    uint32_t bound[kBins + 1];                   // bin q holds the codes bound[q] .. bound[q + 1] - 1 (the last: .. hi)
    double mass_total[kBins];
    int count_total[kBins];
    uint16_t list[kListCap];                     // indices of the tokens still in play, in token order
    unsigned long long scan_w[kFilterWarps];
    int red_i[kFilterWarps][2];
    int scan_i[kFilterWarps];
    unsigned long long pick_above;               // histogram entries above the picked bin
    unsigned long long row_bar;                  // mbarrier of the row's bulk copy
    int copy_gave_up;
    int needs_cleaning;
    int pick_bin;
    int found;
    int nan_flag;
};

// ordered code of a value's bit pattern: larger value <=> larger code, equal values <=> equal codes; NaN counts as -inf.
// 2-byte rows: the 16-bit pattern (all that distinguishes two bf16 values); 4-byte rows: all 32 bits.
template <typename T>
struct RowCodes;
template <>
struct RowCodes<__nv_bfloat16> {
    static constexpr int kBits = 16;
    static constexpr int kPerVec = 8;                                               // values in 16 bytes
    __device__ static __forceinline__ uint32_t code_of_bits(uint32_t h) {       // h: the 16-bit pattern
        if ((h & 0x7FFFu) > 0x7F80u) h = 0xFF80u;                                  // NaN -> -inf
        if (h == 0x8000u) h = 0u;                                                  // -0 and +0 are one value
        return (h & 0x8000u) ? (~h & 0xFFFFu) : (h | 0x8000u);
    }
    __device__ static __forceinline__ uint32_t bits(const unsigned char* row, int i) { return ((const uint16_t*)row)[i]; }
    __device__ static __forceinline__ uint32_t code(const unsigned char* row, int i) { return code_of_bits(bits(row, i)); }
    __device__ static __forceinline__ float value_of_bits(uint32_t h) { return __uint_as_float(h << 16); }
    __device__ static __forceinline__ float value_of_code(uint32_t c) {
        const uint32_t h = (c & 0x8000u) ? (c & 0x7FFFu) : (~c & 0xFFFFu);
        return __uint_as_float(h << 16);
    }
    __device__ static __forceinline__ bool bits_nan(uint32_t h) { return (h & 0x7FFFu) > 0x7F80u; }
    __device__ static __forceinline__ uint32_t code_of_float(float v) { return code_of_bits(__float_as_uint(v) >> 16); }   // (truncated)
    // the 16-bit patterns of the 8 values of a 16-byte word
    __device__ static __forceinline__ void unpack_bits(const uint4& w, uint32_t (&h)[8]) {
        const uint32_t q[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) { h[2 * j] = q[j] & 0xFFFFu; h[2 * j + 1] = q[j] >> 16; }
    }
    __device__ static __forceinline__ uint4 pack_bits(const uint32_t (&h)[8]) {
        return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
    }
    static constexpr uint32_t kNegInfCode = 0x007Fu;                               // code of -inf (0xFF80)
    static constexpr uint32_t kNegInfBits = 0xFF80u;
};
template <>
struct RowCodes<float> {
    static constexpr int kBits = 32;
    static constexpr int kPerVec = 4;
    __device__ static __forceinline__ uint32_t code_of_bits(uint32_t u) {
        if ((u & 0x7FFFFFFFu) > 0x7F800000u) u = 0xFF800000u;
        if (u == 0x80000000u) u = 0u;                                              // -0 and +0 are one value
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static __forceinline__ uint32_t bits(const unsigned char* row, int i) { return ((const uint32_t*)row)[i]; }
    __device__ static __forceinline__ uint32_t code(const unsigned char* row, int i) { return code_of_bits(bits(row, i)); }
    __device__ static __forceinline__ float value_of_bits(uint32_t u) { return __uint_as_float(u); }
    __device__ static __forceinline__ float value_of_code(uint32_t c) {
        return __uint_as_float((c & 0x80000000u) ? (c & 0x7FFFFFFFu) : ~c);
    }
    __device__ static __forceinline__ bool bits_nan(uint32_t u) { return (u & 0x7FFFFFFFu) > 0x7F800000u; }
    __device__ static __forceinline__ uint32_t code_of_float(float v) { return code_of_bits(__float_as_uint(v)); }
    __device__ static __forceinline__ void unpack_bits(const uint4& w, uint32_t (&h)[4]) { h[0] = w.x; h[1] = w.y; h[2] = w.z; h[3] = w.w; }
    __device__ static __forceinline__ uint4 pack_bits(const uint32_t (&h)[4]) { return make_uint4(h[0], h[1], h[2], h[3]); }
    static constexpr uint32_t kNegInfCode = 0x007FFFFFu;
    static constexpr uint32_t kNegInfBits = 0xFF800000u;
};

// Largest value of a 16-byte word of the row (NaN ignored); `odd` is set when the word holds a NaN or a -inf.
template <typename T>
struct RowStats;
template <>
struct RowStats<__nv_bfloat16> {
    __device__ static __forceinline__ float largest(const uint4& w, bool& odd) {
        const uint32_t q[4] = {w.x, w.y, w.z, w.w};
        uint32_t m = 0xFF80FF80u, bad = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t le;
            asm("max.bf16x2 %0, %0, %1;" : "+r"(m) : "r"(q[j]));
            asm("set.leu.u32.bf16x2 %0, %1, %2;" : "=r"(le) : "r"(q[j]), "r"(0xFF80FF80u));   // <= -inf, or NaN
            bad |= le;
        }
        if (bad) odd = true;
        return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    }
};
template <>
struct RowStats<float> {
    __device__ static __forceinline__ float largest(const uint4& w, bool& odd) {
        const float v[4] = {__uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z), __uint_as_float(w.w)};
        float m = kNegInf;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            m = fmaxf(m, v[j]);
            if (!(v[j] > kNegInf)) odd = true;
        }
        return m;
    }
};

// Tests on a whole 16-byte word of the row.  They compare values, so +0 and -0 count as equal although their codes
// differ: callers treat the answers as a superset and look at the codes where that matters.
template <typename T>
struct RowVec;
template <>
struct RowVec<__nv_bfloat16> {
    __device__ static __forceinline__ uint32_t twice(float v) { return (__float_as_uint(v) >> 16) * 0x00010001u; }
    // bit j set when first <= entry j <= last
    __device__ static __forceinline__ uint32_t between(const uint4& w, float first, float last) {
        const uint32_t q[4] = {w.x, w.y, w.z, w.w}, f2 = twice(first), l2 = twice(last);
        uint32_t acc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t ge, le;
            asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(ge) : "r"(q[j]), "r"(f2));
            asm("set.le.u32.bf16x2 %0, %1, %2;" : "=r"(le) : "r"(q[j]), "r"(l2));
            acc |= ge & le & ((1u << (2 * j)) | (1u << (2 * j + 17)));
        }
        return (acc | (acc >> 16)) & 0xFFu;
    }
    // the word with -inf at the entries below `cut`; any_eq != 0 when an entry equals `cut`
    __device__ static __forceinline__ uint4 at_least(const uint4& w, float cut, uint32_t& any_eq) {
        const uint32_t q[4] = {w.x, w.y, w.z, w.w}, c2 = twice(cut);
        uint32_t o[4];
        any_eq = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t ge, eq;
            asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(ge) : "r"(q[j]), "r"(c2));
            asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(eq) : "r"(q[j]), "r"(c2));
            o[j] = (q[j] & ge) | (0xFF80FF80u & ~ge);
            any_eq |= eq;
        }
        return make_uint4(o[0], o[1], o[2], o[3]);
    }
};
template <>
struct RowVec<float> {
    __device__ static __forceinline__ uint32_t between(const uint4& w, float first, float last) {
        const float v[4] = {__uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z), __uint_as_float(w.w)};
        uint32_t acc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) acc |= (v[j] >= first && v[j] <= last) ? 1u << j : 0u;
        return acc;
    }
    __device__ static __forceinline__ uint4 at_least(const uint4& w, float cut, uint32_t& any_eq) {
        const uint32_t q[4] = {w.x, w.y, w.z, w.w};
        uint32_t o[4];
        any_eq = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float v = __uint_as_float(q[j]);
            o[j] = v >= cut ? q[j] : 0xFF800000u;
            any_eq |= v == cut ? 1u : 0u;
        }
        return make_uint4(o[0], o[1], o[2], o[3]);
    }
};

// A cut in the order (value descending, token ascending): a token is at or before the cut iff its code is larger,
// or equal with a token index not beyond `tok`.
struct Cut {
    uint32_t code;
    int tok;
};
__device__ __forceinline__ bool within(const Cut& c, uint32_t code, int i) { return code > c.code || (code == c.code && i <= c.tok); }

// inclusive prefix sum of a 64-bit word over the block (sm.scan_w as scratch); `total` = the sum over all threads
__device__ __forceinline__ unsigned long long block_scan_u64(unsigned long long v, unsigned long long* scratch, unsigned long long& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += up;
    }
    if (lane == 31) scratch[warp] = v;
    __syncthreads();
    unsigned long long before = 0;
    total = 0;
#pragma unroll
    for (int w = 0; w < kFilterWarps; ++w) {
        const unsigned long long s = scratch[w];
        if (w < warp) before += s;
        total += s;
    }
    __syncthreads();
    return v + before;
}

template <typename T>
struct RowFilter {
    FilterSmem& sm;
    const unsigned char* row;   // shared memory, NaN already turned into -inf
    int V;
    float k, neg_c;             // weight of a value: 2^(value * k + neg_c)
    int n_list;                 // >= 0: the tokens still in play are sm.list[0 .. n_list); -1: the whole row

    static constexpr int kPerVec = RowCodes<T>::kPerVec;

    __device__ __forceinline__ float weight_of_value(float v) const { return ex2_approx(fmaf(v, k, neg_c)); }
    __device__ __forceinline__ float weight(uint32_t code) const { return weight_of_value(RowCodes<T>::value_of_code(code)); }
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

    // f(i, bits) for every token i of the row (the row as 16-byte words, then the few entries past the last whole word)
    template <typename F>
    __device__ __forceinline__ void for_each_token(F f) const {
        const int n_vec = V / kPerVec;
        for (int m = threadIdx.x; m < n_vec; m += kFilterThreads) {
            uint32_t h[kPerVec];
            RowCodes<T>::unpack_bits(((const uint4*)row)[m], h);
#pragma unroll
            for (int j = 0; j < kPerVec; ++j) f(m * kPerVec + j, h[j]);
        }
        for (int i = n_vec * kPerVec + threadIdx.x; i < V; i += kFilterThreads) f(i, RowCodes<T>::bits(row, i));
    }

    // Bins of equal width in value over [v_lo, v_hi], bin 0 at the top; values below v_lo fall into the last bin.
    struct Coarse {
        float v_hi, scale;
        __device__ __forceinline__ int bin(float v) const {
            const float d = fminf((v_hi - v) * scale, (float)(kCoarseBins - 1));
            return (int)(__float_as_uint(d + 12582912.0f) & (uint32_t)(kCoarseBins - 1));   // round to nearest, in the low mantissa bits
        }
    };

    // First step of a search over the whole row: one sweep into the histogram, the bin that brings the tally to `need`,
    // and that bin's tokens gathered into the list.  Returns false (nothing changed but r.total_mass and `need`) when
    // the interval is too narrow for bins in value or the bin holds more tokens than the list.
    template <bool BY_MASS>
    __device__ __forceinline__ bool coarse_step(uint32_t& lo, uint32_t& hi, double& need, double need_frac, bool need_is_frac,
                                                const Cut& inside, bool everything, Found& r) {
        const int tid = threadIdx.x;
        Coarse cb;
        cb.v_hi = RowCodes<T>::value_of_code(hi);
        const float v_lo = fmaxf(RowCodes<T>::value_of_code(lo), cb.v_hi - kValueRange * kLog2e / k);
        const float width = cb.v_hi - v_lo;
        if (!(width > 0.0f) || !(width < 3.0e38f) || hi - lo < 4096u || V > 65536) return false;
        cb.scale = (float)(kCoarseBins - 1) / width;
        // Fixed point of the weights: V weights of at most 1 must fit below the count.  32 fraction bits up to 32,767
        // entries, 31 up to 65,535 (the conversion saturates at 2^32 - 1, which only the row's largest value can reach).
        // A weight is off by at most half a unit, so the tally is within V 2^-(bits + 1) of the exact sum relative to
        // the row's largest weight (4e-6 for 32,000 entries in the worst case, around 1e-8 in practice).
        const int frac_bits = min(32, kCountShift - (32 - __clz(V)));
        const float to_fixed = __uint_as_float((uint32_t)(127 + frac_bits) << 23);
        for (int q = tid; q < kCoarseBins; q += kFilterThreads) { sm.hist.lo[q] = 0u; sm.hist.hi[q] = 0u; }
        __syncthreads();
        for_each_token([&](int i, uint32_t h) {
            const float v = RowCodes<T>::value_of_bits(h);
            if (everything) {
                if (!(v > kNegInf)) return;                       // -inf (NaN is gone): neither counted nor weighed
            } else {
                const uint32_t code = RowCodes<T>::code_of_bits(h);
                if (code < lo || code > hi || !within(inside, code, i) || code <= RowCodes<T>::kNegInfCode) return;
            }
            const int q = cb.bin(v);
            uint32_t up = 1u << (kCountShift - 32);                // the count's unit in the high half
            if (BY_MASS) {                                         // a 64-bit addition as two 32-bit ones with the carry
                const uint32_t w = __float2uint_rn(weight_of_value(v) * to_fixed);
                const uint32_t old = atomicAdd(&sm.hist.lo[q], w);
                up += (old + w < old) ? 1u : 0u;
            }
            atomicAdd(&sm.hist.hi[q], up);
        });
        __syncthreads();
        // ---- tally from the top bin down: eight bins per thread, then a prefix sum over the threads ---------------------
        constexpr int kPer = kCoarseBins / kFilterThreads;
        unsigned long long mine = 0;
#pragma unroll
        for (int e = 0; e < kPer; ++e) mine += ((unsigned long long)sm.hist.hi[tid * kPer + e] << 32) | sm.hist.lo[tid * kPer + e];
        unsigned long long total;
        const unsigned long long incl = block_scan_u64(mine, sm.scan_w, total);
        const unsigned long long mass_mask = (1ull << kCountShift) - 1ull;
        const double from_fixed = 1.0 / (double)(1ull << frac_bits);
        if (BY_MASS) {
            r.total_mass = (double)(total & mass_mask) * from_fixed;
            if (need_is_frac) need = need_frac * r.total_mass;
        }
        if (tid == 0) sm.pick_bin = -1;
        __syncthreads();
        {
            unsigned long long run = incl - mine;   // everything above this thread's bins
            auto tally = [&](unsigned long long w) { return BY_MASS ? (double)(w & mass_mask) * from_fixed : (double)(w >> kCountShift); };
            if (tally(run) < need && tally(incl) >= need) {
#pragma unroll
                for (int e = 0; e < kPer; ++e) {
                    const unsigned long long w = ((unsigned long long)sm.hist.hi[tid * kPer + e] << 32) | sm.hist.lo[tid * kPer + e];
                    if (tally(run + w) >= need) { sm.pick_bin = tid * kPer + e; sm.pick_above = run; break; }
                    run += w;
                }
            }
        }
        __syncthreads();
        const int pick = sm.pick_bin;
        if (pick < 0) return false;                                 // (need beyond the total: left to the search over the row)
        const unsigned long long above = sm.pick_above;
        const int population = (int)(sm.hist.hi[pick] >> (kCountShift - 32));
        __syncthreads();
        if (population > kListCap) return false;
        // ---- the codes of the picked bin: the bin index does not increase with the code, so both ends come from a
        // bisection over the codes with the same arithmetic as the sweep ----------------------------------------------------
        if (threadIdx.x == 0) {                                      // (two threads of two warps: the others sleep at the barrier)
            uint32_t a_ = lo, b_ = hi;                               // smallest code with bin <= pick
            while (a_ < b_) {
                const uint32_t mid = a_ + ((b_ - a_) >> 1);
                if (cb.bin(RowCodes<T>::value_of_code(mid)) <= pick) b_ = mid; else a_ = mid + 1u;
            }
            sm.bound[0] = a_;
        } else if (threadIdx.x == 32) {
            uint32_t a_ = lo, b_ = hi;                               // largest code with bin >= pick
            while (a_ < b_) {
                const uint32_t mid = a_ + ((b_ - a_ + 1u) >> 1);
                if (cb.bin(RowCodes<T>::value_of_code(mid)) >= pick) a_ = mid; else b_ = mid - 1u;
            }
            sm.bound[1] = a_;
        }
        __syncthreads();
        const uint32_t first_in = sm.bound[0], last_in = sm.bound[1];   // smallest and largest code of [lo, hi] in the bin
        __syncthreads();
        if (first_in > last_in) return false;
        gather(first_in, last_in, inside, everything);
        if (n_list < 0) return false;
        r.above_mass = (double)(above & mass_mask) * from_fixed;
        r.above_count = (int)(above >> kCountShift);
        lo = first_in;
        hi = last_in;
        return true;
    }

    // The largest code t in [lo, hi] with F(t) >= need, F(t) = the number (BY_MASS = false) or the weight (BY_MASS = true)
    // of the tokens within `inside` whose code is >= t.  need = need_abs, or, when need_abs < 0, need_frac times the
    // total weight of the tokens within `inside` (they all lie in [lo, hi]: the first pass measures it).  F is
    // non-increasing, F(lo) >= need, nothing within `inside` lies above hi.  `everything`: `inside` holds every finite
    // token of the row and lo is the smallest finite code (the checks per token then reduce to "finite").
    template <bool BY_MASS>
    __device__ __forceinline__ Found search(uint32_t lo, uint32_t hi, double need_abs, double need_frac, const Cut& inside, bool everything) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        Found r = {lo, 0.0, 0, 0.0};
        double need = need_abs;
        int level = 0;
        if (n_list < 0 && coarse_step<BY_MASS>(lo, hi, need, need_frac, need_abs < 0.0, inside, everything, r)) {
            level = 1;
            if (lo >= hi) { r.t = lo; return r; }
        } else {
            r.above_mass = 0.0;
            r.above_count = 0;
        }
        const bool total_known = level > 0;   // (a first step that gave up leaves everything to the passes below)
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
                    bd = (c < lo || c > hi) ? hi : c;                        // bins past the interval's end are empty:
                }                                                            // they all start at hi, and only the last holds it
                sm.bound[tid] = bd;
            }
            if (tid < kFineThreads) {
#pragma unroll
                for (int q = 0; q < kBins; ++q) { sm.fine.mass[q][tid] = 0.0f; sm.fine.count[q][tid] = 0; }
            }
            __syncthreads();
            // bins that start at the same code: only the last of them is used (the search below takes the largest q)
            const int n_items = items();
            for (int m = tid; m < n_items && tid < kFineThreads; m += kFineThreads) {
                const int i = index(m);
                const uint32_t code = RowCodes<T>::code(row, i);
                if (code < lo || code > hi || !within(inside, code, i) || code <= RowCodes<T>::kNegInfCode) continue;
                int q = code >= sm.bound[8] ? 8 : 0;
                q += code >= sm.bound[q + 4] ? 4 : 0;
                q += code >= sm.bound[q + 2] ? 2 : 0;
                q += code >= sm.bound[q + 1] ? 1 : 0;
                if (q == kBins) q = kBins - 1;                               // code == hi == bound[16]
                sm.fine.mass[q][tid] += weight(code);
                sm.fine.count[q][tid] += 1;
            }
            __syncthreads();
            // ---- totals of the bins: warp w adds up bin w, every lane eight threads' entries in order, then a fixed
            // tree over the lanes -----------------------------------------------------------------------------------------------
            static_assert(kFilterWarps == kBins, "one warp per bin");
            {
                const int q = warp;
                double v = 0.0;
                int c = 0;
#pragma unroll
                for (int e = 0; e < kFineThreads / 32; ++e) {
                    v += (double)sm.fine.mass[q][lane * (kFineThreads / 32) + e];
                    c += (int)sm.fine.count[q][lane * (kFineThreads / 32) + e];
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                c = __reduce_add_sync(0xFFFFFFFFu, c);
                if (lane == 0) { sm.mass_total[q] = v; sm.count_total[q] = c; }
            }
            __syncthreads();
            if (level == 0 && !total_known) {
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
            if (n_list < 0 && population <= kListCap && V <= 65536) gather(lo, hi, inside, false);
        }
        r.t = lo;
        return r;
    }

    // The indices of the tokens within `inside` with a code in [lo, hi], in token order, into sm.list (n_list stays -1
    // when they do not fit).  Threads own consecutive runs of 16-byte words; one prefix count over the block.
    __device__ __forceinline__ void gather(uint32_t lo, uint32_t hi, const Cut& inside, bool everything) {
        const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
        const int n_vec = (V + kPerVec - 1) / kPerVec;                 // the row's buffer is padded to whole words with -inf
        const int per = (n_vec + kFilterThreads - 1) / kFilterThreads;
        const int m0 = min(n_vec, tid * per), m1 = min(n_vec, m0 + per);
        auto member = [&](int i, uint32_t h) {
            const uint32_t code = RowCodes<T>::code_of_bits(h);
            return code >= lo && code <= hi && code > RowCodes<T>::kNegInfCode && (everything || within(inside, code, i)) && i < V;
        };
        // bit (m - m0) * kPerVec + j of `marks`: entry j of word m may belong (`everything`: a test on the values of
        // whole words, which is a superset; the passes over the list look at the codes again)
        const float v_first = RowCodes<T>::value_of_code(lo), v_last = RowCodes<T>::value_of_code(hi);
        const bool by_word = everything && per * kPerVec <= 128 && lo > RowCodes<T>::kNegInfCode;   // (padding is -inf: never marked)
        unsigned long long marks[2] = {0ull, 0ull};
        int mine = 0;
        for (int m = m0; m < m1; ++m) {
            if (by_word) {
                const unsigned long long in = RowVec<T>::between(((const uint4*)row)[m], v_first, v_last);
                const int at_bit = (m - m0) * kPerVec;               // (a word's bits never straddle the two halves)
                if (at_bit < 64) marks[0] |= in << at_bit;
                else marks[1] |= in << (at_bit - 64);
            } else {
                uint32_t h[kPerVec];
                RowCodes<T>::unpack_bits(((const uint4*)row)[m], h);
#pragma unroll
                for (int j = 0; j < kPerVec; ++j) mine += member(m * kPerVec + j, h[j]) ? 1 : 0;
            }
        }
        if (by_word) mine = __popcll(marks[0]) + __popcll(marks[1]);
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
        if (total <= kListCap && mine > 0) {
            if (by_word) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    unsigned long long left = marks[half];
                    while (left) {
                        const int bit = __ffsll((long long)left) - 1;
                        left &= left - 1ull;
                        sm.list[at++] = (uint16_t)(m0 * kPerVec + half * 64 + bit);
                    }
                }
            } else {
                for (int m = m0; m < m1; ++m) {
                    uint32_t h[kPerVec];
                    RowCodes<T>::unpack_bits(((const uint4*)row)[m], h);
#pragma unroll
                    for (int j = 0; j < kPerVec; ++j)
                        if (member(m * kPerVec + j, h[j])) sm.list[at++] = (uint16_t)(m * kPerVec + j);
                }
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
    extern __shared__ __align__(16) unsigned char row_sm[];   // the row, padded with -inf to whole 16-byte words
    __shared__ FilterSmem sm;
    constexpr int kElem = (int)sizeof(T);
    constexpr int kPerVec = RowCodes<T>::kPerVec;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / a.R, r = blockIdx.x % a.R, V = a.V;
    const unsigned char* src = (const unsigned char*)a.data + ((int64_t)b * a.seq_stride + (int64_t)r * a.row_stride) * kElem;
    unsigned char* dst = (unsigned char*)a.out + ((int64_t)b * a.R + r) * (int64_t)V * kElem;
    const int n_vec = V / kPerVec;                               // whole 16-byte words of the row

    // ---- the row into shared memory, NaN as -inf; its largest value and the number of finite entries ------------------
    // Rows that start on a 16-byte boundary come in by one bulk copy of the whole words, the others by plain loads.  A
    // first look takes the largest value and notes whether anything is NaN or -inf; only then is the row gone over
    // entry by entry to replace and count them.
    const bool bulk = ((uintptr_t)src & 15u) == 0 && n_vec > 0;
    if (tid == 0) {
        sm.nan_flag = 0;
        sm.copy_gave_up = 0;
        sm.needs_cleaning = 0;
        if (bulk) {
            mbar_init(&sm.row_bar, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
    }
    __syncthreads();
    if (bulk) {
        if (tid == 0) {
            // (an mbarrier counts at most 2^20 - 1 bytes per phase, a row has fewer)
            mbar_expect_tx(&sm.row_bar, (uint32_t)n_vec * 16u);
            bulk_load(row_sm, src, (uint32_t)n_vec * 16u, &sm.row_bar);
        }
    } else {
        for (int i = tid; i < n_vec * kPerVec; i += kFilterThreads) {
            if (kElem == 2) ((uint16_t*)row_sm)[i] = (uint16_t)RowCodes<T>::bits(src, i);
            else ((uint32_t*)row_sm)[i] = RowCodes<T>::bits(src, i);
        }
    }
    if (tid < kPerVec && n_vec * kPerVec < V) {                  // the last, partial word, padded with -inf
        const int i = n_vec * kPerVec + tid;
        const uint32_t h = i < V ? RowCodes<T>::bits(src, i) : RowCodes<T>::kNegInfBits;
        if (kElem == 2) ((uint16_t*)row_sm)[i] = (uint16_t)h;
        else ((uint32_t*)row_sm)[i] = h;
    }
    if (bulk && warp == 0) wait_bar(&sm.row_bar, 0, &sm.copy_gave_up);   // one warp polls, the others sleep at the barrier
    __syncthreads();
    if (bulk && warp != 0 && !sm.copy_gave_up) wait_bar(&sm.row_bar, 0, &sm.copy_gave_up);   // (done: every thread has now seen the copy's completion itself)
    __syncthreads();
    if (sm.copy_gave_up) {                                        // the copy never landed: report, write nothing
        if (tid == 0) atomicOr(&a.status[b], 32);                 // RSD_ST_TIMEOUT
        return;
    }
    uint32_t top = RowCodes<T>::kNegInfCode;
    int finite = V;
    {
        const int n_all = (V + kPerVec - 1) / kPerVec;           // with the padded word
        float vtop = kNegInf;
        bool odd = false;                                        // something is NaN or -inf
        for (int m = tid; m < n_all; m += kFilterThreads) {
            const uint4 w = ((const uint4*)row_sm)[m];
            vtop = fmaxf(vtop, RowStats<T>::largest(w, odd));
        }
        if (odd) sm.needs_cleaning = 1;
        // (+0 and -0 are equal as values but not as codes: the larger code stands for both)
        top = vtop == 0.0f ? RowCodes<T>::code_of_float(0.0f) : (vtop > kNegInf ? RowCodes<T>::code_of_float(vtop) : RowCodes<T>::kNegInfCode);
    }
    __syncthreads();
    if (sm.needs_cleaning) {
        bool saw_nan = false;
        int not_finite = 0;
        const int n_all = (V + kPerVec - 1) / kPerVec;
        for (int m = tid; m < n_all; m += kFilterThreads) {
            uint32_t h[kPerVec];
            RowCodes<T>::unpack_bits(((const uint4*)row_sm)[m], h);
#pragma unroll
            for (int j = 0; j < kPerVec; ++j) {
                if (RowCodes<T>::bits_nan(h[j])) { saw_nan = true; h[j] = RowCodes<T>::kNegInfBits; }
                not_finite += (h[j] == RowCodes<T>::kNegInfBits && m * kPerVec + j < V) ? 1 : 0;
            }
            ((uint4*)row_sm)[m] = RowCodes<T>::pack_bits(h);
        }
        finite = -not_finite;                                    // (V is added back after the sum over the block)
        if (saw_nan) sm.nan_flag = 1;
    } else {
        finite = 0;
    }
    top = __reduce_max_sync(0xFFFFFFFFu, top);
    finite = __reduce_add_sync(0xFFFFFFFFu, finite);
    if (lane == 0) { sm.red_i[warp][0] = (int)top; sm.red_i[warp][1] = finite; }
    __syncthreads();
    top = 0u;
    finite = V;
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
    bool everything = true;

    // ---- top-k: the value of the k-th largest entry, then the last kept token among its equals -------------------------
    if (a.top_k > 0 && a.top_k < V && finite > a.top_k) {
        const typename RowFilter<T>::Found r = f.template search<false>(RowCodes<T>::kNegInfCode + 1u, top, (double)a.top_k, 0.0, cut, true);
        int ties;
        const int tok = f.nth_with_code(r.t, a.top_k - r.above_count, cut, ties);   // that many of the entries equal to t stay
        cut.code = r.t;
        cut.tok = tok >= 0 ? tok : V;
        kept = a.top_k;
        f.n_list = -1;                                            // (the list was gathered for the old cut)
        everything = false;
    }
    // ---- top-p: of what is left, the shortest prefix (value descending, token ascending) whose mass reaches top_p -------
    if (a.top_p > 0.0f && a.top_p < 1.0f && kept > 0 && !plus_inf) {
        const typename RowFilter<T>::Found r = f.template search<true>(everything ? RowCodes<T>::kNegInfCode + 1u : cut.code, top, -1.0,
                                                                       (double)a.top_p, cut, everything);
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
    {
        auto keep_bits = [&](int i, uint32_t h) {
            const uint32_t c = RowCodes<T>::code_of_bits(h);
            return (c > RowCodes<T>::kNegInfCode && within(cut, c, i)) ? h : RowCodes<T>::kNegInfBits;
        };
        const bool dst16 = ((uintptr_t)dst & 15u) == 0;
        const float cut_value = RowCodes<T>::value_of_code(cut.code);
        for (int m = tid; m < n_vec; m += kFilterThreads) {
            const uint4 w = ((const uint4*)row_sm)[m];
            uint32_t any_eq;
            uint4 o = RowVec<T>::at_least(w, cut_value, any_eq);   // right wherever no entry equals the cut's value
            if (any_eq) {                                          // there the codes and the tokens decide
                uint32_t h[kPerVec];
                RowCodes<T>::unpack_bits(w, h);
#pragma unroll
                for (int j = 0; j < kPerVec; ++j) h[j] = keep_bits(m * kPerVec + j, h[j]);
                o = RowCodes<T>::pack_bits(h);
            }
            if (dst16) {
                ((uint4*)dst)[m] = o;
            } else {
                uint32_t h[kPerVec];
                RowCodes<T>::unpack_bits(o, h);
#pragma unroll
                for (int j = 0; j < kPerVec; ++j) {
                    if (kElem == 2) ((uint16_t*)dst)[m * kPerVec + j] = (uint16_t)h[j];
                    else ((uint32_t*)dst)[m * kPerVec + j] = h[j];
                }
            }
        }
        for (int i = n_vec * kPerVec + tid; i < V; i += kFilterThreads) {
            const uint32_t h = keep_bits(i, RowCodes<T>::bits(row_sm, i));
            if (kElem == 2) ((uint16_t*)dst)[i] = (uint16_t)h;
            else ((uint32_t*)dst)[i] = h;
        }
    }
    if (tid == 0) {
        if (a.kept) a.kept[(int64_t)b * a.R + r] = kept;
        if (sm.nan_flag) atomicOr(&a.status[b], 1);               // RSD_ST_NAN_INPUT
    }
}

}  // namespace rsd
