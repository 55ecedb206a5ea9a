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

#ifndef RSD_VERIFY_MIN_BLOCKS
#define RSD_VERIFY_MIN_BLOCKS 3       // blocks per SM the walk is compiled for, 2-byte rows
#endif
#ifndef RSD_VERIFY_MIN_BLOCKS_F32
#define RSD_VERIFY_MIN_BLOCKS_F32 2   // 4-byte rows: a group in flight is 16 registers per row
#endif
#ifndef RSD_VERIFY_THREADS
#define RSD_VERIFY_THREADS 256
#endif
constexpr int kVerifyThreads = RSD_VERIFY_THREADS;
constexpr int kVerifyWarps = kVerifyThreads / 32;
constexpr int kMaxTiles = 512;        // tiles of 512 elements: V <= 262144
constexpr int kMaxCachedNodes = 384;  // trees up to this size are copied to shared memory
constexpr int kMaxRemoved = 32;      // removed tokens tracked per node (later ones carry no residual mass)
constexpr int kPassUnroll = 4;        // turns of a pass whose warp-wide sums are taken together
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

struct VerifySmem {
    double tile_sum[kMaxTiles];
    double red_d[kVerifyWarps], red_d2[kVerifyWarps];
    float red_f[kVerifyWarps], red_f2[kVerifyWarps];
    int red_i[kVerifyWarps];
    int nan_flag;
    int pick;
    // tokens removed from the draft at the current node: index, the two exponentials, and the weight frozen at removal
    int par[kMaxCachedNodes], tok[kMaxCachedNodes];   // the sequence's tree (small trees only)
    int n_removed;
    int rem_x[kMaxRemoved];
    float rem_qh[kMaxRemoved], rem_ph[kMaxRemoved], rem_w[kMaxRemoved];
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

// Row maximum over the first block-wide sweep (cheap reference), or over the whole row when asked.
template <typename T, bool ALIGNED>
__device__ __forceinline__ float row_reference(const char* row, int V, bool whole_row, VerifySmem& sm, bool& saw_nan) {
    const int n_groups = (V + 15) >> 4;
    float m = kNegInf;
    float v[16];
    for (int g = threadIdx.x; g < n_groups; g += kVerifyThreads) {
        m = fmaxf(m, load_clean<T, ALIGNED>(row, g, V, v, saw_nan));
        if (!whole_row) break;
    }
    return block_max<kVerifyThreads>(m, sm.red_f);
}

// One pass over the row(s): weights w(y) = (qhat(y) - a phat(y))+ with qhat = exp(lt - m_q), phat = exp(ld - m_p)
// (a = 0, no draft row: plain exponentials of the target).  Leaves the sum of every 512-element tile in
// sm.tile_sum, returns their total (summed in tile order, identically on all threads) and the true row maxima.
template <typename T, bool ALIGNED, int MODE>
__device__ __forceinline__ double weight_pass(const char* rowq, const char* rowp, int V, float mq, float mp, float kq, float kp,
                              float a_hi, float a_lo,
                              VerifySmem& sm, bool& saw_nan, float* true_max_q, float* true_max_p, float c_seq = 0.0f) {
    constexpr bool WITH_DRAFT = MODE != kTargetOnly;
    const int n_groups = (V + 15) >> 4;
    const int n_tiles = (n_groups + 31) >> 5;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float cq_ = mq * kq, cp_ = mp * kp;   // kq, kp = log2(e) / temperature of the row
    float tmq = kNegInf, tmp_ = kNegInf;
    const int n_iter = (n_groups + kVerifyThreads - 1) / kVerifyThreads;
    // The groups of the next turn are loaded before the current ones are worked on, and the warp-wide sums of
    // kPassUnroll turns are taken together: a block that has an SM to itself (the long walks at the end of a launch)
    // is otherwise idle for one load latency plus one chain of shuffles per turn.
    Packed<T> nq, np;
    if ((int)threadIdx.x < n_groups) {
        load_raw<T, ALIGNED>(nq, rowq, threadIdx.x, V);
        if (WITH_DRAFT) load_raw<T, ALIGNED>(np, rowp, threadIdx.x, V);
    }
    for (int it0 = 0; it0 < n_iter; it0 += kPassUnroll) {
        float gs[kPassUnroll];
#pragma unroll
        for (int u = 0; u < kPassUnroll; ++u) {
            const int g = (it0 + u) * kVerifyThreads + threadIdx.x;
            gs[u] = 0.0f;
            if (it0 + u < n_iter) {
                const Packed<T> cq = nq, cp = np;
                if (g + kVerifyThreads < n_groups) {
                    load_raw<T, ALIGNED>(nq, rowq, g + kVerifyThreads, V);
                    if (WITH_DRAFT) load_raw<T, ALIGNED>(np, rowp, g + kVerifyThreads, V);
                }
                if (g < n_groups) {
                    float q[16], w[16];
                    tmq = fmaxf(tmq, clean<T>(cq, q, saw_nan));
                    if (WITH_DRAFT) {
                        float p[16];
                        tmp_ = fmaxf(tmp_, clean<T>(cp, p, saw_nan));
                        exp16(q, kq, cq_, q);
                        exp16(p, kp, cp_, p);
                        weights16<MODE>(q, p, a_hi, a_lo, c_seq, w);
                    } else {
                        exp16(q, kq, cq_, w);
                    }
                    gs[u] = tree_sum16(w);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kPassUnroll; ++u) {
            const double ts = warp_sum((double)gs[u]);
            const int tile = (it0 + u) * kVerifyWarps + warp;
            if (lane == 0 && tile < n_tiles) sm.tile_sum[tile] = ts;
        }
    }
    if (true_max_q) *true_max_q = block_max<kVerifyThreads>(tmq, sm.red_f);
    if (true_max_p) *true_max_p = block_max<kVerifyThreads>(tmp_, sm.red_f);
    __syncthreads();
    if (MODE == kResidual && sm.n_removed > 0) {  // removed tokens weigh what they weighed at removal
        if (threadIdx.x == 0) {
            for (int i = 0; i < sm.n_removed; ++i) {
                const float generic = residual_weight(sm.rem_qh[i], sm.rem_ph[i], a_hi, a_lo);
                if (generic != sm.rem_w[i]) sm.tile_sum[sm.rem_x[i] >> 9] += (double)sm.rem_w[i] - (double)generic;
            }
        }
        __syncthreads();
    }
    // total in a fixed order (strided partial sums, then warps), the same on every thread
    double part = 0.0;
    for (int t = threadIdx.x; t < n_tiles; t += kVerifyThreads) part += sm.tile_sum[t];
    return block_sum<kVerifyThreads>(part, sm.red_d);
}

// Both normalisers of a node in one pass: S_q = sum exp(lt - m_q), S_p = sum exp(ld - m_p).
template <typename T, bool ALIGNED>
__device__ __forceinline__ void softmax_sums(const char* rowq, const char* rowp, int V, float mq, float mp, float kq, float kp,
                             VerifySmem& sm,
                             bool& saw_nan, double* Sq, double* Sp, float* true_max_q, float* true_max_p) {
    const int n_groups = (V + 15) >> 4;
    const float cq = mq * kq, cp = mp * kp;   // kq, kp = log2(e) / temperature of the row
    float tmq = kNegInf, tmp_ = kNegInf;
    double accq = 0.0, accp = 0.0;
    Packed<T> nq, np;
    if ((int)threadIdx.x < n_groups) {
        load_raw<T, ALIGNED>(nq, rowq, threadIdx.x, V);
        load_raw<T, ALIGNED>(np, rowp, threadIdx.x, V);
    }
    for (int g = threadIdx.x; g < n_groups; g += kVerifyThreads) {
        const Packed<T> cq_raw = nq, cp_raw = np;
        if (g + kVerifyThreads < n_groups) {   // next turn's groups first
            load_raw<T, ALIGNED>(nq, rowq, g + kVerifyThreads, V);
            load_raw<T, ALIGNED>(np, rowp, g + kVerifyThreads, V);
        }
        float q[16], p[16];
        tmq = fmaxf(tmq, clean<T>(cq_raw, q, saw_nan));
        tmp_ = fmaxf(tmp_, clean<T>(cp_raw, p, saw_nan));
        exp16(q, kq, cq, q);
        exp16(p, kp, cp, p);
        accq += (double)tree_sum16(q);
        accp += (double)tree_sum16(p);
    }
    // the four block-wide results behind one pair of barriers
    accq = warp_sum(accq);
    accp = warp_sum(accp);
    tmq = warp_max(tmq);
    tmp_ = warp_max(tmp_);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) {
        const int w = threadIdx.x >> 5;
        sm.red_d[w] = accq;
        sm.red_d2[w] = accp;
        sm.red_f[w] = tmq;
        sm.red_f2[w] = tmp_;
    }
    __syncthreads();
    double sq = 0.0, sp = 0.0;
    float xq = sm.red_f[0], xp = sm.red_f2[0];
#pragma unroll
    for (int w = 0; w < kVerifyWarps; ++w) {   // fixed order: the same on every thread
        sq += sm.red_d[w];
        sp += sm.red_d2[w];
        xq = fmaxf(xq, sm.red_f[w]);
        xp = fmaxf(xp, sm.red_f2[w]);
    }
    *Sq = sq;
    *Sp = sp;
    *true_max_q = xq;
    *true_max_p = xp;
}

// Inverse CDF over the weights of the last weight_pass: the smallest y whose running sum exceeds u * total; if
// rounding leaves none, the largest y with positive weight; -1 if there is no weight at all.
template <typename T, bool ALIGNED, int MODE>
__device__ __forceinline__ int inverse_cdf_pick(const char* rowq, const char* rowp, int V, float mq, float mp, float kq, float kp,
                                float a_hi, float a_lo,
                                double total, double u, VerifySmem& sm, float c_seq = 0.0f) {
    constexpr bool WITH_DRAFT = MODE != kTargetOnly;
    const int n_groups = (V + 15) >> 4;
    const int n_tiles = (n_groups + 31) >> 5;
    if (!(total > 0.0) || total > 1.7e308) return -1;
    const double target = u * total;
    // every thread finds the tile the same way
    int tile = -1, last_pos_tile = -1;
    double before = 0.0, before_last = 0.0;
    {
        double cum = 0.0;
        for (int t = 0; t < n_tiles; ++t) {
            const double s = sm.tile_sum[t];
            if (s > 0.0) { last_pos_tile = t; before_last = cum; }
            if (cum + s > target) { tile = t; before = cum; break; }
            cum += s;
        }
    }
    bool take_last = false;
    if (tile < 0) { tile = last_pos_tile; before = before_last; take_last = true; }
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        const int g = tile * 32 + lane;
        float w[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) w[j] = 0.0f;
        if (g < n_groups) {
            float q[16];
            bool dummy = false;
            load_clean<T, ALIGNED>(rowq, g, V, q, dummy);
            const float cq = mq * kq, cp = mp * kp;   // kq, kp = log2(e) / temperature of the row
            if (WITH_DRAFT) {
                float p[16];
                load_clean<T, ALIGNED>(rowp, g, V, p, dummy);
                exp16(q, kq, cq, q);
                exp16(p, kp, cp, p);
                weights16<MODE>(q, p, a_hi, a_lo, c_seq, w);
                for (int i = 0; MODE == kResidual && i < sm.n_removed; ++i) {
                    if ((sm.rem_x[i] >> 4) != g) continue;
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (j == (sm.rem_x[i] & 15)) w[j] = sm.rem_w[i];
                }
            } else {
                exp16(q, kq, cq, w);
            }
        }
        const double gs = (double)tree_sum16(w);
        double incl = gs;  // inclusive prefix over lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        const double excl = before + (incl - gs);
        const unsigned crossing = __ballot_sync(0xFFFFFFFFu, !take_last && (before + incl > target));
        const unsigned positive = __ballot_sync(0xFFFFFFFFu, gs > 0.0);
        int src;
        bool last_mode = take_last;
        if (crossing) src = __ffs(crossing) - 1;
        else { src = positive ? 31 - __clz(positive) : 0; last_mode = true; }
        if (lane == src) {
            int y = -1, last_pos = -1;
            double c = excl;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                c += (double)w[j];
                if (w[j] > 0.0f) last_pos = g * 16 + j;
                if (!last_mode && y < 0 && c > target) y = g * 16 + j;
            }
            sm.pick = (y >= 0) ? y : last_pos;
        }
    }
    __syncthreads();
    const int y = sm.pick;
    __syncthreads();
    return y;
}

// State of one sibling chain at a node; all threads hold identical copies.
// BASELINES: the chain also knows the two baseline rules; the plain instantiation carries none of their code.
template <typename T, bool ALIGNED, bool BASELINES = false>
struct NodeChain {
    const char* rowq;
    const char* rowp;
    int V;
    float mq, mp;       // reference values (raw units)
    float kq, kp;       // log2(e) / temperature of the target and draft rows
    double Sq, Sp;      // normalisers relative to the references
    double A, P, Z;     // closed-form chain state
    double total;       // sum of the weights of the last weight_pass (valid if tiles_current)
    float a_hi, a_lo;
    float c_seq;        // K-SEQ: the factor of its residual, set by seq_finish()
    int rule;           // 0 recursive, 1 multi-round (the draft is never changed), 2 K-SEQ
    double gamma;       // K-SEQ's parameter
    bool with_draft, tiles_current, seq_residual;

    __device__ void split_a() {
        const double a = A * Sq / Sp;
        a_hi = (float)a;
        a_lo = (float)(a - (double)a_hi);
    }

    // reference maxima and normalisers of the node (both rows)
    __device__ void open_both(const char* q, const char* p, int V_, float kq_, float kp_, VerifySmem& sm, bool& saw_nan) {
        rowq = q; rowp = p; V = V_; kq = kq_; kp = kp_; with_draft = true; tiles_current = false;
        A = 0.0; P = 0.0; Z = 1.0; a_hi = a_lo = 0.0f; c_seq = 0.0f; seq_residual = false;
        __syncthreads();
        if (threadIdx.x == 0) sm.n_removed = 0;
        __syncthreads();
        {   // first sweep of both rows, both loads in flight together, one pair of barriers
            float a = kNegInf, c = kNegInf;
            if ((int)threadIdx.x < ((V + 15) >> 4)) {
                Packed<T> pq, pp;
                load_raw<T, ALIGNED>(pq, rowq, threadIdx.x, V);
                load_raw<T, ALIGNED>(pp, rowp, threadIdx.x, V);
                float v[16];
                a = clean<T>(pq, v, saw_nan);
                c = clean<T>(pp, v, saw_nan);
            }
            a = warp_max(a);
            c = warp_max(c);
            if ((threadIdx.x & 31) == 0) { sm.red_f[threadIdx.x >> 5] = a; sm.red_f2[threadIdx.x >> 5] = c; }
            __syncthreads();
            mq = sm.red_f[0];
            mp = sm.red_f2[0];
#pragma unroll
            for (int w = 1; w < kVerifyWarps; ++w) { mq = fmaxf(mq, sm.red_f[w]); mp = fmaxf(mp, sm.red_f2[w]); }
        }
        if (!(mq > kNegInf)) mq = row_reference<T, ALIGNED>(rowq, V, true, sm, saw_nan);
        if (!(mp > kNegInf)) mp = row_reference<T, ALIGNED>(rowp, V, true, sm, saw_nan);
        for (int attempt = 0; attempt < 2; ++attempt) {
            float tq, tp;
            softmax_sums<T, ALIGNED>(rowq, rowp, V, mq, mp, kq, kp, sm, saw_nan, &Sq, &Sp, &tq, &tp);
            const bool redo = ((tq - mq) * kq > kRefSlack * kLog2e) || ((tp - mp) * kp > kRefSlack * kLog2e);
            if (!redo) break;
            mq = tq; mp = tp;
        }
    }

    // plain target row: weights exp(lt - m_q), total = S_q, tile sums ready for the draw
    __device__ void open_target_only(const char* q, int V_, float kq_, VerifySmem& sm, bool& saw_nan) {
        rowq = q; rowp = q; V = V_; kq = kq_; kp = kq_; with_draft = false; tiles_current = true;
        A = 0.0; P = 0.0; Z = 1.0; a_hi = a_lo = 0.0f; Sp = 1.0; mp = 0.0f; c_seq = 0.0f; seq_residual = false;
        __syncthreads();
        if (threadIdx.x == 0) sm.n_removed = 0;
        __syncthreads();
        mq = row_reference<T, ALIGNED>(rowq, V, false, sm, saw_nan);
        if (!(mq > kNegInf)) mq = row_reference<T, ALIGNED>(rowq, V, true, sm, saw_nan);
        for (int attempt = 0; attempt < 2; ++attempt) {
            float tq;
            total = weight_pass<T, ALIGNED, kTargetOnly>(rowq, rowq, V, mq, 0.0f, kq, kq, 0.0f, 0.0f, sm, saw_nan, &tq, nullptr);
            if (!((tq - mq) * kq > kRefSlack * kLog2e)) break;
            mq = tq;
        }
        Sq = total;
    }

    // probabilities of a token from its two row values (loaded by the caller, usually one pass early)
    __device__ double prob_q(float l) const {
        return (l == l) ? (double)ex2_approx(fmaf(l, kq, -mq * kq)) / Sq : 0.0;
    }
    __device__ double prob_p(float l) const {
        return (l == l) ? (double)ex2_approx(fmaf(l, kp, -mp * kp)) / Sp : 0.0;
    }

    // Eq. 3 for the next child, given its target and draft row values (K-SEQ: min{1, q(x) / (gamma p(x))})
    __device__ double threshold(float lq, float lp, int& st) const {
        const double qx = prob_q(lq), px = prob_p(lp);
        if (BASELINES && rule == 2) {
            if (px > 0.0) return fmin(1.0, qx / (gamma * px));
            st |= 8;
            return qx > 0.0 ? 1.0 : 0.0;
        }
        const double r = fmax(qx - A * px, 0.0);
        if (px > 0.0) return fmin(1.0, r * (1.0 - P) / (Z * px));
        st |= 8;  // RSD_ST_ZERO_DRAFT_PROB
        return r > 0.0 ? 1.0 : 0.0;
    }

    // Eqs. 1-2 after rejecting x (row values lq, lp).  Returns false if the draft has no mass left.
    __device__ bool reject(int x, float lq, float lp, VerifySmem& sm, bool& saw_nan, int& st) {
        const double px = prob_p(lp);
        const double A_new = A + Z / (1.0 - P);
        const double A_old = A;
        A = A_new;
        split_a();
        const double zhat = weight_pass<T, ALIGNED, kResidual>(rowq, rowp, V, mq, mp, kq, kp, a_hi, a_lo, sm, saw_nan, nullptr, nullptr);
        const double Z_new = zhat / Sq;
        if (Z_new > 0.0 && Z_new < 1.7e308) {
            Z = Z_new;
            total = zhat;
            tiles_current = true;
        } else {
            st |= 4;  // RSD_ST_ZERO_RESIDUAL: keep the previous residual
            A = A_old;
            split_a();
            tiles_current = false;
        }
        if (BASELINES && rule == 1) return true;   // multi-round rejection sampling: the draft stays as it is
        P += px;
        __syncthreads();
        if (threadIdx.x == 0 && sm.n_removed < kMaxRemoved) {
            const int i = sm.n_removed++;
            sm.rem_x[i] = x;
            sm.rem_qh[i] = (lq == lq) ? ex2_approx(fmaf(lq, kq, -mq * kq)) : 0.0f;
            sm.rem_ph[i] = (lp == lp) ? ex2_approx(fmaf(lp, kp, -mp * kp)) : 0.0f;
            sm.rem_w[i] = residual_weight(sm.rem_qh[i], sm.rem_ph[i], a_hi, a_lo);
        }
        __syncthreads();
        if (!(1.0 - P > 0.0)) { st |= 16; return false; }  // RSD_ST_DRAFT_EXHAUSTED
        return true;
    }

    // K-SEQ after all K children were rejected: beta = sum min{p, q / gamma}, then the residual
    // (q - min{p, q / gamma} (1 - (1 - beta)^K) / beta)+ with its tile sums ready for the draw
    __device__ void seq_finish(int K, VerifySmem& sm, bool& saw_nan, int& st) {
        const float a = (float)(Sq / Sp), g = (float)(1.0 / gamma);
        const double overlap = weight_pass<T, ALIGNED, kSeqOverlap>(rowq, rowp, V, mq, mp, kq, kp, a, g, sm, saw_nan, nullptr, nullptr);
        const double beta = overlap / Sq;
        double miss = 1.0;   // (1 - beta)^K, K = the node's number of children
        for (int i = 0; i < K; ++i) miss *= 1.0 - beta;
        const double c = beta > 0.0 ? (1.0 - miss) / beta : (double)K;
        const double t = weight_pass<T, ALIGNED, kSeqResidual>(rowq, rowp, V, mq, mp, kq, kp, a, g, sm, saw_nan, nullptr, nullptr, (float)c);
        if (t > 0.0 && t < 1.7e308) {
            a_hi = a; a_lo = g; c_seq = (float)c;
            total = t;
            tiles_current = true;
            seq_residual = true;
        } else {
            st |= 4;  // RSD_ST_ZERO_RESIDUAL: draw from the target row itself
            tiles_current = false;
        }
    }

    // draw from the current residual
    __device__ int draw(double u, VerifySmem& sm, bool& saw_nan) {
        if (BASELINES && seq_residual)
            return inverse_cdf_pick<T, ALIGNED, kSeqResidual>(rowq, rowp, V, mq, mp, kq, kp, a_hi, a_lo, total, u, sm, c_seq);
        if (!with_draft || A == 0.0) {
            if (!tiles_current || with_draft) {
                float tq;
                total = weight_pass<T, ALIGNED, kTargetOnly>(rowq, rowq, V, mq, 0.0f, kq, kq, 0.0f, 0.0f, sm, saw_nan, &tq, nullptr);
            }
            return inverse_cdf_pick<T, ALIGNED, kTargetOnly>(rowq, rowq, V, mq, 0.0f, kq, kq, 0.0f, 0.0f, total, u, sm);
        }
        if (!tiles_current)
            total = weight_pass<T, ALIGNED, kResidual>(rowq, rowp, V, mq, mp, kq, kp, a_hi, a_lo, sm, saw_nan, nullptr, nullptr);
        return inverse_cdf_pick<T, ALIGNED, kResidual>(rowq, rowp, V, mq, mp, kq, kp, a_hi, a_lo, total, u, sm);
    }
};

// smallest node c > after with parent[c] == cur and a token in [0, V), or -1.  Trees of up to kMaxCachedNodes nodes
// sit in shared memory and every warp searches them by itself (no barrier); larger trees are searched in global
// memory by the whole block.
__device__ __forceinline__ int next_child(const int32_t* par, const int32_t* tok, int num_nodes, int V, int cur, int after, VerifySmem& sm) {
    if (num_nodes <= kMaxCachedNodes) {
        const int lane = threadIdx.x & 31;
        for (int c0 = after + 1; c0 < num_nodes; c0 += 32) {
            const int c = c0 + lane;
            const bool ok = c < num_nodes && sm.par[c] == cur && sm.tok[c] >= 0 && sm.tok[c] < V;
            const unsigned m = __ballot_sync(0xFFFFFFFFu, ok);
            if (m) return c0 + __ffs(m) - 1;
        }
        return -1;
    }
    int best = 0x7FFFFFFF;
    for (int c = after + 1 + (int)threadIdx.x; c < num_nodes; c += kVerifyThreads) {
        if (par[c] == cur && tok[c] >= 0 && tok[c] < V) { best = c; break; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xFFFFFFFFu, best, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm.red_i[threadIdx.x >> 5] = best;
    __syncthreads();
    int r = sm.red_i[0];
#pragma unroll
    for (int w = 1; w < kVerifyWarps; ++w) r = min(r, sm.red_i[w]);
    return r == 0x7FFFFFFF ? -1 : r;
}

template <typename T, bool ALIGNED, bool BASELINES>
__global__ void __launch_bounds__(kVerifyThreads, sizeof(T) == 2 ? RSD_VERIFY_MIN_BLOCKS : RSD_VERIFY_MIN_BLOCKS_F32)
verify_tree_kernel(const VerifyArgs a) {
    __shared__ VerifySmem sm;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int32_t* par = a.parent + (a.shared_topology ? 0 : (int64_t)b * a.num_nodes);
    const int32_t* tok = a.token + (int64_t)b * a.num_nodes;
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    bool saw_nan = false;
    int st = 0;
    if (tid == 0) sm.nan_flag = 0;
    for (int i = tid; i < a.L; i += kVerifyThreads) {
        a.accepted_node[(int64_t)b * a.L + i] = -1;
        a.accepted_token[(int64_t)b * a.L + i] = -1;
    }
    if (a.dbg_theta)
        for (int n = tid; n < a.num_nodes; n += kVerifyThreads) a.dbg_theta[(int64_t)b * a.num_nodes + n] = __int_as_float(0x7FC00000);
    const bool cached = a.num_nodes <= kMaxCachedNodes;
    if (cached)
        for (int n = tid; n < a.num_nodes; n += kVerifyThreads) { sm.par[n] = par[n]; sm.tok[n] = tok[n]; }
    __syncthreads();

    NodeChain<T, ALIGNED, BASELINES> chain;
    chain.rule = BASELINES ? a.rule : 0;
    chain.gamma = (double)a.gamma;
    const int rule = chain.rule;
    int cur = 0, len = 0, reason;
    for (;;) {
        int c = next_child(par, tok, a.num_nodes, a.V, cur, 0, sm);
        if (c < 0 || len >= a.L) {
            reason = (len >= a.L) ? 2 : 1;  // RSD_STOP_LEAF : RSD_STOP_NO_CHILDREN
            chain.open_target_only(row_ptr<T>(a.target, b, cur), a.V, kLog2e * a.target.inv_temp, sm, saw_nan);
            break;
        }
        const char* rowq = row_ptr<T>(a.target, b, cur);
        const char* rowp = row_ptr<T>(a.draft, b, cur);
        chain.open_both(rowq, rowp, a.V, kLog2e * a.target.inv_temp, kLog2e * a.draft.inv_temp, sm, saw_nan);
        int accepted = -1, j = 0;
        while (c >= 0) {
            const int x = cached ? sm.tok[c] : tok[c];
            const float lq = RowIO<T>::scalar(rowq, x), lp = RowIO<T>::scalar(rowp, x);
            const double theta = chain.threshold(lq, lp, st);
            const uint4 rw = rng_draw(key, (uint32_t)cur, kTagAccept, (uint32_t)j);
            const double U = (double)(rw.x >> 8) * (1.0 / 16777216.0);
            if (a.dbg_theta && tid == 0) a.dbg_theta[(int64_t)b * a.num_nodes + c] = (float)theta;
            if (U < theta) { accepted = c; break; }
            ++j;
            if (!(BASELINES && rule == 2) && !chain.reject(x, lq, lp, sm, saw_nan, st)) break;
            c = next_child(par, tok, a.num_nodes, a.V, cur, c, sm);
        }
        if (accepted < 0) {  // RSD_STOP_ALL_REJECTED
            if (BASELINES && rule == 2) chain.seq_finish(j, sm, saw_nan, st);
            reason = 0;
            break;
        }
        if (tid == 0) {
            a.accepted_node[(int64_t)b * a.L + len] = accepted;
            a.accepted_token[(int64_t)b * a.L + len] = cached ? sm.tok[accepted] : tok[accepted];
        }
        ++len;
        cur = accepted;
    }
    const uint4 rw = rng_draw(key, (uint32_t)cur, kTagResample, 0u);
    const double u = ((double)rw.x + 0.5) * (1.0 / 4294967296.0);
    const int last = chain.draw(u, sm, saw_nan);
    if (saw_nan) sm.nan_flag = 1;
    __syncthreads();
    if (tid == 0) {
        a.accepted_len[b] = len;
        a.last_token[b] = last;
        a.stop_reason[b] = reason;
        a.status[b] = st | (sm.nan_flag ? 1 : 0);
    }
}

template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kVerifyThreads) resample_residual_kernel(const ResampleArgs a) {
    __shared__ VerifySmem sm;
    const int b = blockIdx.x, tid = threadIdx.x;
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    bool saw_nan = false;
    int st = 0;
    if (tid == 0) sm.nan_flag = 0;
    __syncthreads();
    int n_rej = 0;
    if (a.rejected)
        for (int i = 0; i < a.max_k; ++i) { const int x = a.rejected[(int64_t)b * a.max_k + i]; n_rej += (x >= 0 && x < a.V) ? 1 : 0; }
    NodeChain<T, ALIGNED> chain;
    chain.rule = 0;
    chain.gamma = 1.0;
    const char* rowq = row_ptr<T>(a.target, b, 0);
    if (n_rej == 0) {
        chain.open_target_only(rowq, a.V, kLog2e * a.target.inv_temp, sm, saw_nan);
    } else {
        chain.open_both(rowq, row_ptr<T>(a.draft, b, 0), a.V, kLog2e * a.target.inv_temp, kLog2e * a.draft.inv_temp, sm, saw_nan);
        for (int i = 0; i < a.max_k; ++i) {
            const int x = a.rejected[(int64_t)b * a.max_k + i];
            if (x < 0 || x >= a.V) continue;
            if (!chain.reject(x, RowIO<T>::scalar(rowq, x), RowIO<T>::scalar(chain.rowp, x), sm, saw_nan, st)) break;
        }
    }
    const uint4 rw = rng_draw(key, (uint32_t)a.rng_node[b], kTagResample, 0u);
    const double u = ((double)rw.x + 0.5) * (1.0 / 4294967296.0);
    const int y = chain.draw(u, sm, saw_nan);
    if (a.out_residual) {
        // normalised weights, recomputed element by element
        const bool with_draft = chain.with_draft && chain.A != 0.0;
        const float cq = chain.mq * chain.kq, cp = chain.mp * chain.kp;
        const double inv = chain.total > 0.0 ? 1.0 / chain.total : 0.0;
        for (int x = tid; x < a.V; x += kVerifyThreads) {
            float lq = RowIO<T>::scalar(rowq, x);
            if (lq != lq) lq = kNegInf;
            float w = ex2_approx(fmaf(lq, chain.kq, -cq));
            if (with_draft) {
                float lp = RowIO<T>::scalar(chain.rowp, x);
                if (lp != lp) lp = kNegInf;
                const float ph = ex2_approx(fmaf(lp, chain.kp, -cp));
                w = residual_weight(w, ph, chain.a_hi, chain.a_lo);
                for (int i = 0; i < sm.n_removed; ++i)
                    if (sm.rem_x[i] == x) w = sm.rem_w[i];
            }
            a.out_residual[(int64_t)b * a.V + x] = (float)((double)w * inv);
        }
    }
    if (saw_nan) sm.nan_flag = 1;
    __syncthreads();
    if (tid == 0) {
        a.out_token[b] = y;
        a.status[b] = st | (sm.nan_flag ? 1 : 0);
    }
}

}  // namespace rsd
