// Recursive rejection sampling along the draft tree (Eqs. 1-4, Algorithm 1; Section 3.2.2, Algorithm 6) with the
// visited node's two rows held in shared memory.
//
// One block of 512 threads walks one sequence and has the SM to itself (its shared memory holds a whole target row
// and a whole draft row, so one block fits per SM and the hardware hands the next sequence to whichever SM finishes
// first).  When the walk reaches a node, one thread asks the copy engine for both rows in chunks of 4096 elements
// (cp.async.bulk, one mbarrier per chunk); the block computes both soft-max normalisers chunk by chunk as the
// chunks land, so the arithmetic of the first pass overlaps the transfer.  Every later pass over the node (one per
// rejected child, Eq. 2 in closed form as in rsd_verify.cuh, and the draw of the last token) reads shared memory
// only: a row is read from HBM exactly once per visit and never again through L2.
//
// Used for rows on 16-byte boundaries whose pair fits in shared memory (2 V sizeof(element) <= about 208 KB: bf16
// up to V = 53,248, fp32 up to V = 26,624), recursive rejection sampling with the inverse-CDF last draw; everything
// else takes the streaming kernels of rsd_verify_walk.inc.
#pragma once
#include "rsd_verify.cuh"

namespace rsd {
namespace walk_res {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kChunkElems = 4096;              // elements per bulk copy (8 KB of bf16, 16 KB of fp32): 8 tiles of 512
constexpr int kTileElems = 512;                // one warp-wide step: 16 elements per lane
constexpr int kMaxChunks = 16;                 // V <= 65,536
constexpr int kMaxTilesRes = kMaxChunks * (kChunkElems / kTileElems);
constexpr int kMaxRemovedRes = 64;             // rejected tokens remembered per node (to recognise a repeated sibling)
constexpr long long kWaitCycles = 1ll << 31;   // about a second: a copy that has not landed by then never will

struct ResSmem {
    unsigned long long full[kMaxChunks];       // one mbarrier per chunk pair
    double tile_sum[kMaxTilesRes];
    double red_d[2][kWarps];
    float red_f[2][kWarps];
    int par[kMaxCachedNodes], tok[kMaxCachedNodes];
    int rem_x[kMaxRemovedRes];
    int n_removed;
    int pick;
    int abort;                                 // a wait ran out: the walk is abandoned and reported
    int nan_flag;
};

// ---- mbarrier / bulk copy (this GPU's own memory; no cluster, no multicast) -------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
// global -> shared, `bytes` a multiple of 16, both addresses 16-byte aligned; completion counts on `bar`
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// Wait for phase `parity` of `bar`, at most about a second.  A wait that runs out sets sm.abort and returns: the
// caller goes on with whatever the slot holds and the walk is abandoned at the next block-wide decision point.
__device__ __forceinline__ void wait_full(ResSmem& sm, int chunk, uint32_t parity) {
    if (mbar_try_wait(&sm.full[chunk], parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(&sm.full[chunk], parity)) {
        if (clock64() - t0 > kWaitCycles) {
            sm.abort = 1;
            return;
        }
    }
}

// ---- a lane's 16 elements of a tile ------------------------------------------------------------------------------------
// A tile is 512 consecutive elements.  For the sums a lane takes the 16-byte pieces lane, lane + 32, ... of the tile
// (conflict-free 128-bit shared-memory loads); `first_elem` tells which elements those are.
template <typename T>
struct TileIO;
template <>
struct TileIO<__nv_bfloat16> {
    static constexpr int kBytes = 2;
    static constexpr int kPieces = 2;          // pieces per lane
    static constexpr int kPerPiece = 8;        // elements per piece
    __device__ static __forceinline__ void load(Packed<__nv_bfloat16>& pk, const unsigned char* tile, int lane) {
        pk.w[0] = *(const uint4*)(tile + 16 * lane);
        pk.w[1] = *(const uint4*)(tile + 512 + 16 * lane);
    }
    // consecutive layout (lane owns elements 16 lane .. 16 lane + 15): only the last draw's exact scan uses it
    __device__ static __forceinline__ void load_consecutive(Packed<__nv_bfloat16>& pk, const unsigned char* tile, int lane) {
        pk.w[0] = *(const uint4*)(tile + 32 * lane);
        pk.w[1] = *(const uint4*)(tile + 32 * lane + 16);
    }
};
template <>
struct TileIO<float> {
    static constexpr int kBytes = 4;
    static constexpr int kPieces = 4;
    static constexpr int kPerPiece = 4;
    __device__ static __forceinline__ void load(Packed<float>& pk, const unsigned char* tile, int lane) {
#pragma unroll
        for (int i = 0; i < 4; ++i) pk.w[i] = *(const uint4*)(tile + 512 * i + 16 * lane);
    }
    __device__ static __forceinline__ void load_consecutive(Packed<float>& pk, const unsigned char* tile, int lane) {
#pragma unroll
        for (int i = 0; i < 4; ++i) pk.w[i] = *(const uint4*)(tile + 64 * lane + 16 * i);
    }
};
// element index (within the tile) of slot j of a lane's 16 values in the piece-wise layout
template <typename T>
__device__ __forceinline__ int piecewise_elem(int lane, int j) {
    return (j / TileIO<T>::kPerPiece) * (32 * TileIO<T>::kPerPiece) + lane * TileIO<T>::kPerPiece + (j % TileIO<T>::kPerPiece);
}

// State of the walk at one node; all threads hold identical copies (the closed-form chain of rsd_verify.cuh).
struct NodeState {
    float mq, mp;       // reference values of the exponentials (raw units)
    float kq, kp;       // log2(e) / temperature
    double Sq, Sp;      // normalisers relative to the references
    double A, P, Z;     // chain state
    float a_hi, a_lo;   // A Sq / Sp as a two-float sum
    double total;       // sum of the weights of the last pass
    bool with_draft;
};

template <typename T>
struct Walker {
    ResSmem& sm;
    unsigned char* slots;      // [n_chunks][2][chunk bytes]: target chunk, then draft chunk
    float* gsum;               // [n_tiles * 32] per-lane sums of the last pass
    int V, n_chunks, n_tiles;
    uint32_t parity;           // phase of the full barriers for the node being worked on
    bool saw_nan;

    static constexpr int kChunkBytes = kChunkElems * TileIO<T>::kBytes;
    static constexpr int kTileBytes = kTileElems * TileIO<T>::kBytes;

    __device__ __forceinline__ const unsigned char* tile_ptr(int tile, int which) const {
        const int chunk = tile >> 3;
        return slots + ((size_t)chunk * 2 + which) * kChunkBytes + (size_t)(tile & 7) * kTileBytes;
    }
    // value x of the resident target (0) or draft (1) row
    __device__ __forceinline__ float elem(int which, int x) const {
        const unsigned char* p = slots + ((size_t)(x / kChunkElems) * 2 + which) * kChunkBytes +
                                 (size_t)(x % kChunkElems) * TileIO<T>::kBytes;
        if (sizeof(T) == 2) return __uint_as_float((uint32_t)(*(const uint16_t*)p) << 16);
        return *(const float*)p;
    }

    // Ask for the rows of a node: target always, draft unless target_only.  Called by one thread, after a block
    // barrier that follows every read of the previous node's rows.
    __device__ __forceinline__ void request(const char* rowq, const char* rowp, bool target_only) {
        const int row_bytes16 = (V * TileIO<T>::kBytes) & ~15;   // whole 16-byte units (a shorter tail is copied by hand)
        for (int c = 0; c < n_chunks; ++c) {
            const int off = c * kChunkBytes;
            int bytes = row_bytes16 - off;
            bytes = bytes > kChunkBytes ? kChunkBytes : bytes;
            if (bytes <= 0) {   // the last chunk holds only the hand-copied tail
                mbar_expect_tx(&sm.full[c], 0);
                continue;
            }
            mbar_expect_tx(&sm.full[c], target_only ? bytes : 2 * bytes);
            bulk_load(slots + (size_t)c * 2 * kChunkBytes, rowq + off, bytes, &sm.full[c]);
            if (!target_only) bulk_load(slots + ((size_t)c * 2 + 1) * kChunkBytes, rowp + off, bytes, &sm.full[c]);
        }
    }
    // The last V sizeof(T) mod 16 bytes of a row cannot go through the copy engine: plain loads and stores.
    __device__ __forceinline__ void copy_tail(const char* rowq, const char* rowp, bool target_only) {
        const int first = ((V * TileIO<T>::kBytes) & ~15) / TileIO<T>::kBytes;
        for (int x = first + (int)threadIdx.x; x < V; x += kThreads) {
            unsigned char* dq = slots + ((size_t)(x / kChunkElems) * 2) * kChunkBytes + (size_t)(x % kChunkElems) * TileIO<T>::kBytes;
            if (sizeof(T) == 2) {
                *(uint16_t*)dq = ((const uint16_t*)rowq)[x];
                if (!target_only) *(uint16_t*)(dq + kChunkBytes) = ((const uint16_t*)rowp)[x];
            } else {
                *(uint32_t*)dq = ((const uint32_t*)rowq)[x];
                if (!target_only) *(uint32_t*)(dq + kChunkBytes) = ((const uint32_t*)rowp)[x];
            }
        }
    }

    // a lane's 16 values of a tile, NaN -> -inf (reported), elements beyond V -> -inf; returns their maximum
    __device__ __forceinline__ float load_tile(int tile, int which, int lane, float (&v)[16]) {
        Packed<T> pk;
        TileIO<T>::load(pk, tile_ptr(tile, which), lane);
        if ((tile + 1) * kTileElems > V) {   // the row's last, partial tile: what lies beyond V is stale memory
            pk.unpack(v);
            float m = kNegInf;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (tile * kTileElems + piecewise_elem<T>(lane, j) >= V) v[j] = kNegInf;
                if (v[j] != v[j]) { v[j] = kNegInf; saw_nan = true; }
                m = fmaxf(m, v[j]);
            }
            return m;
        }
        return clean<T>(pk, v, saw_nan);
    }

    // block-wide sums of two doubles and maxima of two floats behind one pair of barriers (identical on all threads)
    __device__ __forceinline__ void reduce4(double& s0, double& s1, float& m0, float& m1) {
        s0 = warp_sum(s0);
        s1 = warp_sum(s1);
        m0 = warp_max(m0);
        m1 = warp_max(m1);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) {
            const int w = threadIdx.x >> 5;
            sm.red_d[0][w] = s0;
            sm.red_d[1][w] = s1;
            sm.red_f[0][w] = m0;
            sm.red_f[1][w] = m1;
        }
        __syncthreads();
        s0 = 0.0;
        s1 = 0.0;
        m0 = sm.red_f[0][0];
        m1 = sm.red_f[1][0];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            s0 += sm.red_d[0][w];
            s1 += sm.red_d[1][w];
            m0 = fmaxf(m0, sm.red_f[0][w]);
            m1 = fmaxf(m1, sm.red_f[1][w]);
        }
    }

    // First pass over a node whose rows are on their way: references from chunk 0, then both normalisers chunk by
    // chunk as the copies land.  target_only: the draft row is absent; weights exp(lt - m_q) go to gsum for the draw.
    __device__ __forceinline__ void first_pass(NodeState& st, bool target_only) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        float v[16];
        // references: maxima over chunk 0 (any value near the row maximum will do)
        float rq = kNegInf, rp = kNegInf;
        wait_full(sm, 0, parity);
        if (warp < 8 && warp < n_tiles) {
            rq = load_tile(warp, 0, lane, v);
            if (!target_only) rp = load_tile(warp, 1, lane, v);
        }
        double d0 = 0.0, d1 = 0.0;
        reduce4(d0, d1, rq, rp);
        st.mq = rq > kNegInf ? rq : 0.0f;                       // chunk 0 without a finite value: start from 0
        st.mp = (!target_only && rp > kNegInf) ? rp : 0.0f;
        for (int attempt = 0; attempt < 3; ++attempt) {
            const float cq = st.mq * st.kq, cp = st.mp * st.kp;
            double accq = 0.0, accp = 0.0;
            float tq = kNegInf, tp = kNegInf;
            int have = 0;   // chunks known to have landed
            for (int tile = warp; tile < n_tiles; tile += kWarps) {
                const int chunk = tile >> 3;
                for (; have <= chunk; ++have) wait_full(sm, have, parity);
                float q[16];
                tq = fmaxf(tq, load_tile(tile, 0, lane, q));
                exp16(q, st.kq, cq, q);
                const float sq = tree_sum16(q);
                accq += (double)sq;
                if (target_only) {
                    gsum[tile * 32 + lane] = sq;
                } else {
                    float p[16];
                    tp = fmaxf(tp, load_tile(tile, 1, lane, p));
                    exp16(p, st.kp, cp, p);
                    accp += (double)tree_sum16(p);
                }
            }
            for (; have < n_chunks; ++have) wait_full(sm, have, parity);   // every thread has seen every chunk land
            reduce4(accq, accp, tq, tp);
            st.Sq = accq;
            st.Sp = target_only ? 1.0 : accp;
            // a reference that lies far below (overflow) or far above (everything underflows) the maximum: once more
            const bool redo_q = (tq > kNegInf) && fabsf((tq - st.mq) * st.kq) > kRefSlack * kLog2e;
            const bool redo_p = !target_only && (tp > kNegInf) && fabsf((tp - st.mp) * st.kp) > kRefSlack * kLog2e;
            if (!redo_q && !redo_p) break;
            if (redo_q) st.mq = tq;
            if (redo_p) st.mp = tp;
        }
        st.total = st.Sq;
    }

    // One pass over the resident rows: weights (qh - a ph)+, per-lane sums to gsum, returns the total.
    __device__ __forceinline__ double residual_pass(const NodeState& st) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const float cq = st.mq * st.kq, cp = st.mp * st.kp;
        double acc = 0.0, none = 0.0;
        for (int tile = warp; tile < n_tiles; tile += kWarps) {
            float q[16], p[16], w[16];
            load_tile(tile, 0, lane, q);
            load_tile(tile, 1, lane, p);
            exp16(q, st.kq, cq, q);
            exp16(p, st.kp, cp, p);
            residual16(q, p, st.a_hi, st.a_lo, w);
            const float s = tree_sum16(w);
            gsum[tile * 32 + lane] = s;
            acc += (double)s;
        }
        float f0 = 0.0f, f1 = 0.0f;
        reduce4(acc, none, f0, f1);
        return acc;
    }

    // Inverse CDF over the weights of the last pass (per-lane sums in gsum): the smallest y whose running sum exceeds
    // u * total; if rounding leaves none, the largest y with positive weight; -1 if there is no weight at all.
    __device__ __forceinline__ int pick(const NodeState& st, bool residual, double u) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        __syncthreads();   // gsum is complete
        for (int t = warp; t < n_tiles; t += kWarps) {
            const double s = warp_sum((double)gsum[t * 32 + lane]);
            if (lane == 0) sm.tile_sum[t] = s;
        }
        __syncthreads();
        double total = 0.0;
        for (int t = 0; t < n_tiles; ++t) total += sm.tile_sum[t];
        if (!(total > 0.0) || total > 1.7e308) return -1;
        const double target = u * total;
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
        if (warp == 0) {
            // the tile's weights once more, in token order: lane owns elements 16 lane .. 16 lane + 15
            const float cq = st.mq * st.kq, cp = st.mp * st.kp;
            Packed<T> pq;
            TileIO<T>::load_consecutive(pq, tile_ptr(tile, 0), lane);
            float q[16], w[16];
            pq.unpack(q);
            const int x0 = tile * kTileElems + 16 * lane;
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (x0 + j >= V || q[j] != q[j]) q[j] = kNegInf;
            if (residual) {
                Packed<T> pp;
                TileIO<T>::load_consecutive(pp, tile_ptr(tile, 1), lane);
                float p[16];
                pp.unpack(p);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (x0 + j >= V || p[j] != p[j]) p[j] = kNegInf;
                exp16(q, st.kq, cq, q);
                exp16(p, st.kp, cp, p);
                residual16(q, p, st.a_hi, st.a_lo, w);
            } else {
                exp16(q, st.kq, cq, w);
            }
            double gs = 0.0;
#pragma unroll
            for (int j = 0; j < 16; ++j) gs += (double)w[j];
            double incl = gs;
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
                    if (w[j] > 0.0f) last_pos = x0 + j;
                    if (!last_mode && y < 0 && c > target) y = x0 + j;
                }
                sm.pick = (y >= 0) ? y : last_pos;
            }
        }
        __syncthreads();
        return sm.pick;
    }
};

struct ResidentLaunch {
    int n_chunks, n_tiles;
    size_t gsum_offset;    // bytes from the start of dynamic shared memory
    size_t dyn_bytes;
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 1) verify_tree_resident_kernel(const VerifyArgs a, const ResidentLaunch rl) {
    extern __shared__ __align__(128) unsigned char dyn[];
    __shared__ ResSmem sm;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int32_t* par = a.parent + (a.shared_topology ? 0 : (int64_t)b * a.num_nodes);
    const int32_t* tok = a.token + (int64_t)b * a.num_nodes;
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};

    Walker<T> wk = {sm, dyn, (float*)(dyn + rl.gsum_offset), a.V, rl.n_chunks, rl.n_tiles, 0u, false};
    if (tid == 0) {
        for (int c = 0; c < rl.n_chunks; ++c) mbar_init(&sm.full[c], 1);
        sm.abort = 0;
        sm.nan_flag = 0;
        sm.n_removed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < a.L; i += kThreads) {
        a.accepted_node[(int64_t)b * a.L + i] = -1;
        a.accepted_token[(int64_t)b * a.L + i] = -1;
    }
    if (a.dbg_theta)
        for (int n = tid; n < a.num_nodes; n += kThreads) a.dbg_theta[(int64_t)b * a.num_nodes + n] = __int_as_float(0x7FC00000);
    const bool cached = a.num_nodes <= kMaxCachedNodes;
    if (cached)
        for (int n = tid; n < a.num_nodes; n += kThreads) { sm.par[n] = par[n]; sm.tok[n] = tok[n]; }
    __syncthreads();

    // smallest node c > after with parent cur and a token in [0, V), or -1; every warp searches by itself (the shared
    // copy of the tree, or global memory for trees too large for it)
    auto find_child = [&](int cur_node, int after) -> int {
        const int lane = tid & 31;
        for (int c0 = after + 1; c0 < a.num_nodes; c0 += 32) {
            const int cc = c0 + lane;
            bool ok = false;
            if (cc < a.num_nodes) {
                const int p = cached ? sm.par[cc] : par[cc];
                const int t = cached ? sm.tok[cc] : tok[cc];
                ok = p == cur_node && t >= 0 && t < a.V;
            }
            const unsigned m = __ballot_sync(0xFFFFFFFFu, ok);
            if (m) return c0 + __ffs(m) - 1;
        }
        return -1;
    };
    const bool has_tail = ((a.V * (int)sizeof(T)) & 15) != 0;
    NodeState st;
    st.kq = kLog2e * a.target.inv_temp;
    st.kp = kLog2e * a.draft.inv_temp;
    int status = 0, cur = 0, len = 0, reason = 0, last = -1;
    uint32_t opened = 0;   // nodes whose rows were asked for so far: the phase of every chunk barrier
    bool requested = false;
    for (;;) {
        int c = find_child(cur, 0);
        const bool target_only = c < 0 || len >= a.L;
        const char* rowq = row_ptr<T>(a.target, b, cur);
        const char* rowp = target_only ? rowq : row_ptr<T>(a.draft, b, cur);
        __syncthreads();   // nobody reads the previous node's rows any more
        if (tid == 0) {
            wk.request(rowq, rowp, target_only);
            sm.n_removed = 0;
        }
        requested = true;
        wk.parity = opened & 1u;
        ++opened;
        if (has_tail) {
            wk.copy_tail(rowq, rowp, target_only);
            __syncthreads();
        }
        st.A = 0.0; st.P = 0.0; st.Z = 1.0; st.a_hi = st.a_lo = 0.0f; st.with_draft = !target_only;
        wk.first_pass(st, target_only);
        if (sm.abort) break;
        if (target_only) {
            reason = (len >= a.L) ? 2 : 1;  // RSD_STOP_LEAF : RSD_STOP_NO_CHILDREN
            break;
        }
        int accepted = -1, j = 0;
        bool tiles_current = false;
        while (c >= 0) {
            const int x = cached ? sm.tok[c] : tok[c];
            const float lq = wk.elem(0, x), lp = wk.elem(1, x);
            const float qh = (lq == lq) ? ex2_approx(fmaf(lq, st.kq, -st.mq * st.kq)) : 0.0f;
            const float ph = (lp == lp) ? ex2_approx(fmaf(lp, st.kp, -st.mp * st.kp)) : 0.0f;
            const double qx = (double)qh / st.Sq;
            double px = (double)ph / st.Sp;
            bool repeated = false;   // a sibling with the same token was rejected before: its draft mass is gone (Eq. 1)
            for (int i = 0; i < sm.n_removed; ++i) repeated |= sm.rem_x[i] == x;
            if (repeated) px = 0.0;
            const double r = fmax(qx - st.A * ((double)ph / st.Sp), 0.0);
            double theta;
            if (px > 0.0) theta = fmin(1.0, r * (1.0 - st.P) / (st.Z * px));
            else { status |= 8; theta = r > 0.0 ? 1.0 : 0.0; }   // RSD_ST_ZERO_DRAFT_PROB
            const uint4 rw = rng_draw(key, (uint32_t)cur, kTagAccept, (uint32_t)j);
            const double U = (double)(rw.x >> 8) * (1.0 / 16777216.0);
            if (a.dbg_theta && tid == 0) a.dbg_theta[(int64_t)b * a.num_nodes + c] = (float)theta;
            if (U < theta) { accepted = c; break; }
            ++j;
            // Eqs. 1-2 in closed form: A_{j+1} = A_j + Z_j / (1 - P_j), Z_{j+1} = sum (q - A_{j+1} p)+
            const double A_old = st.A;
            st.A = st.A + st.Z / (1.0 - st.P);
            {
                const double aa = st.A * st.Sq / st.Sp;
                st.a_hi = (float)aa;
                st.a_lo = (float)(aa - (double)st.a_hi);
            }
            const double zhat = wk.residual_pass(st);
            if (sm.abort) break;
            const double Z_new = zhat / st.Sq;
            if (Z_new > 0.0 && Z_new < 1.7e308) {
                st.Z = Z_new;
                st.total = zhat;
                tiles_current = true;
            } else {
                status |= 4;   // RSD_ST_ZERO_RESIDUAL: keep the previous residual
                st.A = A_old;
                const double aa = st.A * st.Sq / st.Sp;
                st.a_hi = (float)aa;
                st.a_lo = (float)(aa - (double)st.a_hi);
                tiles_current = false;
            }
            st.P += px;
            if (tid == 0 && !repeated && sm.n_removed < kMaxRemovedRes) sm.rem_x[sm.n_removed++] = x;
            __syncthreads();
            if (!(1.0 - st.P > 0.0)) { status |= 16; break; }   // RSD_ST_DRAFT_EXHAUSTED
            c = find_child(cur, c);   // next sibling
        }
        if (sm.abort) break;
        if (accepted < 0) {   // RSD_STOP_ALL_REJECTED: draw from the last residual
            reason = 0;
            if (st.A != 0.0 && !tiles_current) {   // the last pass was not kept: weights of the residual in force
                st.total = wk.residual_pass(st);
            }
            break;
        }
        if (tid == 0) {
            a.accepted_node[(int64_t)b * a.L + len] = accepted;
            a.accepted_token[(int64_t)b * a.L + len] = cached ? sm.tok[accepted] : tok[accepted];
        }
        ++len;
        cur = accepted;
    }
    if (!sm.abort) {
        const uint4 rw = rng_draw(key, (uint32_t)cur, kTagResample, 0u);
        const double u = ((double)rw.x + 0.5) * (1.0 / 4294967296.0);
        if (st.with_draft && st.A == 0.0) {
            // every child was turned away without a usable residual: the target row itself (weights exp(lt - m_q))
            NodeState plain = st;
            plain.a_hi = plain.a_lo = 0.0f;
            wk.residual_pass(plain);
            last = wk.pick(plain, false, u);
        } else {
            last = wk.pick(st, st.with_draft, u);
        }
    } else if (requested) {
        // a copy never completed: wait once more (bounded) for whatever is still in flight before the block's shared
        // memory is given back, then report
        for (int cch = 0; cch < rl.n_chunks; ++cch) wait_full(sm, cch, wk.parity);
        status |= 32;   // RSD_ST_TIMEOUT
    }
    if (wk.saw_nan) sm.nan_flag = 1;
    __syncthreads();
    if (tid == 0) {
        a.accepted_len[b] = len;
        a.last_token[b] = last;
        a.stop_reason[b] = reason;
        a.status[b] = status | (sm.nan_flag ? 1 : 0);
    }
}

}  // namespace walk_res
}  // namespace rsd
