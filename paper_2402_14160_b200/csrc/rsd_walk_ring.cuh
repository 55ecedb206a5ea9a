// Recursive rejection sampling along the draft tree (Eqs. 1-4, Algorithm 1; Section 3.2.2, Algorithm 6): the walk
// whose passes stream a node's rows through a ring of shared-memory slots filled by the copy engine.
//
// One block walks one sequence and reads only the rows of visited nodes.  The chain of residuals is carried in
// closed form (see rsd_verify.cuh), so every pass is a read-only sweep over the node's target and draft rows: the
// first pass gives both soft-max normalisers, each rejected child costs one more pass, the last token is drawn from
// the tile sums of the last pass.
//
// A block has eight working warps and one control warp.  The control warp alone walks the tree: it takes every
// decision (thresholds, acceptance tests, the chain's scalars, the last draw), tells the working warps which pass to
// run next through a command word in shared memory, and asks the copy engine for the rows in chunks of 8 KB per row
// (cp.async.bulk into a ring of four slots, one mbarrier pair per slot: "full" counts the bytes that landed, "empty"
// counts the working warps that are done with the slot).  A block thus keeps up to 64 KB in flight without holding
// a register for it, the scalar part of the walk is executed once instead of by every warp, and three blocks share an
// SM: while one walk waits for a decision or for its next node's rows, the other two keep the SM's special-function
// unit and its memory pipe busy.
// Chunk c of a row lives in slot c mod 4, and successive passes over one node run in opposite directions: a pass
// ends with the last four chunks it read in the ring, the next pass starts with exactly those (no copy, no wait) and
// fetches the others behind them, so half of a 32000-entry row pair is read from L2 again per rejection, not all.
// Whatever the next decision needs and does not depend on the running pass (the child's uniform, its row values,
// the scalars of Eq. 2) is prepared by the control warp while the pass runs.
// Every wait on an mbarrier is bounded (about a second); a wait that runs out abandons the walk with RSD_ST_TIMEOUT.
//
// Used for rows whose base and strides are multiples of 16 bytes, recursive rejection sampling with the inverse-CDF
// last draw; everything else takes the register-fed kernels of rsd_verify_walk.inc.
#pragma once
#include "rsd_verify.cuh"

namespace rsd {
namespace walk_ring {

constexpr int kWorkWarps = 8;
constexpr int kThreads = (kWorkWarps + 1) * 32;   // the last warp feeds the ring
constexpr int kSlots = 4;                         // power of two
constexpr int kRowChunkBytes = 8192;              // bytes of one row per slot (a slot holds a target and a draft chunk)
constexpr int kTileElems = 512;                   // one warp-wide step: 16 elements per lane
constexpr int kMaxRingChunks = 64;                // chunks per row the ring's bookkeeping covers (one bit each)
constexpr int kMaxRemovedRing = 64;               // rejected tokens remembered per node (to recognise a repeated sibling)
constexpr float kSumFloor = 8.673617379884035e-19f;   // 2^-60: a normaliser below this has lost its small terms to underflow
constexpr int kRingBytes = kSlots * 2 * kRowChunkBytes;

// What the working warps do next (written by the control warp, read after a block barrier).
struct PassCmd {
    int kind;            // kPassEnd, or a pass kind below
    int clean;           // 1: NaN inputs are turned into -inf (a NaN was seen in the node's rows)
    int store_tiles;     // 1: the pass leaves the sum of every 512-element tile in tile_sum
    int rest;            // kPassTarget only, 1: the row summed is the draft row (kq, cq are its), without sm.gone_tok
    float kq, kp;        // log2(e) / temperature of the target and draft rows
    float cq, cp;        // reference * k: exponentials are 2^(value * k - c)
    float a_hi, a_lo;    // coefficient of the residual pass, as a two-float sum
    int backward;        // 1: the pass takes the chunks from the last to the first
    unsigned long long parity;   // bit c: phase parity of slot c mod kSlots' "full" barrier that holds chunk c
};

struct RingSmem {
    unsigned long long full[kSlots], empty[kSlots];
    PassCmd cmd;
    float4 red[kWorkWarps];                       // per working warp: two sums, two maxima of its last pass
    double tile_sum[kMaxTiles];
    int par[kMaxCachedNodes], tok[kMaxCachedNodes];
    int nan_seen;                                 // a cleaning pass met a NaN
    int abort;                                    // a wait ran out: the walk is abandoned and reported
    // for the pass that sums what is left of the draft row: the tokens rejected at the node so far, and per working
    // warp the chunks in which its tile holds one of them
    int gone_tok[kMaxRemovedRing];
    int n_gone_tok;
    unsigned gone_chunks[kWorkWarps][2];
};

// Which lane and which of its 16 values hold element `o` (0..511) of a tile as load_pieces() deals them out.
template <typename T>
__device__ __forceinline__ void piece_of(int o, int& lane, int& j) {
    constexpr int kPer = 16 / (int)sizeof(T);     // elements per 16-byte piece
    const int piece = o / kPer;
    lane = piece & 31;
    j = (piece >> 5) * kPer + o % kPer;
}

// A lane's 16 values of a 512-element tile in shared memory: the 16-byte pieces lane, lane + 32, ... of the tile
// (conflict-free 128-bit loads).  Which elements a lane sums does not matter; the one place that needs token order
// (the last draw) reads its tile from global memory.
__device__ __forceinline__ void load_pieces(Packed<__nv_bfloat16>& pk, const unsigned char* tile, int lane) {
    pk.w[0] = *(const uint4*)(tile + 16 * lane);
    pk.w[1] = *(const uint4*)(tile + 512 + 16 * lane);
}
__device__ __forceinline__ void load_pieces(Packed<float>& pk, const unsigned char* tile, int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) pk.w[i] = *(const uint4*)(tile + 512 * i + 16 * lane);
}

__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max_nan(float v) {   // NaN if any lane holds one
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max_nan(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// unpack a loaded group; CLEAN: NaN -> -inf
template <typename T, bool CLEAN>
__device__ __forceinline__ void values16(const Packed<T>& pk, float (&v)[16]) {
    pk.unpack(v);
    if (CLEAN) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
            if (v[j] != v[j]) v[j] = kNegInf;
    }
}

enum { kPassEnd = -1, kPassFirst = 0, kPassTarget = 1, kPassResidual = 2 };

// State of the walk at one node (control warp only): the closed-form chain of rsd_verify.cuh.
struct NodeState {
    float mq, mp;       // reference values of the exponentials (raw units)
    float kq, kp;       // log2(e) / temperature
    double Sq, Sp;      // normalisers relative to the references
    double A, Z;        // chain state (1 - P is kept by the walk itself)
    float a_hi, a_lo;   // A Sq / Sp as a two-float sum
    bool with_draft;    // false: a node without children, only its target row is read
    bool has_nan;       // a NaN was seen in the node's rows: the passes clean their inputs
};

template <typename T>
struct Ring {
    RingSmem& sm;
    unsigned char* slots;      // [kSlots][2][kRowChunkBytes]: target chunk, then draft chunk
    int V, n_chunks, n_tiles;
    // control warp only (identical on its lanes): the state of the ring as bit sets, so that a pass is planned
    // without a loop
    unsigned long long resident;   // chunks of the current node that sit in their slots
    unsigned fill_par;             // bit s: parity of slot s' latest "full" phase (1 before the first copy)
    unsigned round_par;            // bit s: parity of slot s' latest "empty" phase (1 before the first use)
    unsigned round_used;           // bit s: the slot was given to the working warps at least once
    int backward;                  // direction of the next pass over the current node

    static constexpr int kElem = (int)sizeof(T);
    static constexpr int kChunkElems = kRowChunkBytes / kElem;
    static constexpr int kTPC = kChunkElems / kTileElems;   // tiles per chunk: 8 (2-byte elements) or 4
    static constexpr unsigned long long kEveryFourth = 0x1111111111111111ull;

    __device__ __forceinline__ void reset() {
        resident = 0ull;
        fill_par = (1u << kSlots) - 1u;
        round_par = (1u << kSlots) - 1u;
        round_used = 0u;
        backward = 0;
    }
    __device__ __forceinline__ void forget_node() {
        resident = 0ull;
        backward = 0;
    }

    // ---- control warp: which chunks of the coming pass must be copied (`missing`), its direction, and its parity word
    // (bit c: phase parity of the "full" barrier that will hold chunk c when the pass reaches it).  Chunk c lives in
    // slot c mod 4; the pass ends with its last four chunks in the ring. ----------------------------------------------------
    __device__ __forceinline__ void plan(int& dir, unsigned long long& parity, unsigned long long& missing) {
        static_assert(kSlots == 4, "the bit tricks below assume four slots");
        const unsigned long long all = n_chunks >= 64 ? ~0ull : (1ull << n_chunks) - 1ull;
        dir = backward;
        backward ^= 1;
        missing = all & ~resident;
        // number of copies into chunk c's slot up to and including chunk c, in pass order, modulo 2
        unsigned long long x = missing;
        if (dir) { x ^= x >> 4; x ^= x >> 8; x ^= x >> 16; x ^= x >> 32; }
        else { x ^= x << 4; x ^= x << 8; x ^= x << 16; x ^= x << 32; }
        parity = (x ^ ((unsigned long long)fill_par * kEveryFourth)) & all;
#pragma unroll
        for (int s = 0; s < kSlots; ++s) fill_par ^= (unsigned)(__popcll(missing & (kEveryFourth << s)) & 1) << s;
        resident = dir ? (all & 0xFull) : (all & ~(all >> 4));
    }

    // ---- control warp: ask for chunk c (the slot's previous use must be over).  All lanes call it together. -------------
    __device__ __forceinline__ void fetch(const char* rowq, const char* rowp, bool with_draft, int c, bool was_used, uint32_t wait_parity) {
        const int lane = threadIdx.x & 31;
        const int slot = c & (kSlots - 1);
        const int row_bytes = V * kElem, row_bytes16 = row_bytes & ~15;
        if (was_used) wait_bar(&sm.empty[slot], wait_parity, &sm.abort);
        const int off = c * kRowChunkBytes;
        int bytes = row_bytes16 - off;
        bytes = bytes > kRowChunkBytes ? kRowChunkBytes : (bytes < 0 ? 0 : bytes);
        unsigned char* dq = slots + (size_t)slot * 2 * kRowChunkBytes;
        unsigned char* dp = dq + kRowChunkBytes;
        if (c == n_chunks - 1) {
            // End of the row: the last V sizeof(T) mod 16 bytes cannot go through the copy engine and are copied by
            // hand; what follows, up to the end of the tile, is filled with -inf so that the working warps never have
            // to look at an index.  Published by the barrier arrival below.
            const int first = row_bytes16 / kElem;                        // first element copied by hand
            const int tile_end = ((V + kTileElems - 1) / kTileElems) * kTileElems;
            for (int x = first + lane; x < tile_end; x += 32) {
                const int at = (x - c * kChunkElems) * kElem;
                if (kElem == 2) {
                    *(uint16_t*)(dq + at) = x < V ? ((const uint16_t*)rowq)[x] : (uint16_t)0xFF80u;
                    if (with_draft) *(uint16_t*)(dp + at) = x < V ? ((const uint16_t*)rowp)[x] : (uint16_t)0xFF80u;
                } else {
                    *(uint32_t*)(dq + at) = x < V ? ((const uint32_t*)rowq)[x] : 0xFF800000u;
                    if (with_draft) *(uint32_t*)(dp + at) = x < V ? ((const uint32_t*)rowp)[x] : 0xFF800000u;
                }
            }
            __syncwarp();
        }
        if (lane == 0) {
            mbar_expect_tx(&sm.full[slot], with_draft ? 2u * (uint32_t)bytes : (uint32_t)bytes);
            if (bytes > 0) {
                bulk_load(dq, rowq + off, (uint32_t)bytes, &sm.full[slot]);
                if (with_draft) bulk_load(dp, rowp + off, (uint32_t)bytes, &sm.full[slot]);
            }
        }
    }

    // ---- control warp: the first `early` (<= kSlots) steps of the pass at once, lane i taking step i: their slots are
    // distinct, and what they wait for, if anything, are uses of earlier passes, which are over.  The row's last chunk
    // needs the whole warp (hand-copied tail) and goes first if it is among them. -------------------------------------------
    __device__ __forceinline__ void produce_early(const char* rowq, const char* rowp, bool with_draft, int dir,
                                                  unsigned long long missing, int early) {
        const int lane = threadIdx.x & 31;
        const int row_bytes16 = (V * kElem) & ~15;
        const int i_last = dir ? 0 : n_chunks - 1;                 // step of chunk n_chunks - 1
        if (i_last < early && ((missing >> (n_chunks - 1)) & 1ull)) {
            const int slot = (n_chunks - 1) & (kSlots - 1);
            fetch(rowq, rowp, with_draft, n_chunks - 1, (round_used >> slot) & 1u, (round_par >> slot) & 1u);
        }
        if (lane < early && lane != i_last) {
            const int c = dir ? n_chunks - 1 - lane : lane;
            const int slot = c & (kSlots - 1);
            if ((missing >> c) & 1ull) {
                if ((round_used >> slot) & 1u) wait_bar(&sm.empty[slot], (round_par >> slot) & 1u, &sm.abort);
                const int off = c * kRowChunkBytes;                // (not the last chunk: a whole chunk)
                const uint32_t bytes = (uint32_t)(row_bytes16 - off > kRowChunkBytes ? kRowChunkBytes : row_bytes16 - off);
                unsigned char* dq = slots + (size_t)slot * 2 * kRowChunkBytes;
                mbar_expect_tx(&sm.full[slot], with_draft ? 2u * bytes : bytes);
                bulk_load(dq, rowq + off, bytes, &sm.full[slot]);
                if (with_draft) bulk_load(dq + kRowChunkBytes, rowp + off, bytes, &sm.full[slot]);
            }
        }
        __syncwarp();
        for (int i = 0; i < early; ++i) {                          // each of these steps is its slot's next round
            const int slot = (dir ? n_chunks - 1 - i : i) & (kSlots - 1);
            round_used |= 1u << slot;
            round_par ^= 1u << slot;
        }
    }

    // ---- control warp: steps [i_begin, i_end) of the pass, in order ------------------------------------------------------------
    __device__ __forceinline__ void produce(const char* rowq, const char* rowp, bool with_draft, int dir, unsigned long long missing,
                                            int i_begin, int i_end) {
        for (int i = i_begin; i < i_end; ++i) {
            const int c = dir ? n_chunks - 1 - i : i;
            const int slot = c & (kSlots - 1);
            const bool was_used = (round_used >> slot) & 1u;
            const uint32_t wait_parity = (round_par >> slot) & 1u;
            round_used |= 1u << slot;                              // this step is the slot's next round
            round_par ^= 1u << slot;
            if ((missing >> c) & 1ull) fetch(rowq, rowp, with_draft, c, was_used, wait_parity);
        }
    }

    // ---- working warps: every chunk of the pass in its order; fn(tile, q tile, p tile) for this warp's tile of it -------
    template <typename F>
    __device__ __forceinline__ void consume(const PassCmd& cmd, F&& fn) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        for (int i = 0; i < n_chunks; ++i) {
            const int c = cmd.backward ? n_chunks - 1 - i : i;
            const int slot = c & (kSlots - 1);
            const int t = (warp - c * kTPC) & (kWorkWarps - 1);   // tile of the chunk with (c kTPC + t) mod 8 == warp
            const int tile = c * kTPC + t;
            // every warp waits for every chunk, with or without a tile in it: a warp can then never be a whole turn
            // of the ring ahead of another, so an "empty" phase counts each warp exactly once
            wait_bar(&sm.full[slot], (uint32_t)(cmd.parity >> c) & 1u, &sm.abort);
            if (t < kTPC && tile < n_tiles) {
                const unsigned char* q = slots + (size_t)slot * 2 * kRowChunkBytes + (size_t)t * kTileElems * kElem;
                fn(tile, q, q + kRowChunkBytes);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[slot]);
        }
    }

    // One pass of a working warp over the node's rows; leaves the warp's sums and maxima in sm.red[warp].
    //   kPassFirst     both rows: sums of exp(lt k_q - c_q) and exp(ld k_p - c_p)
    //   kPassTarget    target row only: sum of the weights exp(lt k_q - c_q)
    //   kPassResidual  both rows: sum of the weights (qh - a ph)+
    //                  (cmd.rest: of the draft row instead, without the tokens listed in sm.gone_tok: the same code,
    //                  so that this rare pass adds nothing to the kernel's size)
    // CLEAN passes turn NaN into -inf (reported through sm.nan_seen) and also return the rows' maxima; the plain ones
    // carry no code for either.  STORE_TILES: the sum of every tile goes to sm.tile_sum.
    template <int KIND, bool CLEAN, bool STORE_TILES>
    __device__ __forceinline__ void work(const PassCmd& cmd) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        float s0 = 0.0f, s1 = 0.0f, m0 = kNegInf, m1 = kNegInf;
        bool saw_nan = false;
        // cmd.rest, bit c: this warp's tile of chunk c holds one of the listed tokens
        const bool rest = KIND == kPassTarget && cmd.rest != 0;
        const unsigned long long gone_tiles_of_warp =
            rest ? ((unsigned long long)sm.gone_chunks[warp][1] << 32) | sm.gone_chunks[warp][0] : 0ull;
        consume(cmd, [&](int tile, const unsigned char* qt, const unsigned char* pt) {
            Packed<T> pq;
            load_pieces(pq, rest ? pt : qt, lane);
            float q[16];
            if (CLEAN) m0 = fmaxf(m0, clean<T>(pq, q, saw_nan));
            else pq.unpack(q);
            exp16(q, cmd.kq, cmd.cq, q);
            float s;
            if (KIND == kPassTarget) {
                if (rest && ((gone_tiles_of_warp >> (tile / kTPC)) & 1ull)) {
                    for (int i = 0; i < sm.n_gone_tok; ++i) {
                        const int o = sm.gone_tok[i] - tile * kTileElems;
                        if (o < 0 || o >= kTileElems) continue;
                        int l_, j_;
                        piece_of<T>(o, l_, j_);
                        if (l_ == lane) {
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj)
                                if (jj == j_) q[jj] = 0.0f;
                        }
                    }
                }
                s = tree_sum16(q);
                s0 += s;
            } else {
                Packed<T> pp;
                load_pieces(pp, pt, lane);
                float p[16];
                if (CLEAN) m1 = fmaxf(m1, clean<T>(pp, p, saw_nan));
                else pp.unpack(p);
                exp16(p, cmd.kp, cmd.cp, p);
                if (KIND == kPassFirst) {
                    s0 += tree_sum16(q);
                    s1 += tree_sum16(p);
                    s = 0.0f;
                } else {
                    float w[16];
                    residual16(q, p, cmd.a_hi, cmd.a_lo, w);
                    s = tree_sum16(w);
                    s0 += s;
                }
            }
            if (STORE_TILES) {
                const float ts = warp_sum_f32(s);
                if (lane == 0) sm.tile_sum[tile] = (double)ts;
            }
        });
        s0 = warp_sum_f32(s0);
        s1 = warp_sum_f32(s1);
        if (CLEAN) {
            m0 = warp_max(m0);
            m1 = warp_max(m1);
            if (saw_nan) sm.nan_seen = 1;
        }
        if (lane == 0) sm.red[warp] = make_float4(s0, s1, m0, m1);
    }
};

// weights of 16 consecutive tokens of group g, read from global memory (the last draw's exact scan)
template <typename T>
__device__ __forceinline__ void group_weights(const char* rowq, const char* rowp, int g, int V, const NodeState& st, bool residual,
                                              float (&w)[16]) {
    const float cq = st.mq * st.kq, cp = st.mp * st.kp;
    float q[16];
    bool dummy = false;
    load_clean<T, true>(rowq, g, V, q, dummy);
    if (residual) {
        float p[16];
        load_clean<T, true>(rowp, g, V, p, dummy);
        exp16(q, st.kq, cq, q);
        exp16(p, st.kp, cp, p);
        residual16(q, p, st.a_hi, st.a_lo, w);
    } else {
        exp16(q, st.kq, cq, w);
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 3) verify_tree_ring_kernel(const VerifyArgs a) {
    extern __shared__ __align__(128) unsigned char ring_mem[];
    __shared__ RingSmem sm;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t* par = a.parent + (a.shared_topology ? 0 : (int64_t)b * a.num_nodes);
    const int32_t* tok = a.token + (int64_t)b * a.num_nodes;
    constexpr int kChunkElems = Ring<T>::kChunkElems;

    Ring<T> ring = {sm, ring_mem, a.V, (a.V + kChunkElems - 1) / kChunkElems, (a.V + kTileElems - 1) / kTileElems};
    ring.reset();
    if (tid == 0) {
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kWorkWarps);
        }
        sm.abort = 0;
        sm.nan_seen = 0;
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

    // ================================ working warps: run the passes they are told to ===================================
    if (warp < kWorkWarps) {
        for (;;) {
            __syncthreads();   // the command is in place
            const PassCmd cmd = sm.cmd;
            if (cmd.kind == kPassEnd) return;
            if (cmd.kind == kPassFirst) {
                if (cmd.clean) ring.template work<kPassFirst, true, false>(cmd);
                else ring.template work<kPassFirst, false, false>(cmd);
            } else if (cmd.kind == kPassTarget) {
                if (cmd.clean) ring.template work<kPassTarget, true, true>(cmd);
                else ring.template work<kPassTarget, false, true>(cmd);
            } else {
                if (cmd.clean) {
                    if (cmd.store_tiles) ring.template work<kPassResidual, true, true>(cmd);
                    else ring.template work<kPassResidual, true, false>(cmd);
                } else {
                    if (cmd.store_tiles) ring.template work<kPassResidual, false, true>(cmd);
                    else ring.template work<kPassResidual, false, false>(cmd);
                }
            }
            __syncthreads();   // the warps' sums are in place
        }
    }

    // ================================ control warp: the walk itself =======================================================
    const RngKey key = {a.seed_lo, a.seed_hi, a.step, a.seq_base + (uint32_t)b};
    // smallest node c > after with parent cur_node and a token in [0, V), or -1
    auto find_child = [&](int cur_node, int after) -> int {
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

    NodeState st;
    st.kq = kLog2e * a.target.inv_temp;
    st.kp = kLog2e * a.draft.inv_temp;
    const char* rowq = nullptr;
    const char* rowp = nullptr;
    // One pass: plan which chunks must be copied, publish the command, ask for the rows, collect the working warps'
    // results.  The first kSlots steps are taken before the command is published: what they wait for, if anything, are
    // slot uses of earlier passes, which every working warp finished before it reported its sums; so the copies travel
    // while the working warps wake up.  `meanwhile` runs on the control warp while the pass is under way.
    auto run_pass = [&](int kind, bool store_tiles, double& S0, double& S1, float& M0, float& M1, auto&& meanwhile, auto&& early, bool rest = false) {
        const bool with_draft = kind != kPassTarget || rest;   // (the rest pass moves both rows like a residual pass: the ring stays as it is)
        int dir;
        unsigned long long parity, missing;
        ring.plan(dir, parity, missing);
        if (lane == 0) {
            PassCmd cmd;
            cmd.kind = kind; cmd.clean = st.has_nan ? 1 : 0; cmd.store_tiles = store_tiles ? 1 : 0;
            cmd.rest = rest ? 1 : 0;
            cmd.kq = rest ? st.kp : st.kq; cmd.kp = st.kp; cmd.cq = rest ? st.mp * st.kp : st.mq * st.kq; cmd.cp = st.mp * st.kp;
            cmd.a_hi = st.a_hi; cmd.a_lo = st.a_lo;
            cmd.backward = dir; cmd.parity = parity;
            sm.cmd = cmd;
        }
        const int n_early = ring.n_chunks < kSlots ? ring.n_chunks : kSlots;
        ring.produce_early(rowq, rowp, with_draft, dir, missing, n_early);
        early();           // (what else the working warps need: written while the first copies travel)
        __syncthreads();   // the command is in place
        ring.produce(rowq, rowp, with_draft, dir, missing, n_early, ring.n_chunks);
        meanwhile();
        __syncthreads();   // the warps' sums are in place
        static_assert(kWorkWarps == 8, "fixed summation tree over eight warps");
        float4 r[kWorkWarps];
#pragma unroll
        for (int w = 0; w < kWorkWarps; ++w) r[w] = sm.red[w];
        S0 = (((double)r[0].x + (double)r[1].x) + ((double)r[2].x + (double)r[3].x)) +
             (((double)r[4].x + (double)r[5].x) + ((double)r[6].x + (double)r[7].x));
        S1 = (((double)r[0].y + (double)r[1].y) + ((double)r[2].y + (double)r[3].y)) +
             (((double)r[4].y + (double)r[5].y) + ((double)r[6].y + (double)r[7].y));
        M0 = fmaxf(fmaxf(fmaxf(r[0].z, r[1].z), fmaxf(r[2].z, r[3].z)), fmaxf(fmaxf(r[4].z, r[5].z), fmaxf(r[6].z, r[7].z)));
        M1 = fmaxf(fmaxf(fmaxf(r[0].w, r[1].w), fmaxf(r[2].w, r[3].w)), fmaxf(fmaxf(r[4].w, r[5].w), fmaxf(r[6].w, r[7].w)));
    };
    auto nothing = [] {};

    int status = 0, cur = 0, len = 0, reason = 0, last = -1;
    bool tiles_valid = false;   // sm.tile_sum holds the tile sums of the distribution the last token is drawn from
    bool aborted = false;
    for (;;) {
        int c = find_child(cur, 0);
        st.with_draft = !(c < 0 || len >= a.L);
        rowq = row_ptr<T>(a.target, b, cur);
        rowp = st.with_draft ? row_ptr<T>(a.draft, b, cur) : rowq;
        st.A = 0.0; st.Z = 1.0; st.a_hi = st.a_lo = 0.0f; st.has_nan = false;
        st.mq = 0.0f; st.mp = 0.0f; st.Sp = 1.0;
        tiles_valid = false;
        ring.forget_node();
        // The node's first 32 children in stored order, one per lane: node, token and the two row values (the
        // thresholds need them right after the first pass); the loads are in flight while the rows stream.
        int child_node = -1, child_x = -1;
        float child_lq = 0.0f, child_lp = 0.0f;
        if (st.with_draft) {
            int found = 0;
            for (int c0 = 1; c0 < a.num_nodes && found < 32; c0 += 32) {
                const int cc = c0 + lane;
                bool ok = false;
                if (cc < a.num_nodes) {
                    const int p = cached ? sm.par[cc] : par[cc];
                    const int t = cached ? sm.tok[cc] : tok[cc];
                    ok = p == cur && t >= 0 && t < a.V;
                }
                const unsigned m = __ballot_sync(0xFFFFFFFFu, ok);
                const int k = __popc(m);
                if (lane >= found && lane < found + k) child_node = c0 + (int)__fns(m, 0, lane - found + 1);   // its (lane - found)-th
                found += k;
            }
            if (child_node >= 0) {
                child_x = cached ? sm.tok[child_node] : tok[child_node];
                child_lq = RowIO<T>::scalar(rowq, child_x);
                child_lp = RowIO<T>::scalar(rowp, child_x);
            }
        }
        // First pass.  Exponentials are taken relative to a reference, 0 to begin with: the plain pass has no code for
        // maxima or NaN.  If its sums are not finite, or so small that underflow may have eaten them (logits beyond
        // about +-40 / temperature), a cleaning pass finds the rows' maxima and the pass is run again relative to them.
        {
            double S0, S1;
            float M0, M1;
            const int kind = st.with_draft ? kPassFirst : kPassTarget;
            for (int attempt = 0; attempt < 3; ++attempt) {
                run_pass(kind, !st.with_draft, S0, S1, M0, M1, nothing, nothing);
                if (sm.abort) { aborted = true; break; }
                if (!st.with_draft) S1 = 1.0;
                const bool good = S0 >= (double)kSumFloor && S0 < 1e300 && S1 >= (double)kSumFloor && S1 < 1e300;
                if (attempt == 0) {
                    if (good) break;
                    st.has_nan = true;                 // next: the cleaning pass, which also returns the maxima
                    if (lane == 0) sm.nan_seen = 0;    // (published with the next command)
                } else if (attempt == 1) {
                    if (sm.nan_seen) status |= 1;      // RSD_ST_NAN_INPUT: the node's passes keep cleaning
                    else st.has_nan = false;
                    if (good) break;                   // only a NaN was in the way
                    if (M0 > kNegInf) st.mq = M0;      // under- or overflow: once more, relative to the maxima
                    if (st.with_draft && M1 > kNegInf) st.mp = M1;
                }
            }
            if (aborted) break;
            st.Sq = S0;
            st.Sp = S1;
            tiles_valid = !st.with_draft;
        }
        if (!st.with_draft) {
            reason = (len >= a.L) ? 2 : 1;  // RSD_STOP_LEAF : RSD_STOP_NO_CHILDREN
            break;
        }
        const double inv_Sq = 1.0 / st.Sq, inv_Sp = 1.0 / st.Sp, ratio = st.Sq * inv_Sp;
        int rem_x[4];            // rejected tokens of this node, lanes hold them four at a time (lane i: entries 4 i ..)
        int n_removed = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) rem_x[i] = -1;
        // What the test of child j needs and no pass changes: its token, its probabilities under the node's two rows,
        // whether an earlier sibling with the same token was rejected, and its uniform.
        int j = 0, x = -1;
        float qh_x = 0.0f, ph_x = 0.0f, qp = 0.0f;          // weights of x under the two rows; q(x) / p(x)
        uint32_t U24 = 0u;                                 // the uniform, as 24 bits
        bool repeated = false, p_none = false;             // p_none: the draft row gives the token no mass (-inf or NaN)
        // log2(S_p / S_q) for the exponent of q(x)/p(x), by the fast logarithm (absolute error 2^-22)
        const float lg_inv_ratio = lg2_approx((float)fmin(fmax(st.Sp * inv_Sq, 1e-37), 1e37));
        auto prepare = [&](int child) {
            float lq, lp;
            if (j < 32) {
                x = __shfl_sync(0xFFFFFFFFu, child_x, j);
                lq = __shfl_sync(0xFFFFFFFFu, child_lq, j);
                lp = __shfl_sync(0xFFFFFFFFu, child_lp, j);
            } else {
                x = cached ? sm.tok[child] : tok[child];
                lq = RowIO<T>::scalar(rowq, x);
                lp = RowIO<T>::scalar(rowp, x);
            }
            const float eq = fmaf(lq, st.kq, -st.mq * st.kq), ep = fmaf(lp, st.kp, -st.mp * st.kp);
            qh_x = (lq == lq) ? ex2_approx(eq) : 0.0f;
            ph_x = (lp == lp) ? ex2_approx(ep) : 0.0f;
            // The test needs q(x) / p(x) only: taken from the difference of the exponents it survives probabilities
            // below the fp32 range (children drafted from the far tail of a peaked row), where q(x) and p(x) are both 0.
            p_none = !(lp == lp) || !(lp > kNegInf);
            qp = (lq == lq && !p_none) ? ex2_approx((eq - ep) + lg_inv_ratio) : 0.0f;
            bool mine = false;
#pragma unroll
            for (int i = 0; i < 4; ++i) mine |= rem_x[i] == x;
            repeated = __any_sync(0xFFFFFFFFu, mine);   // its draft mass is gone (Eq. 1)
            const uint4 rw = rng_draw(key, (uint32_t)cur, kTagAccept, (uint32_t)j);
            U24 = rw.x >> 8;
        };
        prepare(c);
        // 1 - P of the closed form, the draft mass still in play.  It is carried by subtraction while that is accurate:
        // every p(x) has the relative error of a fast exponential and of the fp32 sums behind S_p, and with a peaked
        // draft the rejected tokens can hold all but 1e-7 of the mass.  Once the error bound passes 2e-6 of what is left,
        // a pass sums the draft row anew without the rejected tokens.
        double one_mP = 1.0, one_mP_err = 0.0;
        double inv_1mP = 1.0;    // 1 / (1 - P)
        auto publish_gone = [&] {   // the rejected tokens for that pass (lane i holds entries 4 i .. 4 i + 3)
            if (lane < 2 * kWorkWarps) (&sm.gone_chunks[0][0])[lane] = 0u;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (rem_x[i] >= 0) {
                    sm.gone_tok[4 * lane + i] = rem_x[i];
                    const int tile = rem_x[i] / kTileElems, chunk = tile / Ring<T>::kTPC;   // tile t belongs to warp t mod 8
                    atomicOr(&sm.gone_chunks[tile & (kWorkWarps - 1)][chunk >> 5], 1u << (chunk & 31));
                }
            }
            if (lane == 0) sm.n_gone_tok = n_removed;
        };
        int accepted = -1;
        while (c >= 0) {
            // Eq. 3 in closed form: accept iff U < min(1, r (1 - P) / (Z p(x))), r = (q(x) - A p(x))+, tested without
            // the division; a child the draft cannot produce any more is taken iff it has residual mass
            const bool no_draft = repeated || p_none;
            const double px_row = (double)ph_x * inv_Sp, U = (double)U24 * (1.0 / 16777216.0);
            const double px = no_draft ? 0.0 : px_row;
            bool take;
            double g;   // the threshold times Z; with no draft mass: 1 or 0 times Z
            if (!no_draft) {   // U < min(1, (q/p - A)+ (1 - P) / Z)
                g = fmax((double)qp - st.A, 0.0) * one_mP;
                take = U * st.Z < g;
            } else {           // RSD_ST_ZERO_DRAFT_PROB
                const double r = fmax((double)qh_x * inv_Sq - st.A * px_row, 0.0);
                status |= 8;
                take = r > 0.0;
                g = take ? st.Z : 0.0;
            }
            if (a.dbg_theta && lane == 0) a.dbg_theta[(int64_t)b * a.num_nodes + c] = (float)fmin(1.0, g / st.Z);
            if (take) { accepted = c; break; }
            // rejected.  Eqs. 1-2 in closed form: A_{j+1} = A_j + Z_j / (1 - P_j), Z_{j+1} = sum (q - A_{j+1} p)+
            ++j;
            const int next = j < 32 ? __shfl_sync(0xFFFFFFFFu, child_node, j) : find_child(cur, c);
            const double A_old = st.A;
            st.A = fma(st.Z, inv_1mP, st.A);
            {
                const double aa = st.A * ratio;
                st.a_hi = (float)aa;
                st.a_lo = (float)(aa - (double)st.a_hi);
            }
            double one_mP_new = one_mP - px, err_new = one_mP_err + 4e-7 * px;   // (px = 0 for a repeated token)
            if (!repeated && n_removed < kMaxRemovedRing) {
                if (lane == (n_removed >> 2)) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (i == (n_removed & 3)) rem_x[i] = x;
                }
                ++n_removed;
            }
            double zhat, none;
            float f0, f1;
            const bool maybe_last = next < 0;   // no sibling left: the last token is drawn from this residual
            run_pass(kPassResidual, maybe_last, zhat, none, f0, f1, [&] {
                inv_1mP = 1.0 / one_mP_new;
                if (next >= 0) prepare(next);
            }, nothing);
            if (sm.abort) { aborted = true; break; }
            const double Z_new = zhat * inv_Sq;
            if (Z_new > 0.0 && Z_new < 1.7e308) {
                st.Z = Z_new;
                tiles_valid = maybe_last;
            } else {
                status |= 4;   // RSD_ST_ZERO_RESIDUAL: keep the previous residual
                st.A = A_old;
                const double aa = st.A * ratio;
                st.a_hi = (float)aa;
                st.a_lo = (float)(aa - (double)st.a_hi);
                tiles_valid = false;
            }
            if (next >= 0 && err_new > 2e-6 * one_mP_new && n_removed < kMaxRemovedRing) {   // (every rejected token is listed)
                double rest, none2;
                float g0, g1;
                run_pass(kPassTarget, true, rest, none2, g0, g1, nothing, publish_gone, true);
                if (sm.abort) { aborted = true; break; }
                one_mP_new = rest * inv_Sp;
                err_new = 4e-7 * one_mP_new;
                inv_1mP = 1.0 / one_mP_new;
            }
            one_mP = one_mP_new;
            one_mP_err = err_new;
            if (!(one_mP > 0.0)) { status |= 16; break; }   // RSD_ST_DRAFT_EXHAUSTED
            c = next;
        }
        if (aborted) break;
        if (accepted < 0) {   // RSD_STOP_ALL_REJECTED: the last token comes from the residual in force
            reason = 0;
            break;
        }
        if (lane == 0) {
            a.accepted_node[(int64_t)b * a.L + len] = accepted;
            a.accepted_token[(int64_t)b * a.L + len] = cached ? sm.tok[accepted] : tok[accepted];
        }
        ++len;
        cur = accepted;
    }

    const bool residual = st.with_draft && st.A != 0.0;
    if (!aborted && !tiles_valid) {   // rare: the last pass was not kept, or it did not store its tile sums
        double s, none;
        float f0, f1;
        if (!residual) { rowp = rowq; ring.forget_node(); }   // (the slots' draft halves are not refreshed by this pass)
        run_pass(residual ? kPassResidual : kPassTarget, true, s, none, f0, f1, nothing, nothing);
        aborted = sm.abort != 0;
    }
    // the working warps are done: let them go, then finish alone
    if (lane == 0) sm.cmd.kind = kPassEnd;
    if (aborted) {
        // A wait ran out.  Before the block gives its shared memory back, wait once more (bounded) for the copies it
        // may still have in flight: the latest one of every slot.
        for (int s = 0; s < kSlots; ++s) wait_bar(&sm.full[s], (ring.fill_par >> s) & 1u, &sm.abort);   // (a slot never filled passes at once)
        status |= 32;   // RSD_ST_TIMEOUT
    }
    __syncthreads();
    if (!aborted) {
        // Inverse CDF over the tile sums of the last pass: the smallest y whose running sum exceeds u * total; if
        // rounding leaves none, the largest y with positive weight; -1 if there is no weight at all.
        const uint4 rw = rng_draw(key, (uint32_t)cur, kTagResample, 0u);
        const double u = ((double)rw.x + 0.5) * (1.0 / 4294967296.0);
        const int n_tiles = ring.n_tiles;
        // lanes take consecutive runs of tiles; running sums in tile order
        const int per = (n_tiles + 31) / 32;
        const int t_lo = lane * per, t_hi = min(n_tiles, t_lo + per);
        double mine = 0.0;
        for (int t = t_lo; t < t_hi; ++t) mine += sm.tile_sum[t];
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        const double total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        int y = -1;
        if (total > 0.0 && total < 1.7e308) {   // (uniform over the warp)
            const double target = u * total;
            // the tile that holds the crossing, or failing that the last tile with weight
            const unsigned crossing = __ballot_sync(0xFFFFFFFFu, incl > target);
            const unsigned positive = __ballot_sync(0xFFFFFFFFu, mine > 0.0);
            const bool take_last = crossing == 0u;
            const int src = take_last ? 31 - __clz(positive) : __ffs(crossing) - 1;
            int tile = -1;
            double before = 0.0;
            if (lane == src) {
                double cum = incl - mine;
                for (int t = t_lo; t < t_hi; ++t) {
                    const double s = sm.tile_sum[t];
                    if (take_last) { if (s > 0.0) { tile = t; before = cum; } }
                    else if (cum + s > target) { tile = t; before = cum; break; }
                    cum += s;
                }
                if (tile < 0) {   // rounding: the lane's total crossed, no tile did: its last tile with weight
                    cum = incl - mine;
                    for (int t = t_lo; t < t_hi; ++t) {
                        const double s = sm.tile_sum[t];
                        if (s > 0.0) { tile = t; before = cum; }
                        cum += s;
                    }
                }
            }
            tile = __shfl_sync(0xFFFFFFFFu, tile, src);
            before = __shfl_sync(0xFFFFFFFFu, before, src);
            // the tile's weights once more, in token order: lane owns tokens 16 lane .. 16 lane + 15 of the tile
            float w[16];
            const int g = tile * 32 + lane;
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) w[jj] = 0.0f;
            if (tile >= 0 && g * 16 < a.V) group_weights<T>(rowq, rowp, g, a.V, st, residual, w);
            double gs = 0.0;
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) gs += (double)w[jj];
            double gincl = gs;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double t = __shfl_up_sync(0xFFFFFFFFu, gincl, o);
                if (lane >= o) gincl += t;
            }
            const unsigned cross2 = __ballot_sync(0xFFFFFFFFu, !take_last && (before + gincl > target));
            const unsigned pos2 = __ballot_sync(0xFFFFFFFFu, gs > 0.0);
            const bool last_mode = cross2 == 0u;
            const int src2 = last_mode ? (pos2 ? 31 - __clz(pos2) : 0) : __ffs(cross2) - 1;
            if (lane == src2) {
                int last_pos = -1;
                double cacc = before + (gincl - gs);
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    cacc += (double)w[jj];
                    if (w[jj] > 0.0f) last_pos = g * 16 + jj;
                    if (!last_mode && y < 0 && cacc > target) y = g * 16 + jj;
                }
                if (y < 0) y = last_pos;
            }
            y = __shfl_sync(0xFFFFFFFFu, y, src2);
        }
        last = y;
    }
    if (lane == 0) {
        a.accepted_len[b] = len;
        a.last_token[b] = last;
        a.stop_reason[b] = reason;
        a.status[b] = status;
    }
}

}  // namespace walk_ring
}  // namespace rsd
