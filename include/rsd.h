/*
 * librsd: the data-parallel hot path of Recursive Speculative Decoding (RSD) on one GPU.
 *
 *   drafting      rsd_gumbel_topk_draft   per-node Gumbel-Top-k (sampling without replacement)
 *                 rsd_sbs_step            one level of Stochastic Beam Search
 *   verification  rsd_verify_tree         recursive rejection sampling along the draft tree
 *                 rsd_resample_residual   draw from a residual distribution on its own
 *
 * The draft and target language models are outside this library: their logits come in as rows of V values.
 *
 * Conventions that hold for every entry point
 *   - Plain C ABI.  Unless an argument says "host", pointers are DEVICE pointers owned by the caller; the library
 *     never allocates or frees device memory.  The small structs (rsd_rows, rsd_tree) live in host memory and are
 *     read before the call returns.
 *   - Work is enqueued on `stream` (a cudaStream_t) and the call returns without waiting for it.
 *   - The return value reports argument and launch errors only (RSD_OK = 0); rsd_last_error() gives a message for
 *     the calling thread.  Data-dependent trouble (NaN logits, rows with fewer than k finite entries, an empty
 *     residual) never traps: it sets bits in the per-sequence `status` output and follows the documented fallback.
 *     Each call overwrites status[0..B).
 *   - Rows: element (b, r, x) of a batch of rows sits at data + b*seq_stride + r*row_stride + x (strides in
 *     elements).  fp32 or bf16 storage; all arithmetic is fp32 or wider.  The vectorised path needs the base
 *     pointer and both strides to be multiples of 16 bytes; anything else takes a slower scalar path with the same
 *     results.
 *   - Tree layout: flat node index, root = 0, then level by level in stored order.  parent[n] is the flat index of
 *     n's parent (root: -1).  Siblings are ordered by increasing flat index, which is the order the drafting calls
 *     produce (decreasing perturbed value).  A node with token[n] < 0 is absent.
 *   - Randomness is a pure function of (seed, step, global sequence index, flat node id, stream tag, index), drawn
 *     from Philox4x32-10 (Salmon et al., SC'11): key = (seed low word, seed high word), counter = (index,
 *     node | tag << 28, sequence, step).  Global sequence index = seq_base + b, so a batch may be split over
 *     several GPUs without changing any result.  Streams (rsd_rng_layout() == 3), with t(u) = -ln u:
 *       tag 0  Gumbel, one 32-bit word w per group g = x >> 4 of 16 consecutive tokens: word (g >> 5) & 3 of the
 *              call with index = (g >> 7) * 32 + (g & 31) (one call serves four groups 32 apart);
 *              t_M = t(((w >> 4) + 1/2) / 2^28), position a = w & 15
 *       tag 1  Gumbel, per token: index = x >> 2, word w = word x & 3; t_x = t((w + 1/2) / 2^32)
 *              G(x) = -ln( t_M / 16 + (x mod 16 != a ? t_x : 0) )
 *              This draws the 16 noises of a group through the order statistics of 16 i.i.d. uniforms (largest
 *              first, at a uniform position; the rest uniform below it), so they are i.i.d. standard Gumbel and
 *              the group's largest noise is known from one word of the coarse stream.
 *       tag 2  acceptance     : index = rank of the child among its siblings; U = (word0 >> 8) / 2^24
 *       tag 3  final token    : index = 0; u = (word0 + 1/2) / 2^32
 *     The same (seed, step, inputs) give bit-identical outputs whatever the launch shape.
 */
#ifndef RSD_H_
#define RSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* rsd_stream_t; /* a cudaStream_t */

enum { RSD_OK = 0, RSD_ERR_INVALID_ARG = 1, RSD_ERR_UNSUPPORTED = 2, RSD_ERR_WORKSPACE = 3, RSD_ERR_CUDA = 4 };
enum { RSD_F32 = 0, RSD_BF16 = 1 };

/* bits of status[b] */
enum {
    RSD_ST_NAN_INPUT = 1,       /* a NaN logit was read; it was treated as -inf */
    RSD_ST_FEWER_THAN_K = 2,    /* a row had fewer finite entries than picks asked for; outputs padded with -1 */
    RSD_ST_ZERO_RESIDUAL = 4,   /* sum of [q - p]+ was not positive; the previous residual was kept */
    RSD_ST_ZERO_DRAFT_PROB = 8, /* a child token had draft probability 0 (in fp32: below 2^-126 of the row's largest
                                   weight); accepted iff its residual mass is > 0 */
    RSD_ST_DRAFT_EXHAUSTED = 16, /* the draft had no mass left after a removal (in fp32: nothing above 2^-126 of the
                                    row's largest weight); later siblings were ignored */
    RSD_ST_TIMEOUT = 32         /* an on-chip copy of a row did not complete within about a second (a hardware or
                                   driver fault, never a property of the data): the walk of this sequence was
                                   abandoned, accepted_len counts what was accepted before, last_token is -1 */
};

/* stop_reason[b] of the verification walk */
enum { RSD_STOP_ALL_REJECTED = 0, RSD_STOP_NO_CHILDREN = 1, RSD_STOP_LEAF = 2 };

enum {
    RSD_MAX_K = 32,              /* largest number of picks per row / beam width */
    RSD_MAX_ROWS_PER_SEQ = 256,  /* largest R of rsd_gumbel_topk_draft and n_par of rsd_sbs_step */
    RSD_MAX_VOCAB = 262144,
    RSD_MAX_TREE_NODES = 4096    /* largest N + 1 */
};

typedef struct rsd_rows {
    const void* data;   /* device */
    int32_t dtype;      /* RSD_F32 or RSD_BF16 */
    int32_t is_logprob; /* 1: rows are log-probabilities already (drafting uses them as given) */
    int64_t seq_stride; /* elements between sequences */
    int64_t row_stride; /* elements between rows of one sequence, >= V */
    float temperature;  /* sampling temperature (Section 4 uses 0.3 and 1.0): every value is divided by it before the
                           log-softmax; 0 or 1 = none.  With a temperature, rows flagged is_logprob are re-scored
                           (their log-softmax is taken again after the division).  Negative, infinite or NaN values
                           are refused. */
} rsd_rows;

typedef struct rsd_tree {
    int32_t num_levels;         /* L */
    int32_t num_nodes;          /* N + 1, root included */
    const int32_t* parent;      /* device, [num_nodes] if topology_is_shared else [B][num_nodes] */
    const int32_t* token;       /* device, [B][num_nodes]; root entry unused */
    int32_t topology_is_shared; /* 1: one parent[] for all sequences (constant branching factors) */
} rsd_tree;

int rsd_version(void);
int rsd_rng_layout(void);
/* Message of the last error on the calling thread ("" if none).  Host pointer, valid until the next call. */
const char* rsd_last_error(void);

/*
 * Timing aid (the paper has no counterpart).  The next rsd_gumbel_topk_draft or rsd_sbs_step call made by this host
 * thread records the CUDA event `before` right before and `after` right after its row-scan kernel, on that call's
 * stream; the request is then cleared.  Either may be NULL.  Host handles (cudaEvent_t) owned by the caller.
 */
int rsd_profile_next_scan(void* before, void* after);

/*
 * Logit warping of rows before drafting or verification: top-k and nucleus (top-p) filtering (Section 4 samples with
 * temperature 0.3 / 1.0 and, for one task, top-p 0.95; the paper gives no formula).  The order is the usual one,
 * temperature -> top-k -> top-p, each applied to what the one before left:
 *   top-k   keep the top_k largest values of a row (equal values: the smaller token first)
 *   top-p   of what is left, in order of decreasing probability under softmax(value / temperature) (equal values: the
 *           smaller token first), keep the shortest prefix whose share of the mass reaches top_p (at least one token)
 * A filtered token counts as log-probability -inf from then on (Algorithms 4 and 9 drop such entries): the call writes a
 * copy of the rows with -inf at the filtered entries and the stored values (not divided by the temperature) elsewhere,
 * to be passed to the drafting and verification calls in place of the rows, with the same temperature.  Draft and
 * target rows are filtered separately, each with its own settings.
 *   rows        [B][R][V]; rows->temperature enters the nucleus masses only; NaN entries count as -inf (RSD_ST_NAN_INPUT)
 *   top_k       0 (or >= V): none;   top_p  >= 1: none
 *   out_rows    [B][R][V] dense, the rows' element type; may not overlap the input
 *   out_kept    optional [B][R] int32: entries kept in each row;   status [B]
 * Values that compare equal (+0 and -0 among them) are one value: the smaller token goes first.
 * A row must fit in shared memory with the call's other data (up to about 101,000 2-byte or 50,700 4-byte entries);
 * longer rows are refused with RSD_ERR_UNSUPPORTED.  A row whose copy into shared memory does not arrive within about a
 * second sets RSD_ST_TIMEOUT for its sequence, and nothing is written for it.
 */
int rsd_filter_rows(const rsd_rows* rows, int B, int R, int V, int top_k, float top_p, void* out_rows, int32_t* out_kept,
                    int32_t* status, rsd_stream_t stream);

/*
 * Gumbel-Top-k drafting for RSD with constant branching factors (Section 3.2.1, Eqs. 5-8; Algorithm 4).
 * For each of the B*R rows: phi = log-softmax(row) (Eq. 5), phi~ = phi + G (Eq. 6), and the k_per_row[r] tokens
 * with the largest phi~ in decreasing order (Eq. 7); equal values go to the smaller token.  The noise of row r is
 * the Gumbel stream of node rng_node[r] of the sequence.  The arg-top-k does not depend on the row's normaliser,
 * so the log-sum-exp is computed only when out_perturbed or out_logprob is asked for.
 *   draft        rows [B][R][V]
 *   k_per_row    host [R], 1 <= k <= max_k <= RSD_MAX_K
 *   rng_node     host [R], flat node id of each row (< 2^28)
 *   out_token    [B][R][max_k] int32; entries beyond k_per_row[r], or beyond the finite entries of the row, are -1
 *   out_perturbed, out_logprob  optional (NULL to skip) [B][R][max_k] fp32: phi~ and phi of each pick
 *   child_base   optional host [R], node_token optional [B][node_stride] int32: when both are given, pick j of row r
 *                is also stored as the token of tree node child_base[r] + j (Eq. 8's (token, parent) pairs in the
 *                flat layout rsd_verify_tree reads); other entries of node_token are left alone
 *   status       [B]
 */
int rsd_gumbel_topk_draft(const rsd_rows* draft, int B, int R, int V, const int32_t* k_per_row,
                          const int32_t* rng_node, int max_k, uint64_t seed, uint32_t step, uint32_t seq_base,
                          int32_t* out_token, float* out_perturbed, float* out_logprob, const int32_t* child_base,
                          int32_t* node_token, int node_stride, int32_t* status, rsd_stream_t stream);

/*
 * One level of Stochastic Beam Search for RSD-S (Section 3.2.1, Eqs. 10-12; Algorithm 9).
 * Parent slot k of a sequence (flat node first_parent_node + k) has the sequence log-probability
 * sum_logprob_in[b][k] and the truncated Gumbel trunc_gumbel_in[b][k] (both NULL at the root: zeros).
 *   phi_k(x)  = sum_logprob_in[k] + log p_k(x)            phi~_k(x) = phi_k(x) + G_k(x)
 *   psi_k(x)  = T(trunc_gumbel_in[k], phi~_k(x)),  T(u, f) = -log(exp(-u) - exp(-max f) + exp(-f))   (Eq. 11)
 * and the W pairs (x, k) with the largest psi are returned in decreasing order (Eq. 12); equal values go to the
 * smaller parent, then the smaller token.  Entries whose log-probability is -inf are dropped.
 *   draft_level       rows [B][n_par][V], n_par <= RSD_MAX_ROWS_PER_SEQ, W <= RSD_MAX_K
 *   out_token, out_parent   int32, pick i of sequence b at [b * out_stride + i], out_stride >= W; the parent is
 *                     parent_base + slot index within the level, so with out_token/out_parent pointing at a level's
 *                     first node inside [B][N+1] tree arrays and parent_base = first_parent_node the tree arrays
 *                     of rsd_verify_tree are filled in place; entries beyond out_count[b] are -1
 *   sum_logprob_out, trunc_gumbel_out  [B][W] fp32: phi and psi of each pick, the next level's inputs; entries
 *                     beyond out_count[b] are -inf.  On input, a parent slot whose sum_logprob_in or
 *                     trunc_gumbel_in is -inf is such an empty slot: it contributes no children.
 *   out_count         [B]
 *   ws                scratch of at least rsd_sbs_workspace_bytes(B, n_par, W) bytes, 256-byte aligned; contents
 *                     are undefined afterwards; calls that overlap on the GPU need separate scratch
 */
size_t rsd_sbs_workspace_bytes(int B, int n_par, int W);
int rsd_sbs_step(const rsd_rows* draft_level, int B, int n_par, int V, int W, int32_t first_parent_node,
                 const float* sum_logprob_in, const float* trunc_gumbel_in, uint64_t seed, uint32_t step,
                 uint32_t seq_base, int32_t* out_token, int32_t* out_parent, int64_t out_stride, int32_t parent_base,
                 float* sum_logprob_out, float* trunc_gumbel_out, int32_t* out_count, int32_t* status, void* ws,
                 size_t ws_bytes, rsd_stream_t stream);

/*
 * A whole Stochastic Beam Search tree in two launches (Algorithm 8's level loop around Algorithm 9; Eqs. 10-12), for
 * draft rows that all exist before drafting starts.  Row r of a sequence is the draft row of flat node r: the root,
 * then the W slots of level 1, ..., level L - 1 (P = 1 + (L - 1) W rows).  That is the case when the rows do not
 * depend on the tokens picked above them (rows attached to tree slots, as in synthetic workloads or with drafters that
 * predict every position at once); with an autoregressive drafter the rows of a level are only known after the
 * level above, and rsd_sbs_step is the call to use.
 * One launch scans all B * P rows (each with the Gumbel stream of its node), one launch runs the L levels in order,
 * carrying the sequence log-probabilities and truncated Gumbels from level to level on the device.  The results are
 * those of L rsd_sbs_step calls (level l: rows first .. first + n_par with first = 0, n_par = 1 at the root, else
 * first = 1 + (l - 1) W, n_par = W; first_parent_node = parent_base = first), bit for bit.
 *   draft             rows [B][P][V]
 *   node_token, node_parent   [B][node_stride] int32, node_stride >= 1 + L W: entries 1 + l W .. (l + 1) W receive the
 *                     tokens and flat parents of level l + 1's nodes (-1 beyond the level's count); entry 0 (the
 *                     root) is left alone: the arrays are rsd_verify_tree's token / parent
 *   sum_logprob_out, trunc_gumbel_out   optional [B][W]: phi and psi of the last level's picks
 *   level_count       [L][B]: picks of every level;  status [B]: OR of the levels' status bits
 *   ws                scratch of at least rsd_sbs_tree_workspace_bytes(B, W, L) bytes, 256-byte aligned
 */
size_t rsd_sbs_tree_workspace_bytes(int B, int W, int L);
int rsd_sbs_draft_tree(const rsd_rows* draft, int B, int V, int W, int L, uint64_t seed, uint32_t step,
                       uint32_t seq_base, int32_t* node_token, int32_t* node_parent, int64_t node_stride,
                       float* sum_logprob_out, float* trunc_gumbel_out, int32_t* level_count, int32_t* status, void* ws,
                       size_t ws_bytes, rsd_stream_t stream);

/*
 * rsd_sbs_step for callers that cannot allocate device memory (the paper has no counterpart).
 * Some hosts of this library may not call cudaMalloc where they draft: code running inside a serving engine whose
 * memory pool is fixed at start-up, a plug-in that is handed a stream but no allocator, a latency-critical loop that
 * must not take the allocator's lock.  This entry point does the same work as rsd_sbs_step, with the same
 * arguments except the scratch: the scratch is a fixed array of RSD_SBS_STATIC_SCRATCH_BYTES inside the library's
 * device image, which every GPU that loads the library holds until the process exits.  The call itself allocates
 * and frees nothing.
 *   - Sizes: rsd_sbs_workspace_bytes(B, n_par, W) must not exceed RSD_SBS_STATIC_SCRATCH_BYTES (for example
 *     B = 1024, n_par = 8, W = 8 needs 851,968 bytes); larger calls return RSD_ERR_WORKSPACE with a message.
 *   - The first call on each device looks up the array's device address (with that device current) and keeps it;
 *     make that first call outside any stream capture.  The kept address belongs to the device's current context:
 *     after a cudaDeviceReset() in this process it is stale and this entry point must not be used any more.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (every entry is written before
 *     it is read) and its contents after a call are unspecified.  Two calls that overlap on the same GPU (different
 *     streams, or different host threads) race on it: order them, or use rsd_sbs_step with separate scratch.
 */
enum { RSD_SBS_STATIC_SCRATCH_BYTES = 1 << 20 };
int rsd_sbs_step_static(const rsd_rows* draft_level, int B, int n_par, int V, int W, int32_t first_parent_node,
                        const float* sum_logprob_in, const float* trunc_gumbel_in, uint64_t seed, uint32_t step,
                        uint32_t seq_base, int32_t* out_token, int32_t* out_parent, int64_t out_stride,
                        int32_t parent_base, float* sum_logprob_out, float* trunc_gumbel_out, int32_t* out_count,
                        int32_t* status, rsd_stream_t stream);

/*
 * Draft-tree verification by recursive rejection sampling (Section 3.1, Eqs. 1-4, Algorithm 1; Section 3.2.2,
 * Algorithm 6).  Per sequence, starting at the root: the children of the current node are tested in stored order
 * with p = softmax(draft row of the node), q = softmax(target row of the node):
 *   accept child j with probability min(1, q_j(x_j) / p_j(x_j))                                      (Eq. 3)
 *   on rejection  q_{j+1} = Norm[(q_j - p_j)+],  p_{j+1} = p_j without x_j, renormalised           (Eqs. 1-2)
 * The first accepted child becomes the current node.  The walk ends with one more token drawn by inverse CDF:
 * from the last residual if every child was rejected, from the node's target row if it has no children
 * (RSD_STOP_NO_CHILDREN) or is at depth L (RSD_STOP_LEAF).  Only the rows of visited nodes are read.
 *   draft   rows of nodes that can have children (flat ids 0 .. P-1);  target  rows of all nodes (0 .. N)
 *   accepted_len [B]; accepted_node, accepted_token [B][L] (-1 padded); last_token [B]; stop_reason [B]
 *   dbg_theta    optional [B][num_nodes] fp32: the acceptance threshold of every child that was tested, NaN elsewhere
 * draft and target must have the same dtype.  Rows given as log-probabilities are renormalised like logits.
 */
int rsd_verify_tree(const rsd_rows* draft, const rsd_rows* target, const rsd_tree* tree, int B, int V,
                    uint64_t seed, uint32_t step, uint32_t seq_base, int32_t* accepted_len, int32_t* accepted_node,
                    int32_t* accepted_token, int32_t* last_token, int32_t* stop_reason, float* dbg_theta,
                    int32_t* status, rsd_stream_t stream);

/*
 * rsd_verify_tree with the verification rule and the sampler of the last token as arguments: recursive rejection
 * sampling, or one of the two
 * earlier tree verifiers that Section 2 describes, run over the same tree layout, rows and random streams, so that
 * acceptance rates can be compared on equal inputs (Figure 1 does this for Bernoulli distributions).
 *   RSD_RULE_RRS         recursive rejection sampling (Section 3.1): exactly rsd_verify_tree
 *   RSD_RULE_MULTIROUND  multi-round rejection sampling with one draft model, p^(k) = p (Section 2, SpecInfer): the
 *                        children of a node are independent draws from p (repeats allowed); child j is accepted
 *                        with probability min(1, q^(j)(x_j) / p(x_j)), q^(j+1) = Norm[(q^(j) - p)+]; the draft is
 *                        never changed
 *   RSD_RULE_KSEQ        K-sequential selection (Section 2, SpecTr), K = the number of children of the node: child j
 *                        is accepted with probability min(1, q(x_j) / (gamma p(x_j))); if all K are rejected the
 *                        token is drawn from Norm[(q - min{p, q/gamma} (1 - (1 - beta)^K) / beta)+] with
 *                        beta = sum_x min{p(x), q(x)/gamma}.  gamma in [1, K]; gamma = K is always admissible
 *                        (smaller values need (1 - (1 - beta)^K) / beta <= gamma, else the clamp at 0 applies)
 * gamma is read only by RSD_RULE_KSEQ (finite, >= 1).
 * final_sampler chooses how the last token is drawn from its distribution w (a residual or a target row):
 *   RSD_FINAL_INVERSE_CDF  one uniform, smallest y whose running sum of w exceeds u * sum(w): rsd_verify_tree's way
 *   RSD_FINAL_GUMBEL_TOP1  arg max over y of log w(y) + G(y) with fresh standard Gumbel noise G (Algorithm 6's last
 *                          step; the same law), drawn group-wise like the drafting noise from streams of its own
 * All other arguments, outputs and status bits as in rsd_verify_tree; RSD_ST_ZERO_RESIDUAL under K-SEQ means the
 * token was drawn from the target row itself.
 */
enum { RSD_RULE_RRS = 0, RSD_RULE_MULTIROUND = 1, RSD_RULE_KSEQ = 2 };
enum { RSD_FINAL_INVERSE_CDF = 0, RSD_FINAL_GUMBEL_TOP1 = 1 };
int rsd_verify_tree_rule(const rsd_rows* draft, const rsd_rows* target, const rsd_tree* tree, int B, int V,
                         int rule, float gamma, int final_sampler, uint64_t seed, uint32_t step, uint32_t seq_base,
                         int32_t* accepted_len, int32_t* accepted_node, int32_t* accepted_token, int32_t* last_token,
                         int32_t* stop_reason, float* dbg_theta, int32_t* status, rsd_stream_t stream);

/*
 * One draw from a residual distribution (Eq. 2 applied along a list of rejected drafts; Section 2's
 * Norm[(q - p)+] is the one-token case).  Per sequence: p = softmax(draft row), q = softmax(target row); for each
 * token of rejected[b][0..max_k) in order (-1 = none) the chain step of Eqs. 1-2 is applied; then one token is
 * drawn by inverse CDF with the final-token stream of node rng_node[b].  With no rejected token this is a plain
 * draw from the target row and `draft` may be NULL.
 *   draft_row, target_row   rows [B][1][V] (row_stride unused)
 *   rejected     [B][max_k] int32 or NULL;  rng_node [B] int32 (device)
 *   out_token    [B];  out_residual  optional [B][V] fp32, the normalised distribution drawn from
 */
int rsd_resample_residual(const rsd_rows* draft_row, const rsd_rows* target_row, int B, int V,
                          const int32_t* rejected, int max_k, const int32_t* rng_node, uint64_t seed, uint32_t step,
                          uint32_t seq_base, int32_t* out_token, float* out_residual, int32_t* status,
                          rsd_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* RSD_H_ */
