/*
 * CPU oracle for Recursive Speculative Decoding (RSD): drafting by sampling
 * without replacement and verification by recursive rejection sampling.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, double-precision
 * restatement of the paper's definitions, used only to check the CUDA library
 * and to serve as a timed CPU baseline.  It shares no code with the CUDA path
 * and nothing in the product may call it.
 *
 * What follows the paper and where:
 *   - log-softmax of a row ......................... Eq. 5
 *   - Gumbel perturbation, sorted arg-top-k ......... Eqs. 6-7, Algorithm 4
 *   - Stochastic Beam Search step .................. Eqs. 10-12, Algorithm 9
 *   - recursive rejection sampling (one sibling chain) Eqs. 1-4, Algorithm 1
 *   - verification walk over the draft tree ......... Section 3.2.2, Algorithm 6
 *   - top-k / nucleus filtering of a row ............ Section 4 (sampling settings), Algorithms 4 and 9 (-inf filter)
 *
 * Random numbers.  The paper only says "standard Gumbel" and "Uniform[0,1]".
 * Both sides of the parity check draw them from the counter-based generator
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with the counter layout
 * documented at draw() and rsd_oracle_gumbel() below (RNG layout version 3).
 *
 * Pins (see tests, "-m 'not gpu'"): Philox known answers and bijectivity,
 * Gumbel moments/CDF, Plackett-Luce law of Gumbel-Top-k, exact enumeration of
 * Theorem 3.1 for small vocabularies, the K=1 and Bernoulli special cases,
 * the sampling-without-replacement law of Stochastic Beam Search on a toy
 * model, hand-built trees for the walk, inverse-CDF edges.
 * Parity unpinned: none of the functions below lacks a pin; what cannot be
 * pinned is only "one whole step at V = 32000 against an external program",
 * because no such program exists.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

/* status bits (same meaning as the library's, restated here on purpose) */
#define ORC_ST_NAN_INPUT 1
#define ORC_ST_FEWER_THAN_K 2
#define ORC_ST_ZERO_RESIDUAL 4
#define ORC_ST_ZERO_DRAFT_PROB 8
#define ORC_ST_DRAFT_EXHAUSTED 16

/* stop reasons of the verification walk */
#define ORC_STOP_ALL_REJECTED 0
#define ORC_STOP_NO_CHILDREN 1
#define ORC_STOP_LEAF 2

/* stream tags of the RNG layout */
#define TAG_GUMBEL_COARSE 0u
#define TAG_GUMBEL_FINE 1u
#define TAG_ACCEPT 2u
#define TAG_RESAMPLE 3u
#define TAG_FINAL_GUMBEL_COARSE 4u /* Gumbel-Top-1 draw of the last token: same group-wise layout, own streams */
#define TAG_FINAL_GUMBEL_FINE 5u

/* ------------------------------------------------------------------------ */
/* Philox4x32-10, written from the published definition: ten rounds of      */
/*   (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)) */
/* with the key bumped by the Weyl constants between rounds.                */
/* ------------------------------------------------------------------------ */
void rsd_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Counter and key of every stream (RNG layout version 3).  key = (seed low word, seed high word).
 * counter = (index, node | tag << 28, sequence, step) where
 *   node     = flat node id inside the sequence's tree (< 2^28),
 *   sequence = global sequence index of the batch,
 *   step     = decode step counter (32 bits),
 *   tag      = which stream; index = position inside that stream.
 */
static void draw(uint64_t seed, uint32_t step, uint32_t seq, uint32_t node, uint32_t tag, uint32_t index,
                 uint32_t out[4]) {
    uint32_t ctr[4] = {index, (node & 0x0FFFFFFFu) | (tag << 28), seq, step};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    rsd_oracle_philox4x32_10(ctr, key, out);
}

int rsd_oracle_rng_layout(void) { return 3; }

/*
 * Gumbel noise of (sequence, node), RNG layout 3.  The noise of the V elements must be i.i.d. standard Gumbel
 * (Eq. 6).  It is drawn group-wise, 16 consecutive elements per group, from the order statistics of 16 i.i.d.
 * uniforms: the largest of them is V^(1/16) for a uniform V, it sits at a uniformly random position a, and the
 * other 15 are i.i.d. uniform below it.  With t(U) = -ln U this reads
 *     coarse stream: one 32-bit word per group g = x >> 4, namely word (g >> 5) & 3 of the call with
 *         index (g >> 7) * 32 + (g & 31); its upper 28 bits -> U_M = (bits + 1/2) / 2^28, its low 4 bits -> a
 *     fine stream, index = x >> 2, word x & 3 -> U_x = (bits + 1/2) / 2^32
 *     G_x = -ln( t(U_M) / 16 + [x mod 16 != a] * t(U_x) ).
 * (max of 16 uniforms M = U_M^(1/16) has -ln M = t(U_M)/16; another element is M * U_x, so -ln of it is
 * t(U_M)/16 + t(U_x); G = -ln(-ln U).)  The element at position a carries the group's largest noise, which is
 * known from the coarse stream alone.
 */
static double neg_log_uniform(uint32_t bits) {
    return -log(((double)bits + 0.5) * (1.0 / 4294967296.0));
}

/* the three ingredients of G_x: t(U_M) of the group, the position a, t(U_x) */
void rsd_oracle_gumbel_parts(uint64_t seed, uint32_t step, uint32_t seq, uint32_t node, uint32_t e,
                             double* t_group, int32_t* argmax_pos, double* t_elem) {
    uint32_t w[4];
    const uint32_t g = e >> 4;
    draw(seed, step, seq, node, TAG_GUMBEL_COARSE, ((g >> 7) << 5) | (g & 31u), w);
    const uint32_t word = w[(g >> 5) & 3u];
    *t_group = -log(((double)(word >> 4) + 0.5) * (1.0 / 268435456.0));
    *argmax_pos = (int32_t)(word & 15u);
    draw(seed, step, seq, node, TAG_GUMBEL_FINE, e >> 2, w);
    *t_elem = neg_log_uniform(w[e & 3u]);
}

double rsd_oracle_gumbel(uint64_t seed, uint32_t step, uint32_t seq, uint32_t node, uint32_t e) {
    double tg, te;
    int32_t a;
    rsd_oracle_gumbel_parts(seed, step, seq, node, e, &tg, &a, &te);
    return -log(tg / 16.0 + ((int32_t)(e & 15u) != a ? te : 0.0));
}

/* Gumbel noise of element e for the Gumbel-Top-1 draw of the last token at `node` (same law and layout as above) */
static double final_gumbel(uint64_t seed, uint32_t step, uint32_t seq, uint32_t node, uint32_t e) {
    uint32_t w[4];
    const uint32_t g = e >> 4;
    draw(seed, step, seq, node, TAG_FINAL_GUMBEL_COARSE, ((g >> 7) << 5) | (g & 31u), w);
    const uint32_t word = w[(g >> 5) & 3u];
    const double tg = -log(((double)(word >> 4) + 0.5) * (1.0 / 268435456.0));
    const int32_t a = (int32_t)(word & 15u);
    draw(seed, step, seq, node, TAG_FINAL_GUMBEL_FINE, e >> 2, w);
    const double te = neg_log_uniform(w[e & 3u]);
    return -log(tg / 16.0 + ((int32_t)(e & 15u) != a ? te : 0.0));
}

/*
 * Last token by Gumbel-Top-1 (Algorithm 6's final step): arg max over y of log w(y) + G(y), entries with
 * w(y) = 0 left out; equal values go to the smaller token.  margin = gap to the runner-up.  -1 if w has no mass.
 */
static int gumbel_top1(const double* w, int V, uint64_t seed, uint32_t step, uint32_t seq, uint32_t node,
                       double* margin) {
    int best = -1;
    double vb = -INFINITY, v2 = -INFINITY;
    for (int y = 0; y < V; ++y) {
        if (!(w[y] > 0.0)) continue;
        double v = log(w[y]) + final_gumbel(seed, step, seq, node, (uint32_t)y);
        if (v > vb) { v2 = vb; vb = v; best = y; }
        else if (v > v2) v2 = v;
    }
    if (margin) *margin = (best >= 0) ? vb - v2 : 0.0;
    return best;
}

/* U for the acceptance test of the j-th child (stored order) of `node`: 24 bits, in [0,1) */
double rsd_oracle_accept_uniform(uint64_t seed, uint32_t step, uint32_t seq, uint32_t node, uint32_t j) {
    uint32_t w[4];
    draw(seed, step, seq, node, TAG_ACCEPT, j, w);
    return (double)(w[0] >> 8) * (1.0 / 16777216.0);
}

/* u for the final-token draw at `node`: 32 bits, in (0,1) */
double rsd_oracle_resample_uniform(uint64_t seed, uint32_t step, uint32_t seq, uint32_t node) {
    uint32_t w[4];
    draw(seed, step, seq, node, TAG_RESAMPLE, 0, w);
    return ((double)w[0] + 0.5) * (1.0 / 4294967296.0);
}

/* ------------------------------------------------------------------------ */
/* rows                                                                      */
/* ------------------------------------------------------------------------ */
static double read_elem(const void* base, int dtype, int64_t idx) {
    if (dtype == ORC_F32) return (double)((const float*)base)[idx];
    uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16; /* bf16 widens exactly */
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

/* sampling temperature (Section 4: 0.3 or 1.0): a value <= 0 or == 1 means "none" */
static int has_temperature(double t) { return t > 0.0 && t != 1.0; }

/* copy a row to double, divided by the temperature; NaN becomes -inf and is reported */
static int load_row(const void* base, int dtype, int64_t off, int V, double temperature, double* out) {
    int saw_nan = 0;
    for (int x = 0; x < V; ++x) {
        double v = read_elem(base, dtype, off + x);
        if (isnan(v)) { v = -INFINITY; saw_nan = 1; }
        out[x] = has_temperature(temperature) ? v / temperature : v;
    }
    return saw_nan;
}

/* log-sum-exp with the maximum taken out; -inf for a row with no finite entry */
static double log_sum_exp(const double* v, int V) {
    double m = -INFINITY;
    for (int x = 0; x < V; ++x) if (v[x] > m) m = v[x];
    if (!(m > -INFINITY) || isinf(m)) return m;
    double s = 0.0;
    for (int x = 0; x < V; ++x) s += exp(v[x] - m);
    return m + log(s);
}

/* Eq. 5: phi = log p(.|tau).  Rows flagged as log-probabilities are used as given. */
static void log_softmax_row(double* v, int V, int is_logprob) {
    if (is_logprob) return;
    double lse = log_sum_exp(v, V);
    if (isinf(lse)) return;
    for (int x = 0; x < V; ++x) v[x] -= lse;
}

/* probabilities of a row: softmax (rows given as log-probabilities are renormalised too) */
static void softmax_row(const double* logits, int V, double* prob) {
    double lse = log_sum_exp(logits, V);
    for (int x = 0; x < V; ++x) prob[x] = isinf(lse) ? 0.0 : exp(logits[x] - lse);
}

/* ------------------------------------------------------------------------ */
/* logit warping: top-k and nucleus (top-p) filtering (Section 4)            */
/* ------------------------------------------------------------------------ */
/*
 * Section 4 samples with temperature 0.3 / 1.0 and, for one task, nucleus (top-p) sampling with p = 0.95; the
 * paper gives no formula.  Reading: the usual order of logit warpers, temperature -> top-k -> top-p, each applied
 * to what the one before left:
 *   top-k   keep the k tokens with the largest probability (equal values: the smaller token first);
 *   top-p   sort what is left by probability, largest first (equal values: the smaller token first), renormalise,
 *           and keep the shortest prefix whose mass reaches top_p (at least one token).
 * A filtered token counts as log-probability -inf from then on ("filter elements whose log-prob is -inf",
 * Algorithms 4 and 9).  top_k <= 0 or >= V and top_p <= 0 or >= 1 mean "no filter".
 *
 * keep[x] = 1 for kept tokens.  *margin = distance of top_p from the two cumulative masses that bracket it
 * (the mass of the kept prefix, and that prefix without its last token), as fractions of the total; +inf if no
 * nucleus filter applies.  Returns the number of kept tokens.
 */
typedef struct { double v; int x; } orc_entry;
static int orc_entry_cmp(const void* a, const void* b) {
    const orc_entry* ea = (const orc_entry*)a;
    const orc_entry* eb = (const orc_entry*)b;
    if (ea->v > eb->v) return -1;
    if (ea->v < eb->v) return 1;
    return (ea->x > eb->x) - (ea->x < eb->x);
}

int rsd_oracle_filter_row(const double* scaled /* row / temperature, NaN already -inf */, int V, int top_k, double top_p,
                          uint8_t* keep, double* margin) {
    orc_entry* e = (orc_entry*)malloc(sizeof(orc_entry) * (size_t)V);
    int n = 0;
    for (int x = 0; x < V; ++x) {
        keep[x] = 0;
        if (scaled[x] > -INFINITY) { e[n].v = scaled[x]; e[n].x = x; ++n; }
    }
    qsort(e, (size_t)n, sizeof(orc_entry), orc_entry_cmp);   /* decreasing value, then increasing token */
    if (top_k > 0 && top_k < V && n > top_k) n = top_k;
    if (margin) *margin = INFINITY;
    if (top_p > 0.0 && top_p < 1.0 && n > 0) {
        double total = 0.0;
        for (int i = 0; i < n; ++i) total += exp(e[i].v - e[0].v);
        double run = 0.0;
        int m = n;
        for (int i = 0; i < n; ++i) {
            double before = run;
            run += exp(e[i].v - e[0].v);
            if (run >= top_p * total) {
                m = i + 1;
                if (margin) {
                    double a = run / total - top_p, b = top_p - before / total;
                    *margin = a < b ? a : b;
                }
                break;
            }
        }
        n = m;
    }
    for (int i = 0; i < n; ++i) keep[e[i].x] = 1;
    free(e);
    return n;
}

/* rows [B][R][V] -> keep [B][R][V] (1 = kept), kept [B][R], margin [B][R] */
int rsd_oracle_filter_rows(const void* data, int dtype, double temperature, int64_t seq_stride, int64_t row_stride,
                           int B, int R, int V, int top_k, double top_p, uint8_t* keep, int32_t* kept, double* margin) {
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int r = 0; r < R; ++r) {
            double* v = (double*)malloc(sizeof(double) * (size_t)V);
            load_row(data, dtype, b * seq_stride + r * row_stride, V, temperature, v);
            kept[(int64_t)b * R + r] = rsd_oracle_filter_row(v, V, top_k, top_p, keep + ((int64_t)b * R + r) * V,
                                                             margin ? margin + (int64_t)b * R + r : NULL);
            free(v);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Gumbel-Top-k (Algorithm 4, Eqs. 6-7)                                      */
/* ------------------------------------------------------------------------ */
/*
 * For each of B*R rows: perturb the log-probabilities with the Gumbel noise of
 * (sequence, rng_node[r]) and return the k_per_row[r] largest, in decreasing
 * order; equal values go to the smaller token.  -inf entries are never
 * selected; missing picks are -1.  out_margin[b][r] = the smallest gap between
 * consecutive sorted values v_1 >= ... >= v_{k+1} (v_{k+1} = best loser).
 */
int rsd_oracle_gumbel_topk(const void* data, int dtype, int is_logprob, double temperature, int64_t seq_stride,
                           int64_t row_stride,
                           int B, int R, int V, const int32_t* k_per_row, const int32_t* rng_node, int max_k,
                           uint64_t seed, uint32_t step, uint32_t seq_base,
                           int32_t* out_token, double* out_perturbed, double* out_logprob, double* out_margin,
                           int32_t* status) {
    for (int b = 0; b < B; ++b) status[b] = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int r = 0; r < R; ++r) {
            double* phi = (double*)malloc(sizeof(double) * (size_t)V);
            double* pert = (double*)malloc(sizeof(double) * (size_t)V);
            char* taken = (char*)calloc((size_t)V, 1);
            int st = 0;
            if (load_row(data, dtype, b * seq_stride + r * row_stride, V, temperature, phi)) st |= ORC_ST_NAN_INPUT;
            log_softmax_row(phi, V, is_logprob && !has_temperature(temperature));   /* scaled rows are scores again */
            for (int x = 0; x < V; ++x)
                pert[x] = phi[x] + rsd_oracle_gumbel(seed, step, seq_base + (uint32_t)b, (uint32_t)rng_node[r], (uint32_t)x);
            int k = k_per_row[r];
            double margin = INFINITY, prev = 0.0;
            int64_t o = ((int64_t)b * R + r) * max_k;
            for (int i = 0; i < max_k; ++i) {
                out_token[o + i] = -1;
                if (out_perturbed) out_perturbed[o + i] = -INFINITY;
                if (out_logprob) out_logprob[o + i] = -INFINITY;
            }
            for (int i = 0; i <= k; ++i) { /* k picks and the best loser */
                int best = -1;
                for (int x = 0; x < V; ++x) {
                    if (taken[x] || !(phi[x] > -INFINITY)) continue;
                    if (best < 0 || pert[x] > pert[best]) best = x; /* strict: smaller token wins ties */
                }
                if (best < 0) { if (i < k) st |= ORC_ST_FEWER_THAN_K; break; }
                taken[best] = 1;
                if (i > 0 && prev - pert[best] < margin) margin = prev - pert[best];
                prev = pert[best];
                if (i < k) {
                    out_token[o + i] = best;
                    if (out_perturbed) out_perturbed[o + i] = pert[best];
                    if (out_logprob) out_logprob[o + i] = phi[best];
                }
            }
            if (out_margin) out_margin[(int64_t)b * R + r] = margin;
            if (st) {
#pragma omp atomic
                status[b] |= st;
            }
            free(phi); free(pert); free(taken);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Stochastic Beam Search step (Algorithm 9, Eqs. 10-12)                     */
/* ------------------------------------------------------------------------ */
/*
 * T(u, phi) of Eq. 11 for one entry: -log(exp(-u) - exp(-z) + exp(-phi)),
 * z = max phi.  The paper prints no stable form; this one follows from Eq. 11:
 *   exp(-phi) - exp(-z) = exp(-phi) * (1 - exp(phi - z)),
 *   w = log1p(-exp(phi - z))            (-inf at the arg-max),
 *   v = u - phi + w,
 *   T = u - log(1 + exp(v)) = u - max(v,0) - log1p(exp(-|v|)).
 */
double rsd_oracle_truncated_gumbel(double u, double phi, double z) {
    if (!(phi > -INFINITY)) return -INFINITY;
    double d = phi - z;
    if (d >= 0.0) return u;
    double w = log1p(-exp(d));
    double v = u - phi + w;
    double av = fabs(v);
    return u - (v > 0.0 ? v : 0.0) - log1p(exp(-av));
}

/*
 * One level for B sequences.  Parent slot k (flat node first_parent_node + k)
 * carries sum_logprob_in[b][k] and trunc_gumbel_in[b][k] (NULL = zeros, the
 * root).  Outputs the W best (token, parent) pairs by psi, decreasing; equal
 * values go to the smaller parent, then the smaller token.
 */
int rsd_oracle_sbs_step(const void* data, int dtype, int is_logprob, double temperature, int64_t seq_stride,
                        int64_t row_stride,
                        int B, int n_par, int V, int W, int32_t first_parent_node,
                        const double* sum_logprob_in, const double* trunc_gumbel_in,
                        uint64_t seed, uint32_t step, uint32_t seq_base,
                        int32_t* out_token, int32_t* out_parent, double* sum_logprob_out, double* trunc_gumbel_out,
                        int32_t* out_count, double* out_margin, int32_t* status) {
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        size_t n = (size_t)n_par * (size_t)V;
        double* phi = (double*)malloc(sizeof(double) * n);  /* sequence log-prob of each child */
        double* psi = (double*)malloc(sizeof(double) * n);  /* truncated perturbed value */
        char* taken = (char*)calloc(n, 1);
        int st = 0;
        for (int k = 0; k < n_par; ++k) {
            double* row = phi + (size_t)k * V;
            if (load_row(data, dtype, b * seq_stride + k * row_stride, V, temperature, row)) st |= ORC_ST_NAN_INPUT;
            log_softmax_row(row, V, is_logprob && !has_temperature(temperature));
            double sigma = sum_logprob_in ? sum_logprob_in[(int64_t)b * n_par + k] : 0.0;
            double gamma = trunc_gumbel_in ? trunc_gumbel_in[(int64_t)b * n_par + k] : 0.0;
            double* pert = psi + (size_t)k * V;
            double z = -INFINITY;
            for (int x = 0; x < V; ++x) {
                row[x] += sigma;                                                       /* phi_l = phi_{l-1} + log p */
                pert[x] = row[x] + rsd_oracle_gumbel(seed, step, seq_base + (uint32_t)b,
                                                     (uint32_t)(first_parent_node + k), (uint32_t)x); /* phi~ */
                if (pert[x] > z) z = pert[x];                                          /* row maximum */
            }
            for (int x = 0; x < V; ++x) pert[x] = rsd_oracle_truncated_gumbel(gamma, pert[x], z);
        }
        double margin = INFINITY, prev = 0.0;
        int count = 0;
        for (int i = 0; i < W; ++i) {
            out_token[(int64_t)b * W + i] = -1;
            out_parent[(int64_t)b * W + i] = -1;
            sum_logprob_out[(int64_t)b * W + i] = -INFINITY;
            trunc_gumbel_out[(int64_t)b * W + i] = -INFINITY;
        }
        for (int i = 0; i <= W; ++i) {
            int64_t best = -1;
            for (size_t c = 0; c < n; ++c) {
                if (taken[c] || !(phi[c] > -INFINITY)) continue;
                if (best < 0 || psi[c] > psi[best]) best = (int64_t)c; /* strict: (parent, token) order wins ties */
            }
            if (best < 0) { if (i < W) st |= ORC_ST_FEWER_THAN_K; break; }
            taken[best] = 1;
            if (i > 0 && prev - psi[best] < margin) margin = prev - psi[best];
            prev = psi[best];
            if (i < W) {
                out_token[(int64_t)b * W + i] = (int32_t)(best % V);
                out_parent[(int64_t)b * W + i] = (int32_t)(best / V);
                sum_logprob_out[(int64_t)b * W + i] = phi[best];
                trunc_gumbel_out[(int64_t)b * W + i] = psi[best];
                ++count;
            }
        }
        out_count[b] = count;
        if (out_margin) out_margin[b] = margin;
        status[b] = st;
        free(phi); free(psi); free(taken);
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* final-token draw: inverse CDF                                             */
/* ------------------------------------------------------------------------ */
/*
 * Smallest y whose running sum exceeds u * total; if rounding leaves none, the
 * largest y with positive weight.  margin = distance of u*total from the two
 * running sums that bracket it, relative to total.
 */
int rsd_oracle_inverse_cdf(const double* w, int V, double u, double* margin) {
    double total = 0.0;
    for (int y = 0; y < V; ++y) total += w[y];
    double target = u * total, run = 0.0;
    int last_pos = -1;
    for (int y = 0; y < V; ++y) {
        double before = run;
        run += w[y];
        if (w[y] > 0.0) last_pos = y;
        if (run > target) {
            if (margin) {
                double a = target - before, c = run - target;
                *margin = (a < c ? a : c) / total;
            }
            return y;
        }
    }
    if (margin) *margin = 0.0;
    return last_pos;
}

/* ------------------------------------------------------------------------ */
/* recursive rejection sampling on one sibling chain (Eqs. 1-4, Algorithm 1) */
/* ------------------------------------------------------------------------ */
/*
 * State of the chain: target residual q^(k) and draft p^(k), both normalised.
 * rrs_threshold = Eq. 3.  rrs_reject = Eq. 2 followed by the removal of the
 * rejected token from the draft (sampling without replacement, Eq. 1): the
 * residual is formed with the draft that generated the token, THEN the token
 * is removed and the draft renormalised.
 */
static double rrs_threshold(const double* q, const double* p, int x, int* st) {
    if (p[x] > 0.0) {
        double r = q[x] / p[x];
        return r < 1.0 ? r : 1.0;
    }
    *st |= ORC_ST_ZERO_DRAFT_PROB; /* a child the draft could not have produced */
    return q[x] > 0.0 ? 1.0 : 0.0;
}

/* returns 0 if the draft has no mass left after the removal, else 1 */
static int rrs_reject(double* q, double* p, int V, int x, int* st) {
    double s = 0.0;
    for (int y = 0; y < V; ++y) {
        double r = q[y] - p[y];
        s += (r > 0.0 ? r : 0.0);
    }
    if (s > 0.0 && isfinite(s)) {
        for (int y = 0; y < V; ++y) {
            double r = q[y] - p[y];
            q[y] = (r > 0.0 ? r : 0.0) / s;
        }
    } else {
        *st |= ORC_ST_ZERO_RESIDUAL; /* q == p up to rounding: keep q */
    }
    p[x] = 0.0;
    double t = 0.0;
    for (int y = 0; y < V; ++y) t += p[y];
    if (!(t > 0.0)) { *st |= ORC_ST_DRAFT_EXHAUSTED; return 0; }
    for (int y = 0; y < V; ++y) p[y] /= t;
    return 1;
}

/*
 * Multi-round rejection sampling (Section 2, the SpecInfer paragraph) with one
 * draft model, p^(k) = p for every k: the children are independent draws from
 * p (repeats allowed), the threshold is min{1, q^(k)(x)/p(x)} and the residual
 * q^(k+1) = Norm[(q^(k) - p)+].  The draft is never changed.
 */
static void multiround_reject(double* q, const double* p, int V, int* st) {
    double s = 0.0;
    for (int y = 0; y < V; ++y) {
        double r = q[y] - p[y];
        s += (r > 0.0 ? r : 0.0);
    }
    if (s > 0.0 && isfinite(s)) {
        for (int y = 0; y < V; ++y) {
            double r = q[y] - p[y];
            q[y] = (r > 0.0 ? r : 0.0) / s;
        }
    } else {
        *st |= ORC_ST_ZERO_RESIDUAL;
    }
}

/*
 * K-sequential draft selection (Section 2, the SpecTr paragraph): each of the
 * K independent drafts x ~ p is accepted with probability
 * min{1, q(x) / (gamma p(x))}; if all K are rejected the token comes from
 * Norm[q - min{p, q/gamma} (1 - (1 - beta)^K) / beta],  beta = sum_x min{p(x), q(x)/gamma}.
 * Negative entries (a gamma too small for these p, q, K) are clamped to 0.
 */
static double kseq_threshold(const double* q, const double* p, double gamma, int x, int* st) {
    if (p[x] > 0.0) {
        double r = q[x] / (gamma * p[x]);
        return r < 1.0 ? r : 1.0;
    }
    *st |= ORC_ST_ZERO_DRAFT_PROB;
    return q[x] > 0.0 ? 1.0 : 0.0;
}

static void kseq_residual(double* q, const double* p, int V, double gamma, int K, int* st) {
    double beta = 0.0;
    for (int y = 0; y < V; ++y) {
        double a = p[y], b = q[y] / gamma;
        beta += (a < b ? a : b);
    }
    double c = beta > 0.0 ? (1.0 - pow(1.0 - beta, (double)K)) / beta : (double)K;
    double s = 0.0;
    for (int y = 0; y < V; ++y) {
        double a = p[y], b = q[y] / gamma;
        double r = q[y] - (a < b ? a : b) * c;
        s += (r > 0.0 ? r : 0.0);
    }
    if (s > 0.0 && isfinite(s)) {
        for (int y = 0; y < V; ++y) {
            double a = p[y], b = q[y] / gamma;
            double r = q[y] - (a < b ? a : b) * c;
            q[y] = (r > 0.0 ? r : 0.0) / s;
        }
    } else {
        *st |= ORC_ST_ZERO_RESIDUAL;
    }
}

/*
 * Deterministic part of the two baseline verifiers for given distributions and
 * an ordered tuple of K drafts: theta[k] assuming all earlier drafts were
 * rejected, residual = the distribution of the token drawn when all K are
 * rejected.  rule 1 = multi-round, rule 2 = K-SEQ.
 */
int rsd_oracle_baseline_chain(int rule, double gamma, const double* p_in, const double* q_in, int V,
                              const int32_t* tokens, int K, double* theta, double* residual) {
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    memcpy(q, q_in, sizeof(double) * (size_t)V);
    int st = 0;
    for (int k = 0; k < K; ++k) {
        if (rule == 1) {
            theta[k] = rrs_threshold(q, p_in, tokens[k], &st);
            multiround_reject(q, p_in, V, &st);
        } else {
            theta[k] = kseq_threshold(q, p_in, gamma, tokens[k], &st);
        }
    }
    if (rule != 1) kseq_residual(q, p_in, V, gamma, K, &st);
    memcpy(residual, q, sizeof(double) * (size_t)V);
    free(q);
    return st;
}

/*
 * Deterministic part of Algorithm 1 for given distributions and an ordered
 * draft tuple: theta[k] = Theta^(k+1) assuming all earlier drafts were
 * rejected, residual = q^(K+1).  Used by the exact-enumeration pins.
 */
int rsd_oracle_rrs_chain(const double* p_in, const double* q_in, int V, const int32_t* tokens, int K,
                         double* theta, double* residual) {
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    memcpy(p, p_in, sizeof(double) * (size_t)V);
    memcpy(q, q_in, sizeof(double) * (size_t)V);
    int st = 0;
    for (int k = 0; k < K; ++k) {
        theta[k] = rrs_threshold(q, p, tokens[k], &st);
        if (!rrs_reject(q, p, V, tokens[k], &st)) {
            for (int j = k + 1; j < K; ++j) theta[j] = 0.0;
            break;
        }
    }
    memcpy(residual, q, sizeof(double) * (size_t)V);
    free(p); free(q);
    return st;
}

/* ------------------------------------------------------------------------ */
/* verification walk over the tree (Section 3.2.2, Algorithm 6)              */
/* ------------------------------------------------------------------------ */
/*
 * Flat node index: root 0, then level-major in stored order.  parent[n] is a
 * flat index (root: -1); token[n] < 0 marks an absent node.  Siblings are
 * tested in increasing flat index.  Draft rows exist for nodes that can have
 * children, target rows for every node.
 *
 * Per sequence: cur = root; repeat { children of cur; none -> draw from
 * q(.|cur) and stop; else run the chain on (p(.|cur), q(.|cur)); first accepted
 * child becomes cur; all rejected -> draw from the last residual and stop }.
 *
 * dbg_theta/dbg_margin [B][N+1]: threshold and |U - theta| of each child that
 * was tested (NaN elsewhere).  final_margin [B]: margin of the last draw.
 * out_final_weights: optional [B][V], the normalised distribution the last
 * token was drawn from.
 */
int rsd_oracle_verify_tree_rule(int rule, double gamma, int final_sampler /* 0 inverse CDF, 1 Gumbel-Top-1 */,
                           const void* draft, int draft_dtype, int64_t draft_seq_stride, int64_t draft_row_stride,
                           double draft_temperature,
                           const void* target, int target_dtype, int64_t target_seq_stride, int64_t target_row_stride,
                           double target_temperature,
                           int B, int V, int n_nodes /* N+1 */, int num_levels,
                           const int32_t* parent, int topology_is_shared, const int32_t* token,
                           uint64_t seed, uint32_t step, uint32_t seq_base,
                           int32_t* accepted_len, int32_t* accepted_node, int32_t* accepted_token,
                           int32_t* last_token, int32_t* stop_reason,
                           double* dbg_theta, double* dbg_margin, double* final_margin, double* out_final_weights,
                           int32_t* status) {
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const int32_t* par = parent + (topology_is_shared ? 0 : (int64_t)b * n_nodes);
        const int32_t* tok = token + (int64_t)b * n_nodes;
        double* lt = (double*)malloc(sizeof(double) * (size_t)V);
        double* ld = (double*)malloc(sizeof(double) * (size_t)V);
        double* q = (double*)malloc(sizeof(double) * (size_t)V);
        double* p = (double*)malloc(sizeof(double) * (size_t)V);
        int st = 0, cur = 0, len = 0, reason = -1;
        uint32_t seq = seq_base + (uint32_t)b;
        for (int i = 0; i < num_levels; ++i) {
            accepted_node[(int64_t)b * num_levels + i] = -1;
            accepted_token[(int64_t)b * num_levels + i] = -1;
        }
        if (dbg_theta) for (int n = 0; n < n_nodes; ++n) dbg_theta[(int64_t)b * n_nodes + n] = NAN;
        if (dbg_margin) for (int n = 0; n < n_nodes; ++n) dbg_margin[(int64_t)b * n_nodes + n] = NAN;

        for (;;) {
            int n_children = 0;
            for (int c = 1; c < n_nodes; ++c) if (par[c] == cur && tok[c] >= 0) ++n_children;
            if (load_row(target, target_dtype, b * target_seq_stride + cur * target_row_stride, V, target_temperature, lt)) st |= ORC_ST_NAN_INPUT;
            softmax_row(lt, V, q);
            if (n_children == 0 || len >= num_levels) {
                reason = (len >= num_levels) ? ORC_STOP_LEAF : ORC_STOP_NO_CHILDREN;
                break;
            }
            if (load_row(draft, draft_dtype, b * draft_seq_stride + cur * draft_row_stride, V, draft_temperature, ld)) st |= ORC_ST_NAN_INPUT;
            softmax_row(ld, V, p);
            int accepted_child = -1, j = 0, alive = 1;
            for (int c = 1; c < n_nodes && alive; ++c) {
                if (par[c] != cur || tok[c] < 0) continue;
                int x = tok[c];
                double theta = (rule == 2) ? kseq_threshold(q, p, gamma, x, &st) : rrs_threshold(q, p, x, &st);
                double U = rsd_oracle_accept_uniform(seed, step, seq, (uint32_t)cur, (uint32_t)j);
                if (dbg_theta) dbg_theta[(int64_t)b * n_nodes + c] = theta;
                if (dbg_margin) dbg_margin[(int64_t)b * n_nodes + c] = fabs(U - theta);
                if (U < theta) { accepted_child = c; break; }
                if (rule == 0) alive = rrs_reject(q, p, V, x, &st);
                else if (rule == 1) multiround_reject(q, p, V, &st);
                ++j;
            }
            if (accepted_child < 0) {
                if (rule == 2) kseq_residual(q, p, V, gamma, n_children, &st);
                reason = ORC_STOP_ALL_REJECTED;
                break;
            }
            accepted_node[(int64_t)b * num_levels + len] = accepted_child;
            accepted_token[(int64_t)b * num_levels + len] = tok[accepted_child];
            ++len;
            cur = accepted_child;
        }
        double fm = 0.0;
        if (final_sampler == 1) {
            last_token[b] = gumbel_top1(q, V, seed, step, seq, (uint32_t)cur, &fm);
        } else {
            double u = rsd_oracle_resample_uniform(seed, step, seq, (uint32_t)cur);
            last_token[b] = rsd_oracle_inverse_cdf(q, V, u, &fm);
        }
        if (final_margin) final_margin[b] = fm;
        if (out_final_weights) memcpy(out_final_weights + (int64_t)b * V, q, sizeof(double) * (size_t)V);
        accepted_len[b] = len;
        stop_reason[b] = reason;
        status[b] = st;
        free(lt); free(ld); free(q); free(p);
    }
    return 0;
}

/* recursive rejection sampling (rule 0): the paper's method */
int rsd_oracle_verify_tree(const void* draft, int draft_dtype, int64_t draft_seq_stride, int64_t draft_row_stride,
                           double draft_temperature,
                           const void* target, int target_dtype, int64_t target_seq_stride, int64_t target_row_stride,
                           double target_temperature,
                           int B, int V, int n_nodes, int num_levels,
                           const int32_t* parent, int topology_is_shared, const int32_t* token,
                           uint64_t seed, uint32_t step, uint32_t seq_base,
                           int32_t* accepted_len, int32_t* accepted_node, int32_t* accepted_token,
                           int32_t* last_token, int32_t* stop_reason,
                           double* dbg_theta, double* dbg_margin, double* final_margin, double* out_final_weights,
                           int32_t* status) {
    return rsd_oracle_verify_tree_rule(0, 1.0, 0, draft, draft_dtype, draft_seq_stride, draft_row_stride, draft_temperature,
                                       target, target_dtype, target_seq_stride, target_row_stride, target_temperature,
                                       B, V, n_nodes, num_levels, parent, topology_is_shared, token, seed, step,
                                       seq_base, accepted_len, accepted_node, accepted_token, last_token, stop_reason,
                                       dbg_theta, dbg_margin, final_margin, out_final_weights, status);
}

/* ------------------------------------------------------------------------ */
/* stand-alone residual draw                                                 */
/* ------------------------------------------------------------------------ */
/*
 * For each sequence: p = softmax(draft row), q = softmax(target row); run the
 * chain over rejected[b][0..max_k) (tokens in rejection order, -1 padded), then
 * draw one token from the residual by inverse CDF with the RESAMPLE stream of
 * (sequence, rng_node[b]).  With no rejected token this is a plain draw from
 * the target row (draft may then be NULL).
 */
int rsd_oracle_resample_residual(const void* draft, int draft_dtype, int64_t draft_seq_stride, double draft_temperature,
                                 const void* target, int target_dtype, int64_t target_seq_stride,
                                 double target_temperature,
                                 int B, int V, const int32_t* rejected, int max_k, const int32_t* rng_node,
                                 uint64_t seed, uint32_t step, uint32_t seq_base,
                                 int32_t* out_token, double* out_residual, double* out_margin, int32_t* status) {
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        double* l = (double*)malloc(sizeof(double) * (size_t)V);
        double* q = (double*)malloc(sizeof(double) * (size_t)V);
        double* p = (double*)malloc(sizeof(double) * (size_t)V);
        int st = 0;
        if (load_row(target, target_dtype, b * target_seq_stride, V, target_temperature, l)) st |= ORC_ST_NAN_INPUT;
        softmax_row(l, V, q);
        int n_rej = 0;
        for (int i = 0; i < max_k; ++i) if (rejected && rejected[(int64_t)b * max_k + i] >= 0) ++n_rej;
        if (n_rej > 0) {
            if (load_row(draft, draft_dtype, b * draft_seq_stride, V, draft_temperature, l)) st |= ORC_ST_NAN_INPUT;
            softmax_row(l, V, p);
            for (int i = 0; i < max_k; ++i) {
                int x = rejected[(int64_t)b * max_k + i];
                if (x < 0) continue;
                if (!rrs_reject(q, p, V, x, &st)) break;
            }
        }
        double u = rsd_oracle_resample_uniform(seed, step, seq_base + (uint32_t)b, (uint32_t)rng_node[b]);
        double m = 0.0;
        out_token[b] = rsd_oracle_inverse_cdf(q, V, u, &m);
        if (out_margin) out_margin[b] = m;
        if (out_residual) memcpy(out_residual + (int64_t)b * V, q, sizeof(double) * (size_t)V);
        status[b] = st;
        free(l); free(q); free(p);
    }
    return 0;
}
