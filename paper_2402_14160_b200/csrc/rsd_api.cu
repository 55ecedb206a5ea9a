// C ABI of librsd (declared in include/rsd.h), drafting half: argument checks and kernel launches, nothing else.
// The verification entry points are in rsd_api_verify.cu (two translation units keep each compile small).
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>

#include "rsd_api_common.h"
#include "rsd_scan.cuh"
#include "rsd_filter.cuh"

namespace rsd_host {
thread_local char g_err[512] = "";
}
using namespace rsd_host;

namespace {

thread_local cudaEvent_t g_scan_before = nullptr, g_scan_after = nullptr;  // one-shot, see rsd_profile_next_scan

template <typename T, bool ALIGNED, bool WIDE, bool NEED_LSE, bool TEMP>
void launch_scan_temp(int blocks, const rsd::ScanArgs& a, cudaStream_t s) {
    const size_t smem = sizeof(float) * (size_t)((((a.V + 15) / 16) + 3) / 4 * 4);  // one bound per group of 16 elements, padded to fours
    if (smem > 48 * 1024) {
        // The attribute belongs to the (function, device) pair; it is only needed beyond 48 KB (V > 196,608), so it
        // is simply set on every such launch instead of being remembered per device.
        if (cudaFuncSetAttribute(rsd::scan_topk_kernel<T, ALIGNED, WIDE, NEED_LSE, TEMP>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(sizeof(float) * (RSD_MAX_VOCAB / 16))) != cudaSuccess)
            return;   // the error stays pending: the caller's check_launch() reports it
    }
    rsd::scan_topk_kernel<T, ALIGNED, WIDE, NEED_LSE, TEMP><<<blocks, rsd::kScanThreads, smem, s>>>(a);
}

template <typename T, bool ALIGNED, bool WIDE, bool NEED_LSE>
void launch_scan_one(int blocks, const rsd::ScanArgs& a, cudaStream_t s) {
    if (a.temp != 1.0f) launch_scan_temp<T, ALIGNED, WIDE, NEED_LSE, true>(blocks, a, s);
    else launch_scan_temp<T, ALIGNED, WIDE, NEED_LSE, false>(blocks, a, s);
}

template <bool NEED_LSE>
void launch_scan_lse(const rsd_rows* rows, int align, int blocks, const rsd::ScanArgs& a, cudaStream_t s) {
    if (rows->dtype == RSD_F32) {
        if (align == 32) launch_scan_one<float, true, true, NEED_LSE>(blocks, a, s);
        else if (align == 16) launch_scan_one<float, true, false, NEED_LSE>(blocks, a, s);
        else launch_scan_one<float, false, false, NEED_LSE>(blocks, a, s);
    } else {
        if (align == 32) launch_scan_one<__nv_bfloat16, true, true, NEED_LSE>(blocks, a, s);
        else if (align == 16) launch_scan_one<__nv_bfloat16, true, false, NEED_LSE>(blocks, a, s);
        else launch_scan_one<__nv_bfloat16, false, false, NEED_LSE>(blocks, a, s);
    }
}

void launch_scan(const rsd_rows* rows, bool need_lse, int blocks, rsd::ScanArgs& a, cudaStream_t s) {
    // vector paths: rows made of whole groups that start on 32- or 16-byte boundaries
    const int aligned = a.V % 16 != 0 ? 0 : rows_aligned(rows, 32) ? 32 : rows_aligned(rows, 16) ? 16 : 0;
    for (int r = 0; r < 10; ++r) {
        a.rk0[r] = a.seed_lo + (uint32_t)r * 0x9E3779B9u;
        a.rk1[r] = a.seed_hi + (uint32_t)r * 0xBB67AE85u;
    }
    if (g_scan_before) cudaEventRecord(g_scan_before, s);
    if (need_lse) launch_scan_lse<true>(rows, aligned, blocks, a, s);
    else launch_scan_lse<false>(rows, aligned, blocks, a, s);
    if (g_scan_after) cudaEventRecord(g_scan_after, s);
    g_scan_before = g_scan_after = nullptr;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

extern "C" {

int rsd_version(void) { return 100; }
int rsd_rng_layout(void) { return 3; }
const char* rsd_last_error(void) { return g_err; }

int rsd_profile_next_scan(void* before, void* after) {
    g_scan_before = (cudaEvent_t)before;
    g_scan_after = (cudaEvent_t)after;
    return RSD_OK;
}

int rsd_gumbel_topk_draft(const rsd_rows* draft, int B, int R, int V, const int32_t* k_per_row, const int32_t* rng_node,
                          int max_k, uint64_t seed, uint32_t step, uint32_t seq_base, int32_t* out_token,
                          float* out_perturbed, float* out_logprob, const int32_t* child_base, int32_t* node_token,
                          int node_stride, int32_t* status, rsd_stream_t stream) {
    g_err[0] = 0;
    if (int e = check_vocab(V)) return e;
    if (int e = check_rows("draft", draft, V, R > 1)) return e;
    if (B < 0 || R < 1) return fail(RSD_ERR_INVALID_ARG, "B = %d, R = %d", B, R);
    if (R > RSD_MAX_ROWS_PER_SEQ) return fail(RSD_ERR_UNSUPPORTED, "R = %d > %d", R, (int)RSD_MAX_ROWS_PER_SEQ);
    if (max_k < 1 || max_k > RSD_MAX_K) return fail(RSD_ERR_UNSUPPORTED, "max_k = %d outside [1, %d]", max_k, (int)RSD_MAX_K);
    if (!k_per_row || !rng_node || !out_token || !status) return fail(RSD_ERR_INVALID_ARG, "null argument");
    if ((int64_t)B * R > 0x7FFFFFFF) return fail(RSD_ERR_UNSUPPORTED, "B * R too large");
    rsd::ScanArgs a;
    memset(&a, 0, sizeof(a));
    for (int r = 0; r < R; ++r) {
        if (k_per_row[r] < 1 || k_per_row[r] > max_k) return fail(RSD_ERR_INVALID_ARG, "k_per_row[%d] = %d outside [1, max_k]", r, k_per_row[r]);
        if (rng_node[r] < 0 || rng_node[r] >= (1 << 28)) return fail(RSD_ERR_INVALID_ARG, "rng_node[%d] = %d outside [0, 2^28)", r, rng_node[r]);
        a.k_row[r] = (uint8_t)k_per_row[r];
        a.node_row[r] = rng_node[r];
        if (node_token) {
            if (!child_base) return fail(RSD_ERR_INVALID_ARG, "node_token needs child_base");
            if (child_base[r] < 0 || child_base[r] + k_per_row[r] > node_stride)
                return fail(RSD_ERR_INVALID_ARG, "child_base[%d] = %d: children fall outside [0, node_stride = %d)", r, child_base[r], node_stride);
            a.child_base[r] = child_base[r];
        }
    }
    if (B == 0) return RSD_OK;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t) * (size_t)B, s) != cudaSuccess) return check_launch("memset(status)");
    a.data = draft->data; a.seq_stride = draft->seq_stride; a.row_stride = draft->row_stride;
    a.R = R; a.V = V; a.max_k = max_k;
    a.seed_lo = (uint32_t)seed; a.seed_hi = (uint32_t)(seed >> 32); a.step = step; a.seq_base = seq_base;
    a.subtract_lse = 1;
    a.out_token = out_token; a.out_perturbed = out_perturbed; a.out_value = out_logprob; a.out_lse = nullptr;
    a.status = status; a.node_token = node_token; a.node_stride = node_stride;
    a.temp = temperature_of(draft); a.inv_temp = 1.0f / a.temp;
    const bool need_lse = !rows_are_logprob(draft) && (out_perturbed || out_logprob);
    launch_scan(draft, need_lse, B * R, a, s);
    return check_launch("rsd_gumbel_topk_draft");
}

size_t rsd_sbs_workspace_bytes(int B, int n_par, int W) {
    if (B < 0 || n_par < 1 || W < 1) return 0;
    const size_t f = (size_t)B * n_par * W;
    return align_up(f * 4, 256) * 3 + align_up((size_t)B * n_par * 4, 256) * 2;
}

int rsd_sbs_step(const rsd_rows* draft_level, int B, int n_par, int V, int W, int32_t first_parent_node,
                 const float* sum_logprob_in, const float* trunc_gumbel_in, uint64_t seed, uint32_t step,
                 uint32_t seq_base, int32_t* out_token, int32_t* out_parent, int64_t out_stride, int32_t parent_base,
                 float* sum_logprob_out, float* trunc_gumbel_out, int32_t* out_count, int32_t* status, void* ws,
                 size_t ws_bytes, rsd_stream_t stream) {
    g_err[0] = 0;
    if (int e = check_vocab(V)) return e;
    if (int e = check_rows("draft_level", draft_level, V, n_par > 1)) return e;
    if (B < 0 || n_par < 1) return fail(RSD_ERR_INVALID_ARG, "B = %d, n_par = %d", B, n_par);
    if (n_par > RSD_MAX_ROWS_PER_SEQ) return fail(RSD_ERR_UNSUPPORTED, "n_par = %d > %d", n_par, (int)RSD_MAX_ROWS_PER_SEQ);
    if (W < 1 || W > RSD_MAX_K) return fail(RSD_ERR_UNSUPPORTED, "W = %d outside [1, %d]", W, (int)RSD_MAX_K);
    if (n_par * W > 1024) return fail(RSD_ERR_UNSUPPORTED, "n_par * W = %d > 1024", n_par * W);
    if (first_parent_node < 0 || (int64_t)first_parent_node + n_par > (1 << 28)) return fail(RSD_ERR_INVALID_ARG, "first_parent_node out of range");
    if (!out_token || !out_parent || !sum_logprob_out || !trunc_gumbel_out || !out_count || !status) return fail(RSD_ERR_INVALID_ARG, "null output");
    if (out_stride < W) return fail(RSD_ERR_INVALID_ARG, "out_stride = %lld < W = %d", (long long)out_stride, W);
    if (parent_base < 0) return fail(RSD_ERR_INVALID_ARG, "parent_base = %d", parent_base);
    if ((int64_t)B * n_par > 0x7FFFFFFF) return fail(RSD_ERR_UNSUPPORTED, "B * n_par too large");
    if (B == 0) return RSD_OK;
    const size_t need = rsd_sbs_workspace_bytes(B, n_par, W);
    if (!ws || ws_bytes < need) return fail(RSD_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
    if ((uintptr_t)ws % 256 != 0) return fail(RSD_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    cudaStream_t s = (cudaStream_t)stream;

    const size_t f = (size_t)B * n_par * W;
    char* w = (char*)ws;
    int32_t* fin_token = (int32_t*)w;
    float* fin_value = (float*)(w + align_up(f * 4, 256));
    float* fin_pert = (float*)(w + 2 * align_up(f * 4, 256));
    float* fin_lse = (float*)(w + 3 * align_up(f * 4, 256));
    int32_t* row_status = (int32_t*)(w + 3 * align_up(f * 4, 256) + align_up((size_t)B * n_par * 4, 256));

    rsd::ScanArgs a;
    memset(&a, 0, sizeof(a));
    for (int r = 0; r < n_par; ++r) { a.k_row[r] = (uint8_t)W; a.node_row[r] = first_parent_node + r; }
    a.data = draft_level->data; a.seq_stride = draft_level->seq_stride; a.row_stride = draft_level->row_stride;
    a.R = n_par; a.V = V; a.max_k = W;
    a.seed_lo = (uint32_t)seed; a.seed_hi = (uint32_t)(seed >> 32); a.step = step; a.seq_base = seq_base;
    a.subtract_lse = 0;
    a.out_token = fin_token; a.out_perturbed = fin_pert; a.out_value = fin_value; a.out_lse = fin_lse;
    a.status = status; a.row_status = row_status;   // status[b] is written by the epilogue
    a.temp = temperature_of(draft_level); a.inv_temp = 1.0f / a.temp; a.raw_values = 1;
    launch_scan(draft_level, !rows_are_logprob(draft_level), B * n_par, a, s);
    if (int e = check_launch("rsd_sbs_step(scan)")) return e;

    rsd::SbsEpilogueArgs e;
    e.n_par = n_par; e.W = W; e.is_logprob = rows_are_logprob(draft_level);
    e.fin_seq_stride = (int64_t)n_par * W; e.row_seq_stride = n_par; e.state_stride = n_par; e.out_state_stride = W; e.inv_temp = 1.0 / (double)temperature_of(draft_level); e.first_parent_node = first_parent_node;
    e.seed_lo = (uint32_t)seed; e.seed_hi = (uint32_t)(seed >> 32); e.step = step; e.seq_base = seq_base;
    e.fin_token = fin_token; e.fin_value = fin_value; e.fin_pert = fin_pert; e.fin_lse = fin_lse;
    e.row_status = row_status;
    e.sum_in = sum_logprob_in; e.gamma_in = trunc_gumbel_in;
    e.out_token = out_token; e.out_parent = out_parent; e.out_stride = out_stride; e.parent_base = parent_base;
    e.sum_out = sum_logprob_out; e.gamma_out = trunc_gumbel_out;
    e.out_count = out_count; e.status = status;
    const size_t smem = rsd::sbs_level_scratch_bytes(n_par, W);
    rsd::sbs_epilogue_kernel<<<B, rsd::kEpilogueThreads, smem, s>>>(e);
    return check_launch("rsd_sbs_step(epilogue)");
}


int rsd_filter_rows(const rsd_rows* rows, int B, int R, int V, int top_k, float top_p, void* out_rows, int32_t* out_kept,
                    int32_t* status, rsd_stream_t stream) {
    g_err[0] = 0;
    if (int e = check_vocab(V)) return e;
    if (int e = check_rows("rows", rows, V, R > 1)) return e;
    if (B < 0 || R < 1) return fail(RSD_ERR_INVALID_ARG, "B = %d, R = %d", B, R);
    if (top_k < 0) return fail(RSD_ERR_INVALID_ARG, "top_k = %d must be >= 0 (0: none)", top_k);
    if (!(top_p > 0.0f)) return fail(RSD_ERR_INVALID_ARG, "top_p = %g must be > 0 (>= 1: none)", (double)top_p);
    if (!out_rows || !status) return fail(RSD_ERR_INVALID_ARG, "null output");
    if ((int64_t)B * R > 0x7FFFFFFF) return fail(RSD_ERR_UNSUPPORTED, "B * R too large");
    const size_t elem = rows->dtype == RSD_F32 ? 4 : 2;
    const size_t smem = (size_t)V * elem + 16;
    constexpr size_t kSharedPerBlock = 227 * 1024;
    if (smem + sizeof(rsd::FilterSmem) + 256 > kSharedPerBlock)
        return fail(RSD_ERR_UNSUPPORTED, "rows of %d %zu-byte entries do not fit in shared memory (at most %zu entries)", V, elem,
                    (kSharedPerBlock - sizeof(rsd::FilterSmem) - 272) / elem);
    if (B == 0) return RSD_OK;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(status, 0, sizeof(int32_t) * (size_t)B, s) != cudaSuccess) return check_launch("memset(status)");
    rsd::FilterArgs a;
    a.data = rows->data; a.out = out_rows; a.seq_stride = rows->seq_stride; a.row_stride = rows->row_stride;
    a.R = R; a.V = V; a.top_k = top_k; a.top_p = top_p;
    a.log2e_over_t = rsd::kLog2e / temperature_of(rows);
    a.kept = out_kept; a.status = status;
    // the attribute belongs to the (function, device) pair: raised once per device to the largest row that fits
    static std::atomic<bool> raised[2][64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return check_launch("cudaGetDevice");
    const int which = rows->dtype == RSD_F32 ? 0 : 1;
    if (dev < 0 || dev >= 64 || !raised[which][dev].load(std::memory_order_acquire)) {
        const int most = (int)(kSharedPerBlock - sizeof(rsd::FilterSmem) - 256);
        const cudaError_t e = rows->dtype == RSD_F32
                                  ? cudaFuncSetAttribute(rsd::filter_rows_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, most)
                                  : cudaFuncSetAttribute(rsd::filter_rows_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
        if (e != cudaSuccess) return check_launch("cudaFuncSetAttribute");
        if (dev >= 0 && dev < 64) raised[which][dev].store(true, std::memory_order_release);
    }
    if (rows->dtype == RSD_F32) rsd::filter_rows_kernel<float><<<B * R, rsd::kFilterThreads, smem, s>>>(a);
    else rsd::filter_rows_kernel<__nv_bfloat16><<<B * R, rsd::kFilterThreads, smem, s>>>(a);
    return check_launch("rsd_filter_rows");
}

size_t rsd_sbs_tree_workspace_bytes(int B, int W, int L) {
    if (B < 0 || W < 1 || L < 1) return 0;
    const size_t P = 1 + (size_t)(L - 1) * W;
    const size_t f = (size_t)B * P * W;
    return align_up(f * 4, 256) * 3 + align_up((size_t)B * P * 4, 256) * 2   // finalists; log-sum-exp, row status
           + align_up((size_t)B * W * 4, 256) * 4                            // two (sum, truncated Gumbel) states
           + align_up((size_t)B * L * 4, 256);                               // status of every level
}

int rsd_sbs_draft_tree(const rsd_rows* draft, int B, int V, int W, int L, uint64_t seed, uint32_t step,
                       uint32_t seq_base, int32_t* node_token, int32_t* node_parent, int64_t node_stride,
                       float* sum_logprob_out, float* trunc_gumbel_out, int32_t* level_count, int32_t* status, void* ws,
                       size_t ws_bytes, rsd_stream_t stream) {
    g_err[0] = 0;
    if (int e = check_vocab(V)) return e;
    if (W < 1 || W > RSD_MAX_K) return fail(RSD_ERR_UNSUPPORTED, "W = %d outside [1, %d]", W, (int)RSD_MAX_K);
    if (L < 1) return fail(RSD_ERR_INVALID_ARG, "L = %d", L);
    const int64_t P = 1 + (int64_t)(L - 1) * W;
    if (P > RSD_MAX_ROWS_PER_SEQ) return fail(RSD_ERR_UNSUPPORTED, "1 + (L - 1) W = %lld parent rows > %d", (long long)P, (int)RSD_MAX_ROWS_PER_SEQ);
    if (W * W > 1024) return fail(RSD_ERR_UNSUPPORTED, "W * W = %d > 1024", W * W);
    if (int e = check_rows("draft", draft, V, P > 1)) return e;
    if (B < 0) return fail(RSD_ERR_INVALID_ARG, "B = %d", B);
    if (!node_token || !node_parent || !level_count || !status) return fail(RSD_ERR_INVALID_ARG, "null output");
    if (node_stride < 1 + (int64_t)L * W) return fail(RSD_ERR_INVALID_ARG, "node_stride = %lld < 1 + L W = %lld", (long long)node_stride, (long long)(1 + (int64_t)L * W));
    if (B * P > 0x7FFFFFFF) return fail(RSD_ERR_UNSUPPORTED, "B * rows too large");
    if (B == 0) return RSD_OK;
    const size_t need = rsd_sbs_tree_workspace_bytes(B, W, L);
    if (!ws || ws_bytes < need) return fail(RSD_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
    if ((uintptr_t)ws % 256 != 0) return fail(RSD_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    cudaStream_t s = (cudaStream_t)stream;

    const size_t f4 = align_up((size_t)B * P * W * 4, 256), r4 = align_up((size_t)B * P * 4, 256), s4 = align_up((size_t)B * W * 4, 256);
    char* w = (char*)ws;
    int32_t* fin_token = (int32_t*)w;
    float* fin_value = (float*)(w + f4);
    float* fin_pert = (float*)(w + 2 * f4);
    float* fin_lse = (float*)(w + 3 * f4);
    int32_t* row_status = (int32_t*)(w + 3 * f4 + r4);
    char* st0 = w + 3 * f4 + 2 * r4;
    int32_t* level_status = (int32_t*)(st0 + 4 * s4);

    // one scan over the parent rows of every level: row r of a sequence is flat node r
    rsd::ScanArgs a;
    memset(&a, 0, sizeof(a));
    for (int r = 0; r < (int)P; ++r) { a.k_row[r] = (uint8_t)W; a.node_row[r] = r; }
    a.data = draft->data; a.seq_stride = draft->seq_stride; a.row_stride = draft->row_stride;
    a.R = (int)P; a.V = V; a.max_k = W;
    a.seed_lo = (uint32_t)seed; a.seed_hi = (uint32_t)(seed >> 32); a.step = step; a.seq_base = seq_base;
    a.subtract_lse = 0;
    a.out_token = fin_token; a.out_perturbed = fin_pert; a.out_value = fin_value; a.out_lse = fin_lse;
    a.status = status; a.row_status = row_status;
    a.temp = temperature_of(draft); a.inv_temp = 1.0f / a.temp; a.raw_values = 1;
    launch_scan(draft, !rows_are_logprob(draft), (int)(B * P), a, s);
    if (int e = check_launch("rsd_sbs_draft_tree(scan)")) return e;

    rsd::SbsChainArgs c;
    memset(&c, 0, sizeof(c));
    c.lvl.W = W; c.lvl.is_logprob = rows_are_logprob(draft); c.lvl.inv_temp = 1.0 / (double)temperature_of(draft);
    c.lvl.fin_seq_stride = P * W; c.lvl.row_seq_stride = P; c.lvl.state_stride = W;
    c.lvl.seed_lo = (uint32_t)seed; c.lvl.seed_hi = (uint32_t)(seed >> 32); c.lvl.step = step; c.lvl.seq_base = seq_base;
    c.lvl.fin_token = fin_token; c.lvl.fin_value = fin_value; c.lvl.fin_pert = fin_pert; c.lvl.fin_lse = fin_lse;
    c.lvl.row_status = row_status;
    c.L = L; c.P = (int)P; c.B = B;
    c.node_token = node_token; c.node_parent = node_parent; c.node_stride = node_stride;
    c.level_count = level_count; c.level_status = level_status; c.status = status;
    c.sum_out = sum_logprob_out; c.gamma_out = trunc_gumbel_out;
    // the finalists of a sequence are staged in shared memory when they fit well inside the default 48 KB
    c.staged = rsd::sbs_chain_smem_bytes(W, (int)P, true) <= 40 * 1024 ? 1 : 0;
    const size_t smem = rsd::sbs_chain_smem_bytes(W, (int)P, c.staged != 0);
    rsd::sbs_chain_kernel<<<B, rsd::kEpilogueThreads, smem, s>>>(c);
    return check_launch("rsd_sbs_draft_tree(levels)");
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------
// rsd_sbs_step_static: the same level of Stochastic Beam Search with built-in scratch, for callers that must not
// allocate.  The array below lives in the library's device image on every GPU that loads it.  In host code its
// name is only a handle: the device address has to be asked for, once per device, with that device current.
// ---------------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_sbs_static_scratch[RSD_SBS_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_scratch_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on the current device (looked up on the first call per device).
int static_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(RSD_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(RSD_ERR_UNSUPPORTED, "device index %d outside [0, %d)", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_sbs_static_scratch);
        if (e != cudaSuccess || !p) return fail(RSD_ERR_CUDA, "cudaGetSymbolAddress(built-in scratch): %s", cudaGetErrorString(e));
        g_static_scratch_ptr[dev] = p;
    }
    *out = g_static_scratch_ptr[dev];
    return RSD_OK;
}
}  // namespace

extern "C" int rsd_sbs_step_static(const rsd_rows* draft_level, int B, int n_par, int V, int W, int32_t first_parent_node,
                                   const float* sum_logprob_in, const float* trunc_gumbel_in, uint64_t seed,
                                   uint32_t step, uint32_t seq_base, int32_t* out_token, int32_t* out_parent,
                                   int64_t out_stride, int32_t parent_base, float* sum_logprob_out,
                                   float* trunc_gumbel_out, int32_t* out_count, int32_t* status, rsd_stream_t stream) {
    g_err[0] = 0;
    // the argument errors rsd_sbs_step would report come first, so that an oversized n_par or W is named as such
    if (B < 0 || n_par < 1 || W < 1) return fail(RSD_ERR_INVALID_ARG, "B = %d, n_par = %d, W = %d", B, n_par, W);
    if (n_par > RSD_MAX_ROWS_PER_SEQ) return fail(RSD_ERR_UNSUPPORTED, "n_par = %d > %d", n_par, (int)RSD_MAX_ROWS_PER_SEQ);
    if (W > RSD_MAX_K) return fail(RSD_ERR_UNSUPPORTED, "W = %d outside [1, %d]", W, (int)RSD_MAX_K);
    if (n_par * W > 1024) return fail(RSD_ERR_UNSUPPORTED, "n_par * W = %d > 1024", n_par * W);
    const size_t need = rsd_sbs_workspace_bytes(B, n_par, W);
    if (need > (size_t)RSD_SBS_STATIC_SCRATCH_BYTES)
        return fail(RSD_ERR_WORKSPACE,
                    "B = %d, n_par = %d, W = %d needs %zu bytes of scratch, the built-in scratch holds %d: "
                    "split the batch or use rsd_sbs_step with your own scratch",
                    B, n_par, W, need, (int)RSD_SBS_STATIC_SCRATCH_BYTES);
    void* scratch = nullptr;
    if (int e = static_scratch_address(&scratch)) return e;
    // nothing in the scratch has to be cleared: the scan writes every finalist slot and every row's log-sum-exp
    // before the epilogue reads them
    return rsd_sbs_step(draft_level, B, n_par, V, W, first_parent_node, sum_logprob_in, trunc_gumbel_in, seed, step,
                        seq_base, out_token, out_parent, out_stride, parent_base, sum_logprob_out, trunc_gumbel_out,
                        out_count, status, scratch, (size_t)RSD_SBS_STATIC_SCRATCH_BYTES, stream);
}
