// C ABI of librsd (declared in include/rsd.h), verification half: rsd_verify_tree, rsd_verify_tree_rule and
// rsd_resample_residual.  Argument checks and kernel launches, nothing else.
#include <atomic>

#include "rsd_api_common.h"
#include "rsd_verify.cuh"
#include "rsd_walk_ring.cuh"

using namespace rsd_host;

namespace {
// SMs of the current device (asked once per device; 148 if the query fails)
int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        cached[dev] = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
    }
    return cached[dev];
}

// The walk fed by the copy engine (rsd_walk_ring.cuh); a launch error stays pending for check_launch().
template <typename T>
void launch_ring_walk(const rsd::VerifyArgs& a, int B, cudaStream_t s) {
    using namespace rsd::walk_ring;
    // The attribute belongs to the (function, device) pair and setting it costs host time: once per device.
    static std::atomic<bool> raised[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return;
    if (dev < 0 || dev >= 64 || !raised[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(verify_tree_ring_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes) != cudaSuccess)
            return;
        if (dev >= 0 && dev < 64) raised[dev].store(true, std::memory_order_release);
    }
    verify_tree_ring_kernel<T><<<B, kThreads, kRingBytes, s>>>(a);
}
}  // namespace

extern "C" {

int rsd_verify_tree(const rsd_rows* draft, const rsd_rows* target, const rsd_tree* tree, int B, int V, uint64_t seed,
                    uint32_t step, uint32_t seq_base, int32_t* accepted_len, int32_t* accepted_node,
                    int32_t* accepted_token, int32_t* last_token, int32_t* stop_reason, float* dbg_theta,
                    int32_t* status, rsd_stream_t stream) {
    return rsd_verify_tree_rule(draft, target, tree, B, V, RSD_RULE_RRS, 1.0f, RSD_FINAL_INVERSE_CDF, seed, step, seq_base, accepted_len,
                                accepted_node, accepted_token, last_token, stop_reason, dbg_theta, status, stream);
}

int rsd_verify_tree_rule(const rsd_rows* draft, const rsd_rows* target, const rsd_tree* tree, int B, int V, int rule,
                         float gamma, int final_sampler, uint64_t seed, uint32_t step, uint32_t seq_base, int32_t* accepted_len,
                         int32_t* accepted_node, int32_t* accepted_token, int32_t* last_token, int32_t* stop_reason,
                         float* dbg_theta, int32_t* status, rsd_stream_t stream) {
    g_err[0] = 0;
    if (rule != RSD_RULE_RRS && rule != RSD_RULE_MULTIROUND && rule != RSD_RULE_KSEQ)
        return fail(RSD_ERR_INVALID_ARG, "unknown verification rule %d", rule);
    if (final_sampler != RSD_FINAL_INVERSE_CDF && final_sampler != RSD_FINAL_GUMBEL_TOP1)
        return fail(RSD_ERR_INVALID_ARG, "unknown sampler of the last token %d", final_sampler);
    if (rule == RSD_RULE_KSEQ && !(gamma >= 1.0f && gamma < 3.0e38f))
        return fail(RSD_ERR_INVALID_ARG, "K-SEQ: gamma = %g must be a finite number >= 1", (double)gamma);
    if (int e = check_vocab(V)) return e;
    if (int e = check_rows("draft", draft, V, true)) return e;
    if (int e = check_rows("target", target, V, true)) return e;
    if (draft->dtype != target->dtype) return fail(RSD_ERR_UNSUPPORTED, "draft and target rows must have the same dtype");
    if (!tree || !tree->parent || !tree->token) return fail(RSD_ERR_INVALID_ARG, "null tree");
    if (tree->num_levels < 0 || tree->num_nodes < 1 || tree->num_nodes > RSD_MAX_TREE_NODES)
        return fail(RSD_ERR_UNSUPPORTED, "num_levels = %d, num_nodes = %d", tree->num_levels, tree->num_nodes);
    if (B < 0) return fail(RSD_ERR_INVALID_ARG, "B = %d", B);
    if (!accepted_len || !accepted_node || !accepted_token || !last_token || !stop_reason || !status) return fail(RSD_ERR_INVALID_ARG, "null output");
    if (B == 0) return RSD_OK;
    rsd::VerifyArgs a;
    a.draft = {draft->data, draft->seq_stride, draft->row_stride, 1.0f / temperature_of(draft)};
    a.target = {target->data, target->seq_stride, target->row_stride, 1.0f / temperature_of(target)};
    a.V = V; a.L = tree->num_levels; a.num_nodes = tree->num_nodes; a.shared_topology = tree->topology_is_shared;
    a.rule = rule; a.gamma = rule == RSD_RULE_KSEQ ? gamma : 1.0f; a.final_sampler = final_sampler;
    a.parent = tree->parent; a.token = tree->token;
    a.seed_lo = (uint32_t)seed; a.seed_hi = (uint32_t)(seed >> 32); a.step = step; a.seq_base = seq_base;
    a.accepted_len = accepted_len; a.accepted_node = accepted_node; a.accepted_token = accepted_token;
    a.last_token = last_token; a.stop_reason = stop_reason; a.dbg_theta = dbg_theta; a.status = status;
    cudaStream_t s = (cudaStream_t)stream;
    const bool aligned = rows_aligned(draft) && rows_aligned(target);
    // at most one sequence per SM: blocks of 512 threads; otherwise blocks of 256
#define RSD_LAUNCH_WALK(NS, BASELINES)                                                                                   \
    do {                                                                                                                 \
        using namespace rsd::NS;                                                                                         \
        if (draft->dtype == RSD_F32) {                                                                                   \
            if (aligned) verify_tree_kernel<float, true, BASELINES><<<B, kVerifyThreads, 0, s>>>(a);                     \
            else verify_tree_kernel<float, false, BASELINES><<<B, kVerifyThreads, 0, s>>>(a);                            \
        } else {                                                                                                         \
            if (aligned) verify_tree_kernel<__nv_bfloat16, true, BASELINES><<<B, kVerifyThreads, 0, s>>>(a);             \
            else verify_tree_kernel<__nv_bfloat16, false, BASELINES><<<B, kVerifyThreads, 0, s>>>(a);                    \
        }                                                                                                                \
    } while (0)
    const bool wide_blocks = B <= sm_count();
    if (rule == RSD_RULE_RRS && final_sampler == RSD_FINAL_INVERSE_CDF) {
        // rows on 16-byte boundaries, of at most 64 chunks (the ring keeps its chunks as bits of one word): the walk
        // whose passes are fed by the copy engine
        const size_t row_bytes = (size_t)V * (draft->dtype == RSD_F32 ? 4 : 2);
        if (aligned && (row_bytes + rsd::walk_ring::kRowChunkBytes - 1) / rsd::walk_ring::kRowChunkBytes <= 64) {
            if (draft->dtype == RSD_F32) launch_ring_walk<float>(a, B, s);
            else launch_ring_walk<__nv_bfloat16>(a, B, s);
        }
        else if (wide_blocks) RSD_LAUNCH_WALK(walk_wide, false);
        else RSD_LAUNCH_WALK(walk_narrow, false);
    } else {
        RSD_LAUNCH_WALK(walk_narrow, true);
    }
#undef RSD_LAUNCH_WALK
    return check_launch("rsd_verify_tree_rule");
}

int rsd_resample_residual(const rsd_rows* draft_row, const rsd_rows* target_row, int B, int V, const int32_t* rejected,
                          int max_k, const int32_t* rng_node, uint64_t seed, uint32_t step, uint32_t seq_base,
                          int32_t* out_token, float* out_residual, int32_t* status, rsd_stream_t stream) {
    g_err[0] = 0;
    if (int e = check_vocab(V)) return e;
    if (int e = check_rows("target_row", target_row, V, false)) return e;
    if (rejected) {
        if (int e = check_rows("draft_row", draft_row, V, false)) return e;
        if (draft_row->dtype != target_row->dtype) return fail(RSD_ERR_UNSUPPORTED, "draft and target rows must have the same dtype");
        if (max_k < 1 || max_k > RSD_MAX_K) return fail(RSD_ERR_UNSUPPORTED, "max_k = %d outside [1, %d]", max_k, (int)RSD_MAX_K);
    }
    if (B < 0) return fail(RSD_ERR_INVALID_ARG, "B = %d", B);
    if (!rng_node || !out_token || !status) return fail(RSD_ERR_INVALID_ARG, "null argument");
    if (B == 0) return RSD_OK;
    rsd::ResampleArgs a;
    a.target = {target_row->data, target_row->seq_stride, 0, 1.0f / temperature_of(target_row)};
    a.draft = rejected ? rsd::RowsDev{draft_row->data, draft_row->seq_stride, 0, 1.0f / temperature_of(draft_row)} : a.target;
    a.V = V; a.max_k = rejected ? max_k : 0; a.rejected = rejected; a.rng_node = rng_node;
    a.seed_lo = (uint32_t)seed; a.seed_hi = (uint32_t)(seed >> 32); a.step = step; a.seq_base = seq_base;
    a.out_token = out_token; a.out_residual = out_residual; a.status = status;
    cudaStream_t s = (cudaStream_t)stream;
    const bool aligned = rows_aligned(target_row) && (!rejected || rows_aligned(draft_row));
    using namespace rsd::walk_narrow;
    if (target_row->dtype == RSD_F32) {
        if (aligned) resample_residual_kernel<float, true><<<B, kVerifyThreads, 0, s>>>(a);
        else resample_residual_kernel<float, false><<<B, kVerifyThreads, 0, s>>>(a);
    } else {
        if (aligned) resample_residual_kernel<__nv_bfloat16, true><<<B, kVerifyThreads, 0, s>>>(a);
        else resample_residual_kernel<__nv_bfloat16, false><<<B, kVerifyThreads, 0, s>>>(a);
    }
    return check_launch("rsd_resample_residual");
}

}  // extern "C"
