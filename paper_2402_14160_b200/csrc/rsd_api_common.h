// Host-side helpers shared by the translation units of librsd: the per-thread error message and argument checks.
#pragma once
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include <cuda_runtime.h>

#include "../../include/rsd.h"

namespace rsd_host {

extern thread_local char g_err[512];   // defined in rsd_api.cu

inline int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

inline int check_launch(const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(RSD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return RSD_OK;
}

inline int check_rows(const char* name, const rsd_rows* r, int V, bool need_row_stride) {
    if (!r || !r->data) return fail(RSD_ERR_INVALID_ARG, "%s: null rows", name);
    if (r->dtype != RSD_F32 && r->dtype != RSD_BF16) return fail(RSD_ERR_UNSUPPORTED, "%s: unknown dtype %d", name, r->dtype);
    if (need_row_stride && r->row_stride < V) return fail(RSD_ERR_INVALID_ARG, "%s: row_stride %lld < V %d", name, (long long)r->row_stride, V);
    if (r->seq_stride < 0 || r->row_stride < 0) return fail(RSD_ERR_INVALID_ARG, "%s: negative stride", name);
    if (!(r->temperature >= 0.0f) || r->temperature > 3.0e38f)
        return fail(RSD_ERR_INVALID_ARG, "%s: temperature %g must be a finite number >= 0 (0 or 1: none)", name, (double)r->temperature);
    return RSD_OK;
}

// temperature that applies (1 when the rows ask for none)
inline float temperature_of(const rsd_rows* r) { return (r->temperature > 0.0f && r->temperature != 1.0f) ? r->temperature : 1.0f; }
// rows usable as log-probabilities as they are: flagged so and not re-scored by a temperature
inline bool rows_are_logprob(const rsd_rows* r) { return r->is_logprob && temperature_of(r) == 1.0f; }

inline bool rows_aligned(const rsd_rows* r, int bytes = 16) {
    const int64_t eb = r->dtype == RSD_F32 ? 4 : 2;
    return ((uintptr_t)r->data % bytes == 0) && ((r->seq_stride * eb) % bytes == 0) && ((r->row_stride * eb) % bytes == 0);
}

inline int check_vocab(int V) {
    if (V < 1 || V > RSD_MAX_VOCAB) return fail(RSD_ERR_UNSUPPORTED, "V = %d outside [1, %d]", V, (int)RSD_MAX_VOCAB);
    return RSD_OK;
}

}  // namespace rsd_host
