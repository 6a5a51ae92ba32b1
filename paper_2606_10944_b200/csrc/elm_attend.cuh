// Workspace layout of elm_attend (byte offsets into the caller's workspace).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/elm.h"

namespace elm {

struct AttendLayout {
    size_t Kc;    // [problems][n_core][d] gathered keys, input dtype
    size_t Vc;    // [problems][n_core][d] gathered values, input dtype
    size_t bias;  // [problems][n_core] log2 of the weights, fp32
    size_t flags; // [problems] "weights differ" flags + one device status word
    size_t total;
};
AttendLayout attend_layout(const elm_params *p, int32_t n_core);

// elm_attend after argument validation
int attend_enqueue(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w, int32_t n_core,
                   const elm_params *params, void *O, void *workspace, cudaStream_t st);

// Tensor-core path (bf16 storage, fp32 accumulation): gather + attention, enqueued on `st`.
// `timed` selects whether the per-stage event timers are used.
int attend_tc(const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V, const int32_t *idx,
              const float *w, int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws,
              cudaStream_t st, bool timed);

}  // namespace elm
