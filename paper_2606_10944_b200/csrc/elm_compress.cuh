// Workspace layout of elm_compress (byte offsets into the caller's workspace).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/elm.h"

namespace elm {

struct CompressLayout {
    size_t vmax_bits;  // [BH] float bits of v_max per attention problem
    size_t cnorm;      // [BH][n]   c_t = ||k_t||^2 / sqrt(d)
    size_t cur;        // [BH][n]   current point sequence (row numbers)
    size_t nxt;        // [BH][n]   next level's sequence
    size_t Mpair;      // [BH][n/2] running shift of each pair
    size_t rdecay;     // [BH][n/2] exp(-(M_i - M_{i-1})/2)
    size_t F;          // [BH][n_out^2] pair Gram of the current level (all calls)
    size_t F_stride;   // elements per problem
    size_t wide;       // E4M3 inputs: K then V widened exactly to bf16, [BH][n][d] each
    size_t total;
};
CompressLayout compress_layout(const elm_params *p);

// elm_compress after argument validation; `pbase` = number of the call's first attention problem.
int compress_enqueue(const void *K, const void *V, const elm_params *params, uint64_t seed, int32_t *idx_out,
                     float *w_out, void *workspace, cudaStream_t st, uint32_t pbase);

// What the Gram kernel needs to also run the halving walk of calls that fit one of its tiles
// (at most 64 pairs): with `fused` set the pair Gram of the level never leaves shared memory and
// the survivors go straight to `out`.
struct WalkArgs {
    int fused;
    int64_t level;           // third counter word, first call and calls per sibling (pack_level in elm_common.cuh)
    uint64_t seed;
    float logfac;
    const float *rdecay;     // [BH][n/2]
    int32_t *out;            // next level's sequence (or the final coreset)
    int64_t out_stride;
    uint32_t pbase;          // number of the first attention problem of this call (uniforms' counter)
};

// Tensor-core pair Gram of one level (bf16 storage, fp32 arithmetic); same output layout as the
// generic kernel.  `status` is a device word that a timed-out wait sets to a non-zero code.
int gram_tc(const __nv_bfloat16 *K, const __nv_bfloat16 *V, const elm_params *p, const int32_t *cur,
            const float *Mpair, const unsigned *vmax_bits, int P, int64_t Ptotal, int groups, float *F,
            int64_t F_stride, int *status, const WalkArgs &wk, cudaStream_t st);

// The halving walk of one level for calls of at least 32 pairs (one CTA or one cluster per call).
// walk_chain_covers says whether a call size fits its shared-memory plan; `status` as above.
// walk_chain returns ELM_OK, a negative elm_status, or 1 when the device cannot keep a cluster of the
// needed size resident (nothing launched: use another kernel).
template <typename T> bool walk_chain_covers(int P);
template <typename T>
int walk_chain(const T *F, int64_t F_stride, const T *rdecay, const int32_t *cur, int32_t *out, int64_t out_stride,
               int64_t n, int P, int groups, int problems, int64_t level, uint64_t seed, T logfac, uint32_t pbase,
               int *status, cudaStream_t st);

}  // namespace elm
