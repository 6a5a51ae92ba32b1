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
    size_t bx;    // [problems][n_pad][16] bf16: the weights as an operand of the tensor-core path's bias MMA
    size_t flags; // [problems] "weights differ" flags + one device status word
    size_t qwide; // E4M3 inputs in fp64 mode: [batch][q_heads][n_q][d] bf16, the queries widened exactly
    size_t total;
};
AttendLayout attend_layout(const elm_params *p, int32_t n_core);

// Which rows of Q / O a launch covers, and a causal tail of the coreset list.  params->n_q is the
// number of query rows of the launch; they are rows q_row0 .. q_row0 + n_q - 1 of each head's
// n_q_total rows.  List entries from tail_start on are visible to row r of the launch only up to
// entry tail_start + r (Algorithm 5 in prefill: the tail holds the launch's own tokens in order).
//
// Lifetimes (Thinformer Express in prefill, where the cache changes from token to token): when `birth` is
// set, entry c of problem p is visible to the query row whose index within its head is t iff
// birth[p][c] <= t < death[p][c], and the tail rule is not used.  Both arrays are [problems][n_pad],
// n_pad = n_core rounded up to 128; blk_birth / blk_death [problems][n_pad / 128] hold the largest birth and
// the smallest death of each block of 128 entries (a block that every row of a tile sees whole takes the
// unmasked path).  `lse`, if set, receives log2 of each row's softmax denominator (logits in base 2,
// weights included) at [batch * q_heads][n_q_total].
//
// Block lists (with lifetimes, tensor-core path only): when `tile_cnt` is set, pair x of 128-query tiles (rows
// 256 x ... of every head) streams only the tile_cnt[x] blocks tile_blk[x * tile_cap + 0 ...] of the list; the
// caller guarantees that every entry some row of the pair sees lies in one of them.
struct AttendWindow {
    int64_t q_row0 = 0;
    int64_t n_q_total = 0;               // 0: params->n_q
    int32_t tail_start = 0x7fffffff;     // no tail
    const int32_t *birth = nullptr, *death = nullptr;
    const int32_t *blk_birth = nullptr, *blk_death = nullptr;
    float *lse = nullptr;
    const int32_t *tile_cnt = nullptr, *tile_blk = nullptr;
    int32_t tile_cap = 0;
    // and, since such pairs differ in length, optionally which pairs each of item_ctas persistent CTAs takes: CTA c the
    // pairs item_tab[c * item_cap + 0 .. item_cnt[c]) (numbered head * pairs per head + x)
    const int32_t *item_tab = nullptr, *item_cnt = nullptr;
    int32_t item_cap = 0, item_ctas = 0;
};

// elm_attend after argument validation
int attend_enqueue(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w, int32_t n_core,
                   const elm_params *params, void *O, void *workspace, cudaStream_t st,
                   const AttendWindow &win = AttendWindow());

// Tensor-core path (bf16 storage, fp32 accumulation): gather + attention, enqueued on `st`.
// `timed` selects whether the per-stage event timers are used.
int attend_tc(const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V, const int32_t *idx,
              const float *w, int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws,
              cudaStream_t st, bool timed, const AttendWindow &win = AttendWindow());

// elm_debug_set for the hooks that live with the tensor-core attention
int debug_set_attend_tc(int32_t what, int64_t value);

// [count] E4M3 bytes -> bf16, exactly (every E4M3 value is a bf16 value)
int widen_e4m3(const void *src, void *dst_bf16, int64_t count, cudaStream_t st);

// Tensor-core path for E4M3 inputs (fp32 mode, d = 128, every row sees the whole list): S = Q K^T with 8-bit
// operands, probabilities and P V in bf16 (the gather widens the coreset's value rows), O in bf16.
int attend_tc_e4m3(const unsigned char *Q, const unsigned char *K, const unsigned char *V, const int32_t *idx, const float *w,
                   int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws, cudaStream_t st, bool timed);

// A few query vectors per KV head (decode): HBM-bound kernels that read the coreset rows once through
// the index list.  Applies to fp32 mode when (q_heads / kv_heads) * n_q <= 8.
bool attend_decode_applies(const elm_params *p);
int attend_decode(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w, int n_core,
                  const elm_params *p, void *O, unsigned char *ws, cudaStream_t st, bool timed);

}  // namespace elm
