// Weighted attention over a coreset on the sm_100a tensor cores (bf16 inputs, fp32 accumulation).
//
//   O[j,:] = sum_c w_c exp(<q_j,k_c>/sqrt(d)) v_c / sum_c w_c exp(<q_j,k_c>/sqrt(d))      Eq. (def:att_approx)
//
// One persistent CTA per SM takes every gridDim.x-th pair of 128-query tiles (numbered with the head
// slowest, so that the CTAs running at one time share one head's coreset in L2) and streams the
// head's coreset in blocks of 128 points for each pair.  Roles (608 threads):
//   warps 0-15       softmax, two passes over the logits in TMEM (row maximum, then probabilities).
//                    Launches without a mask: warps 0-7 own tile 0, warps 8-15 tile 1, a thread owns one
//                    row and half of the block's columns (kept in registers between the passes); the
//                    two groups run out of phase.  Launches with a mask (causal tail, lifetimes): all
//                    16 warps serve the tile whose logits are ready, tile 0 and tile 1 in turn, a thread
//                    owns one row and a quarter of the columns.  Threads that share a row exchange row
//                    maxima through shared memory behind a barrier of their own.  Probabilities go back
//                    to TMEM as packed bf16 (over the logits); the output accumulator is rescaled only
//                    when the maximum grew by more than 2^8.  Same warps: epilogue of each pair of tiles.
//   warp 16          TMA producer: the queries of each pair, K / V^T blocks through a 2-stage ring
//                    that runs on across pairs
//   warps 17, 18     tcgen05.mma issuers, one per query tile: S = Q K^T (operands in shared memory),
//                    O += P V (P read from TMEM, V^T from shared memory); warp 17 owns the TMEM
//                    allocation.  The logits of the
//                    next pair's first block are issued right behind the last O += P V of the
//                    current pair, so the tensor pipe does not drain while a pair is normalised and
//                    stored.
// TMEM columns: [0,128) S of tile 0, [128,256) S of tile 1, [256,256+D) O of tile 0, [384,384+D) O of
// tile 1.  The probabilities of the points of column quarter c are written over the first 16 columns
// of that quarter's logits, so a thread only ever overwrites logits it has already read itself.
// Weights: log2 w_c has to be added to column c of the logits.  When a problem's weights differ (or its
// list does not fill the last block) the tensor pipe adds it: one more MMA per block with K = 16,
// A = a constant tile of ones, B = per column (hi, mid, lo, 0, ...) with hi + mid + lo = log2 w_c /
// (log2 e / sqrt(d)) split into three bf16 terms (columns beyond the list: -1e30, which the exponential
// turns into 0).  The softmax warps then treat every block alike; only the rows of a causal tail,
// whose visible columns end at different places, take the slower masked form of the two passes.
// Every mbarrier wait is bounded; on expiry the CTA records a status word and leaves through the
// common exit, which frees the TMEM it holds.
#include <cuda.h>
#include <cuda_fp8.h>
#include <math.h>
#include <stdlib.h>

#include <atomic>
#include <type_traits>

#include "elm_attend.cuh"
#include "elm_common.cuh"
#include "elm_sm100.cuh"

namespace elm {
namespace tc {

constexpr int BM = 128;          // query rows per tile (= TMEM lanes)
constexpr int BN = 128;          // coreset points per block
constexpr int STAGES = 2;
constexpr int NTHREADS = 608;          // 16 softmax warps + TMA producer + two MMA issuers (one per query tile)
constexpr int TMA_WARP = 16, MMA_WARP = 17;
constexpr uint32_t TMEM_COLS = 512;
constexpr float RESCALE_TAU = 8.0f;      // rescale the accumulator only if the max grew by > 2^8
// Of every 16 column pairs, how many take 2^x from the FMA pipe (a cubic for 2^f, relative error 1e-4 - below the
// bf16 rounding of the probabilities) instead of the special-function unit.  Launches with a mask only: there all
// 16 softmax warps work on one query tile at a time, and a device timeline shows 1350 of a block's 2150 cycles in
// the pass that exponentiates - 16384 exp2 and 8192 conversions through a unit that does 16 a cycle.  A quarter of
// the exponentials on the FMA pipe: prefill of cfg5 21.3 -> 20.8 ms, 524288 tokens in the paper's setting
// 34.7 -> 34.0 ms; half of them: 20.9 and 34.7 ms.  The launches without a mask run their two query tiles out of
// phase and are short of issue slots and latency instead: none 4.04 ms, 1 pair of 16: 4.06, 2: 4.08, 4: 4.25,
// 8: 4.35 ... 4.43 - they do not use it.
constexpr int EMU_PAIRS = 4;
using namespace sm100;

struct __align__(8) Barriers {
    uint64_t q_full, q_free;
    uint64_t k_full[STAGES], v_full[STAGES], kv_free[STAGES];
    uint64_t s_full[2], p_ready[2], o_done[2], o_free[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
    float xchg[2][4][BM];        // per tile, per column quarter: row maxima / denominators being exchanged
};

// QKB: bytes per element of Q and K (2: bf16; 1: E4M3, whose S = Q K^T takes the 8-bit MMA kind)
template <int D, int QKB = 2> struct Smem {
    static constexpr int KH = D * QKB / 128;                // 128-byte slices of a row of Q or K
    static constexpr int Q_TILE = BM * D * QKB;             // bytes
    static constexpr int K_BLOCK = BN * D * QKB;
    static constexpr int V_BLOCK = D * BN * 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + 2 * Q_TILE;
    static constexpr int OFF_V = OFF_K + STAGES * K_BLOCK;
    static constexpr int X_BLOCK = BN * 16 * 2;             // bias operand: 16 bf16 per column, 32-byte swizzle
    static constexpr int OFF_X = OFF_V + STAGES * V_BLOCK;
    static constexpr int OFF_ONES = OFF_X + STAGES * X_BLOCK;   // [BM][16] bf16: the constant A operand of the bias MMA
    static constexpr int OFF_BAR = OFF_ONES + BM * 16 * 2;
    static constexpr int TOTAL = OFF_BAR + 5120 + 1024;     // barrier block + slack for 1024-byte alignment
};

// ---------------------------------------------------------------------------------------------
// gather for the tensor-core path: Kc [p][n_pad][D] (zero rows beyond n_core), Vt [p][n_pad / 128][D][128]
// (per block of 128 entries the transposed values, 32 KB in one piece; zero columns beyond n_core), Bx [p][n_pad][16]: log2 w / scale_log2 as three bf16 terms
// (then zeros), and a per-problem flag that says whether all weights of the problem are equal (then
// the bias cancels in the ratio).
// ---------------------------------------------------------------------------------------------
constexpr int GATHER_COLS = 64;          // list entries per CTA of the gather
// E4M3 = true: K and V hold 8-bit floats; the key rows are copied as they are (Kc then has D bytes per row),
// the value rows are widened to bf16 (exactly) on their way into the transposed tile.
template <int D, bool E4M3 = false>
__global__ void __launch_bounds__(256) gather_tc_kernel(const __nv_bfloat16 *__restrict__ K,
                                                        const __nv_bfloat16 *__restrict__ V,
                                                        const int32_t *__restrict__ idx,
                                                        const float *__restrict__ w, int64_t n, int n_core,
                                                        int n_pad, __nv_bfloat16 *__restrict__ Kc,
                                                        __nv_bfloat16 *__restrict__ Vt,
                                                        __nv_bfloat16 *__restrict__ Bx, float inv_scale_log2,
                                                        int *__restrict__ nonuniform)
{
    constexpr int CH = D / 8;                                  // 16-byte chunks per row
    __shared__ __align__(16) __nv_bfloat16 tile[GATHER_COLS][D + 8];      // rows 16-byte aligned
    const int p = blockIdx.y;
    const int c0 = blockIdx.x * GATHER_COLS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float w0 = w[(int64_t)p * n_core];
    bool differs = false;
    // rows move in 16-byte chunks: lanes 0 .. CH-1 the key row (straight to Kc), lanes 16 .. 16+CH-1 the
    // value row (to shared memory, to be written transposed)
    for (int r = warp; r < GATHER_COLS; r += 8) {
        const int c = c0 + r;
        const bool ok = c < n_core;
        const int64_t row = ok ? checked_row(idx[(int64_t)p * n_core + c], n, nonuniform + gridDim.y) : 0;
        const int chunk = lane & 15;
        if constexpr (E4M3) {
            // a row is D bytes = D / 16 chunks
            const unsigned char *K8 = reinterpret_cast<const unsigned char *>(K), *V8 = reinterpret_cast<const unsigned char *>(V);
            if (chunk < D / 16) {
                const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                if (lane < 16) {
                    const uint4 v = ok ? __ldg(reinterpret_cast<const uint4 *>(K8 + ((int64_t)p * n + row) * D) + chunk) : zero;
                    reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(Kc) + ((int64_t)p * n_pad + c) * D)[chunk] = v;
                } else {
                    const uint4 v = ok ? __ldg(reinterpret_cast<const uint4 *>(V8 + ((int64_t)p * n + row) * D) + chunk) : zero;
                    const unsigned char *b = reinterpret_cast<const unsigned char *>(&v);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)b[e], __NV_E4M3);
                        tile[r][chunk * 16 + e] = __float2bfloat16_rn(__half2float(__half(h)));
                    }
                }
            }
        } else if (chunk < CH) {
            const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
            if (lane < 16) {
                const uint4 v = ok ? __ldg(reinterpret_cast<const uint4 *>(K + ((int64_t)p * n + row) * D) + chunk) : zero;
                reinterpret_cast<uint4 *>(Kc + ((int64_t)p * n_pad + c) * D)[chunk] = v;
            } else {
                const uint4 v = ok ? __ldg(reinterpret_cast<const uint4 *>(V + ((int64_t)p * n + row) * D) + chunk) : zero;
                *reinterpret_cast<uint4 *>(&tile[r][chunk * 8]) = v;
            }
        }
        if (lane < 16) {
            const float wc = ok ? w[(int64_t)p * n_core + c] : 0.f;
            // in the logits' own units (they are multiplied by scale_log2 later); -1e30 hides a padded column
            const float x = ok ? log2f(wc) * inv_scale_log2 : -1e30f;
            const __nv_bfloat16 hi = __float2bfloat16(x);
            const float r1 = ok ? x - __bfloat162float(hi) : 0.f;
            const __nv_bfloat16 mid = __float2bfloat16(r1);
            const __nv_bfloat16 lo = __float2bfloat16(r1 - __bfloat162float(mid));
            Bx[((int64_t)p * n_pad + c) * 16 + lane] = lane == 0 ? hi : (lane == 1 ? mid : (lane == 2 ? lo : __float2bfloat16(0.f)));
            if (lane == 0 && ok && wc != w0) differs = true;
        }
    }
    if (differs) atomicOr(nonuniform + p, 1);
    __syncthreads();
    // transposed write: a warp writes the 64 entries of one dimension e, 128 contiguous bytes
    for (int e = warp; e < D; e += 8) {
        const uint32_t lo = __bfloat16_as_ushort(tile[2 * lane][e]), hi = __bfloat16_as_ushort(tile[2 * lane + 1][e]);
        *reinterpret_cast<uint32_t *>(Vt + (((int64_t)p * (n_pad / 128) + c0 / 128) * D + e) * 128 + (c0 % 128) + 2 * lane) = lo | (hi << 16);
    }
}

// ---------------------------------------------------------------------------------------------
// softmax helpers: a thread owns one row (TMEM lane) and NCH chunks of 32 logit columns
// ---------------------------------------------------------------------------------------------
// Row maximum in base-2 units (SPECIAL: only the columns whose bit is set in `vmask` count); the logits
// stay in TMEM.
template <bool SPECIAL, int NCH>
__device__ __forceinline__ float row_max(uint32_t tS, float scale_log2, uint32_t vmask)
{
    float m0 = -INFINITY, m1 = -INFINITY;
    uint32_t a[2][32];
    tmem_ld32(tS, a[0]);
#pragma unroll
    for (int q = 0; q < NCH; ++q) {
        tmem_wait_ld();
        if (q + 1 < NCH) tmem_ld32(tS + (q + 1) * 32, a[(q + 1) & 1]);
        if (!SPECIAL) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                m0 = max3(m0, __uint_as_float(a[q & 1][c]), __uint_as_float(a[q & 1][c + 1]));
                m1 = max3(m1, __uint_as_float(a[q & 1][c + 2]), __uint_as_float(a[q & 1][c + 3]));
            }
        } else {
            // the same in the logits' own units (scale_log2 > 0), a masked column counting as -inf
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                const float v0 = ((vmask >> c) & 1u) ? __uint_as_float(a[q & 1][c]) : -INFINITY;
                const float v1 = ((vmask >> (c + 1)) & 1u) ? __uint_as_float(a[q & 1][c + 1]) : -INFINITY;
                const float v2 = ((vmask >> (c + 2)) & 1u) ? __uint_as_float(a[q & 1][c + 2]) : -INFINITY;
                const float v3 = ((vmask >> (c + 3)) & 1u) ? __uint_as_float(a[q & 1][c + 3]) : -INFINITY;
                m0 = max3(m0, v0, v1);
                m1 = max3(m1, v2, v3);
            }
        }
    }
    return fmaxf(m0, m1) * scale_log2;
}

// p = 2^(logit - reference): reads the logits, writes the probabilities as packed bf16 to tP
// (16 columns per chunk) and returns their fp32 row sum.  Each chunk is staged (all scalings, then
// all exponentials, ...) so that independent operations interleave.
template <bool SPECIAL, int NCH>
__device__ __forceinline__ float exp_pass(uint32_t tS, uint32_t tP, float scale_log2, float neg_m, uint32_t vmask)
{
    const uint64_t scale2 = pack2(scale_log2, scale_log2), negm2 = pack2(neg_m, neg_m);
    uint64_t sum2 = pack2(0.f, 0.f), sum2b = pack2(0.f, 0.f);
    float sum0 = 0.f;
    uint32_t a[2][32];
    tmem_ld32(tS, a[0]);
#pragma unroll
    for (int q = 0; q < NCH; ++q) {
        tmem_wait_ld();
        if (q + 1 < NCH) tmem_ld32(tS + (q + 1) * 32, a[(q + 1) & 1]);
        uint32_t pk[16];
        if (!SPECIAL) {
            uint64_t x2[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
                x2[i] = fma2(pack2(__uint_as_float(a[q & 1][2 * i]), __uint_as_float(a[q & 1][2 * i + 1])), scale2, negm2);
            float pe[32];
            // EMU_PAIRS of the 16 pairs can take 2^x from the FMA pipe instead of the special-function unit
            // (16 exp2 per clock per SM): x = n + f with n = round(x)
            // (magic-number add), 2^f by a cubic on [-1/2, 1/2] (relative error 1e-4, below the bf16
            // rounding of the probabilities), n added to the exponent field.
#pragma unroll
            for (int i = 0; i < EMU_PAIRS; ++i) {
                float x0, x1;
                unpack2(x2[i], x0, x1);
                const uint64_t xc = pack2(fmaxf(x0, -125.f), fmaxf(x1, -125.f));
                const uint64_t magic = pack2(12582912.f, 12582912.f), nmagic = pack2(-12582912.f, -12582912.f);
                const uint64_t tt = add2(xc, magic);                       // low mantissa bits = n
                const uint64_t nn = add2(tt, nmagic);                      // n as a float
                const uint64_t ff = fma2(nn, pack2(-1.f, -1.f), xc);           // f = x - n
                uint64_t pp = fma2(pack2(0.05500893f, 0.05500893f), ff, pack2(0.24221096f, 0.24221096f));
                pp = fma2(pp, ff, pack2(0.69328293f, 0.69328293f));
                pp = fma2(pp, ff, pack2(1.f, 1.f));
                float p0, p1, t0, t1;
                unpack2(pp, p0, p1);
                unpack2(tt, t0, t1);
                pe[2 * i] = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(t0) << 23));
                pe[2 * i + 1] = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(t1) << 23));
            }
#pragma unroll
            for (int i = EMU_PAIRS; i < 16; ++i) {
                float x0, x1;
                unpack2(x2[i], x0, x1);
                pe[2 * i] = fast_exp2(x0);
                pe[2 * i + 1] = fast_exp2(x1);
            }
#pragma unroll
            for (int i = 0; i < 16; i += 2) {
                sum2 = add2(sum2, pack2(pe[2 * i], pe[2 * i + 1]));
                sum2b = add2(sum2b, pack2(pe[2 * i + 2], pe[2 * i + 3]));
            }
            // one conversion per pair (rounding by two integer adds and a byte permute was 2 % slower: 4.05
            // against 3.98 ms)
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(pe[2 * i], pe[2 * i + 1]);
        } else {
            // the packed arithmetic of the plain form, a masked column's probability replaced by 0
#pragma unroll
            for (int i = 0; i < 16; i += 2) {
                const int c = 2 * i;
                float x0, x1, x2, x3;
                unpack2(fma2(pack2(__uint_as_float(a[q & 1][c]), __uint_as_float(a[q & 1][c + 1])), scale2, negm2), x0, x1);
                unpack2(fma2(pack2(__uint_as_float(a[q & 1][c + 2]), __uint_as_float(a[q & 1][c + 3])), scale2, negm2), x2, x3);
                const float p0 = ((vmask >> c) & 1u) ? fast_exp2(x0) : 0.f, p1 = ((vmask >> (c + 1)) & 1u) ? fast_exp2(x1) : 0.f;
                const float p2 = ((vmask >> (c + 2)) & 1u) ? fast_exp2(x2) : 0.f, p3 = ((vmask >> (c + 3)) & 1u) ? fast_exp2(x3) : 0.f;
                sum2 = add2(sum2, pack2(p0, p1));
                sum2b = add2(sum2b, pack2(p2, p3));
                pk[i] = pack_bf16x2(p0, p1);
                pk[i + 1] = pack_bf16x2(p2, p3);
            }
        }
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
            ::"r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]),
              "r"(pk[8]), "r"(pk[9]), "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15]),
              "r"(tP + q * 16)
            : "memory");
    }
    float s_lo, s_hi;
    unpack2(add2(sum2, sum2b), s_lo, s_hi);
    return sum0 + s_lo + s_hi;
}

// The plain form for one chunk with the 32 logits kept in registers between the two passes (one TMEM load
// per block instead of two).
__device__ __forceinline__ float row_max_keep(uint32_t tS, float scale_log2, uint32_t (&a)[32])
{
    float m0 = -INFINITY, m1 = -INFINITY;
    tmem_ld32(tS, a);
    tmem_wait_ld();
#pragma unroll
    for (int c = 0; c < 32; c += 4) {
        m0 = max3(m0, __uint_as_float(a[c]), __uint_as_float(a[c + 1]));
        m1 = max3(m1, __uint_as_float(a[c + 2]), __uint_as_float(a[c + 3]));
    }
    return fmaxf(m0, m1) * scale_log2;
}
__device__ __forceinline__ float exp_pass_keep(uint32_t tP, float scale_log2, float neg_m, const uint32_t (&a)[32])
{
    const uint64_t scale2 = pack2(scale_log2, scale_log2), negm2 = pack2(neg_m, neg_m);
    uint64_t sum2 = pack2(0.f, 0.f), sum2b = pack2(0.f, 0.f);
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        float x0, x1, x2, x3;
        unpack2(fma2(pack2(__uint_as_float(a[2 * i]), __uint_as_float(a[2 * i + 1])), scale2, negm2), x0, x1);
        unpack2(fma2(pack2(__uint_as_float(a[2 * i + 2]), __uint_as_float(a[2 * i + 3])), scale2, negm2), x2, x3);
        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = fast_exp2(x3);
        sum2 = add2(sum2, pack2(p0, p1));
        sum2b = add2(sum2b, pack2(p2, p3));
        pk[i] = pack_bf16x2(p0, p1);
        pk[i + 1] = pack_bf16x2(p2, p3);
    }
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
        ::"r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]),
          "r"(pk[8]), "r"(pk[9]), "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15]),
          "r"(tP)
        : "memory");
    float s_lo, s_hi;
    unpack2(add2(sum2, sum2b), s_lo, s_hi);
    return s_lo + s_hi;
}

// ---------------------------------------------------------------------------------------------
// TMA producer of a launch with block lists (one thread): the queries of each pair, and the K / V^T / bias blocks
// of each pair's own list through the 2-stage ring.  Same protocol as the producer inside the kernel; kept out of
// line (it is called once per CTA) so that its code does not weigh on the register allocation and scheduling of
// the kernel's softmax warps.
// ---------------------------------------------------------------------------------------------
// An entry of a block list: the block's number, and bit 30 set unless every row of the pair sees the block whole
// (then no lifetime is looked at).
constexpr int BLK_NUMBER = 0x3fffffff, BLK_PARTLY = 1 << 30;
struct ProducerArgs {
    const CUtensorMap *mapQ, *mapK, *mapV, *mapX;
    unsigned char *smem;
    Barriers *bar;
    const int *nonuniform;
    const int32_t *tile_cnt, *tile_blk, *item_tab;
    int n_items, tiles_x, tile_cap, item_cap, q_heads, kv_heads, q_row0, nblk, ragged_end;
    unsigned long long wait_limit_ns;
};
template <int D, int QKB>
__device__ __noinline__ bool produce_block_lists(const ProducerArgs *a)
{
    using SM = Smem<D, QKB>;
    constexpr int KH = SM::KH;
    constexpr int ROW_ELTS = 128 / QKB;
    unsigned char *smem = a->smem;
    Barriers *bar = a->bar;
    const int n_items = a->n_items, tiles_x = a->tiles_x, nblk = a->nblk;
    const unsigned long long limit = a->wait_limit_ns;
    auto item_id = [&](int k) -> int {
        return a->item_tab ? __ldg(a->item_tab + (int64_t)blockIdx.x * a->item_cap + k) : (int)blockIdx.x + k * (int)gridDim.x;
    };
    auto prob_of = [&](int bh) { return (bh / a->q_heads) * a->kv_heads + (int)(((int64_t)(bh % a->q_heads) * a->kv_heads) / a->q_heads); };
    // A cursor stands at block j of item k of the CTA's stream.  What the next load needs - the item's problem, the
    // block's number in the list, whether the item takes the bias operand - is fetched when the cursor moves
    // there, a whole block period before it is used: the ring has two stages, so whatever the producer does
    // between "stage free" and "copy issued" delays the tensor pipe.
    struct Cursor { int k, j, nb, id, prob, blk; bool bias; };
    auto fetch_blk = [&](Cursor &c) {
        c.blk = c.k < n_items ? (a->tile_blk ? (__ldg(a->tile_blk + (int64_t)(c.id % tiles_x) * a->tile_cap + c.j) & BLK_NUMBER) : c.j) : 0;
    };
    auto enter = [&](Cursor &c, bool want_bias) {                // the item the cursor has moved to
        c.id = c.k < n_items ? item_id(c.k) : 0;
        c.nb = c.k < n_items ? (a->tile_cnt ? __ldg(a->tile_cnt + c.id % tiles_x) : nblk) : 0;
        c.prob = prob_of(c.id / tiles_x);
        c.bias = want_bias && c.k < n_items && (a->ragged_end || __ldg(a->nonuniform + c.prob) != 0);
        fetch_blk(c);
    };
    auto cursor_next = [&](Cursor &c, bool want_bias) {
        if (++c.j == c.nb) { c.j = 0; ++c.k; enter(c, want_bias); }
        else fetch_blk(c);
    };
    auto load_q = [&](int id) {
        const int bh = id / tiles_x, q0 = (id % tiles_x) * (2 * BM);
        mbar_expect_tx(&bar->q_full, 2 * SM::Q_TILE);
        for (int t = 0; t < 2; ++t)
            for (int kh = 0; kh < KH; ++kh)
                tma_load_3d(smem + SM::OFF_Q + t * SM::Q_TILE + kh * (BM * 128), a->mapQ, &bar->q_full, kh * ROW_ELTS, a->q_row0 + q0 + t * BM, bh);
    };
    int total = 0;
    if (a->tile_cnt)
        for (int k = 0; k < n_items; ++k) total += __ldg(a->tile_cnt + item_id(k) % tiles_x);
    else
        total = n_items * nblk;
    Cursor kc = {0, 0, 0, 0, 0, 0, false};
    enter(kc, true);
    Cursor vc = kc;
    auto load_k = [&](int G) {
        const int s = G % STAGES;
        mbar_expect_tx(&bar->k_full[s], SM::K_BLOCK + (kc.bias ? SM::X_BLOCK : 0));
        for (int kh = 0; kh < KH; ++kh)
            tma_load_3d(smem + SM::OFF_K + s * SM::K_BLOCK + kh * (BN * 128), a->mapK, &bar->k_full[s], kh * ROW_ELTS, kc.blk * BN, kc.prob);
        if (kc.bias) tma_load_3d(smem + SM::OFF_X + s * SM::X_BLOCK, a->mapX, &bar->k_full[s], 0, kc.blk * BN, kc.prob);
        cursor_next(kc, true);
    };
    auto load_v = [&](int G) {
        const int s = G % STAGES;
        mbar_expect_tx(&bar->v_full[s], SM::V_BLOCK);
        for (int hh = 0; hh < 2; ++hh)
            tma_load_3d(smem + SM::OFF_V + s * SM::V_BLOCK + hh * (D * 128), a->mapV, &bar->v_full[s], hh * 64, 0, vc.prob * nblk + vc.blk);
        cursor_next(vc, false);
    };
    bool ok = true;
    // The queries of item k may replace those of item k - 1 once every S = Q K^T of item k - 1 has been computed
    // (q_free); they are fetched right after the keys of the item's first block (the key cursor then stands
    // behind that block).
    int next_q = 1;
    auto feed_q = [&]() {
        while (ok && next_q < n_items && (kc.k > next_q || (kc.k == next_q && kc.j > 0))) {
            ok = sm100::mbar_wait(&bar->q_free, (uint32_t)(next_q - 1) & 1u, limit);
            if (ok) load_q(item_id(next_q));
            ++next_q;
        }
    };
    if (n_items > 0) load_q(item_id(0));
    // The issuer commits "event" i to kv_free[i % 2] after the prologue (i = 0: S = Q K^T of block 0 issued) and
    // after iteration i - 1 (O += P V of block i - 1 and S = Q K^T of block i issued).  Once event i is complete,
    // K's stage i % 2 (block i) and V's stage (i + 1) % 2 (block i - 1) have been read, so K(i + 2) and V(i + 1)
    // may overwrite them.
    for (int G = 0; G < STAGES && G < total; ++G) { load_k(G); load_v(G); }
    feed_q();
    for (int i = 0; i + 2 < total && ok; ++i) {
        ok = sm100::mbar_wait(&bar->kv_free[i % STAGES], (uint32_t)(i / STAGES) & 1u, limit);
        if (!ok) break;
        load_k(i + 2);
        if (i >= 1) load_v(i + 1);
        feed_q();
    }
    // the last V block: freed by event total - 1
    if (ok && total > STAGES) {
        const int i = total - 2;
        ok = sm100::mbar_wait(&bar->kv_free[i % STAGES], (uint32_t)(i / STAGES) & 1u, limit);
        if (ok) load_v(i + 1);
    }
    return ok;
}

// ---------------------------------------------------------------------------------------------
// the attention kernel
// ---------------------------------------------------------------------------------------------
// MASKED = false: every row sees the whole list (no causal tail, no lifetimes); the masked form of the
// softmax passes is then not compiled in, which keeps the plain form's register allocation to itself.
template <int D, bool MASKED, int QKB = 2>
__global__ void __launch_bounds__(NTHREADS, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                 const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapX,
                 const int *__restrict__ nonuniform, __nv_bfloat16 *__restrict__ O, int q_heads,
                 int kv_heads, int n_q, int n_core, int n_pad, float scale_log2, int tiles_x, int n_items_total,
                 int q_row0, int n_q_total, int tail_start, const int32_t *__restrict__ birth,
                 const int32_t *__restrict__ death, const int32_t *__restrict__ blk_birth,
                 const int32_t *__restrict__ blk_death, float *__restrict__ lse, int *__restrict__ status,
                 int extra_arrivals, unsigned long long wait_limit_ns, const int32_t *__restrict__ tile_cnt,
                 const int32_t *__restrict__ tile_blk, int tile_cap, const int32_t *__restrict__ item_tab,
                 const int32_t *__restrict__ item_cnt, int item_cap)
{
    // every wait of this kernel is bounded by the limit the host passes (2 s unless a test shortened it)
    auto mbar_wait = [wait_limit_ns](uint64_t *b, uint32_t parity) { return sm100::mbar_wait(b, parity, wait_limit_ns); };
    using SM = Smem<D, QKB>;
    constexpr int KH = SM::KH;
    constexpr int ROW_ELTS = 128 / QKB;                            // elements of Q / K in a 128-byte slice of a row
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    Barriers *bar = reinterpret_cast<Barriers *>(smem + SM::OFF_BAR);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nblk = n_pad / BN;
    // Persistent CTA: work item k of this CTA is pair-of-query-tiles number blockIdx.x + k gridDim.x,
    // numbered with the head slowest, so that at any time the CTAs share one head's coreset in L2.
    // (a launch with block lists may also say which items each CTA takes - item_tab[blockIdx.x][0 .. item_cnt[blockIdx.x])
    // - because its items differ in length)
    auto item_id = [&](int k) -> int {
        if constexpr (MASKED) {
            if (item_tab) return __ldg(item_tab + (int64_t)blockIdx.x * item_cap + k);
        }
        return (int)blockIdx.x + k * (int)gridDim.x;
    };
    const int n_items = (MASKED && item_tab) ? __ldg(item_cnt + blockIdx.x)
                                             : (n_items_total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    // A launch with block lists (tile_cnt set; lifetimes only): pair number x of every head streams the
    // tile_cnt[x] blocks tile_blk[x][0 ..] of the list instead of all of them - the list then holds every
    // entry some row of the launch sees, and each pair visits the blocks that hold entries its own rows see.
    auto item_nblk = [&](int k) -> int {
        if constexpr (MASKED) {
            if (tile_cnt) return __ldg(tile_cnt + item_id(k) % tiles_x);
        }
        return nblk;
    };
    auto item_blk = [&](int k, int j) -> int {
        if constexpr (MASKED) {
            if (tile_cnt) return __ldg(tile_blk + (int64_t)(item_id(k) % tiles_x) * tile_cap + j);      // number | BLK_PARTLY
        }
        return j;
    };
    // coreset blocks this CTA streams, over all items
    auto count_blocks = [&]() -> int {
        if constexpr (MASKED) {
            if (tile_cnt) {
                int sum = 0;
                for (int k = 0; k < n_items; ++k) sum += item_nblk(k);
                return sum;
            }
        }
        return n_items * nblk;
    };
    auto item_bh = [&](int k) { return item_id(k) / tiles_x; };
    auto item_q0 = [&](int k) { return (item_id(k) % tiles_x) * (2 * BM); };
    auto prob_of = [&](int bh) { return (bh / q_heads) * kv_heads + (int)(((int64_t)(bh % q_heads) * kv_heads) / q_heads); };
    // does item k take the bias MMA?  (weights differ, or the last block is only partly filled)
    const bool ragged_end = n_core % BN != 0;
    auto item_bias = [&](int k) { return ragged_end || __ldg(nonuniform + prob_of(item_bh(k))) != 0; };

    // a CTA that gave up on a wait poisons the launch: the remaining CTAs leave at once
    if (*reinterpret_cast<volatile int *>(status) != 0) return;

    if (threadIdx.x == 0) {
        mbar_init(&bar->q_full, 1);
        mbar_init(&bar->q_free, 2);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&bar->k_full[s], 1);
            mbar_init(&bar->v_full[s], 1);
            mbar_init(&bar->kv_free[s], 2);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&bar->s_full[t], 1);
            // (extra_arrivals is 0 except in the test that lets a wait run out: arrivals that nobody makes)
            mbar_init(&bar->p_ready[t], (MASKED ? 512 : 256) + extra_arrivals);
            mbar_init(&bar->o_done[t], 1);
            mbar_init(&bar->o_free[t], MASKED ? 16 : 8);
        }
        bar->abort_flag = 0;
        fence_barrier_init();
    }
    // the constant A operand of the bias MMA: every row (1, 1, 1, 0, 0, 0, 0, 0) in both 16-byte halves,
    // so that the 32-byte swizzle (which exchanges the halves of some rows) leaves it unchanged
    for (int i = threadIdx.x; i < BM * 16 / 2; i += NTHREADS)
        reinterpret_cast<uint32_t *>(smem + SM::OFF_ONES)[i] = (i & 3) == 0 ? 0x3F803F80u : ((i & 3) == 1 ? 0x00003F80u : 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == MMA_WARP) tmem_alloc(&bar->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;

    if (warp == TMA_WARP) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            auto load_q = [&](int k) {
                const int bh = item_bh(k), q0 = item_q0(k);
                mbar_expect_tx(&bar->q_full, 2 * SM::Q_TILE);
                for (int t = 0; t < 2; ++t)
                    for (int kh = 0; kh < KH; ++kh)
                        tma_load_3d(smem + SM::OFF_Q + t * SM::Q_TILE + kh * (BM * 128), &mapQ, &bar->q_full, kh * ROW_ELTS, q_row0 + q0 + t * BM, bh);
            };
            bool ok = true;
            if (!MASKED || !tile_cnt) {
                // (every pair streams the whole list: block G of the stream is block G % nblk of item G / nblk)
                // Blocks are numbered G = k nblk + j along the CTA's whole stream (item k, block j).
                const int total = n_items * nblk;
                int flag_item = -1;
                bool flag_now = false, flag_next = n_items > 0 && item_bias(0);
                auto load_k = [&](int G) {
                    const int s = G % STAGES, prob = prob_of(item_bh(G / nblk));
                    // the flag of an item is fetched while the item before it streams, off the critical path
                    if (G / nblk != flag_item) {
                        flag_item = G / nblk;
                        flag_now = flag_next;
                        flag_next = flag_item + 1 < n_items && item_bias(flag_item + 1);
                    }
                    const bool with_bias = flag_now;
                    mbar_expect_tx(&bar->k_full[s], SM::K_BLOCK + (with_bias ? SM::X_BLOCK : 0));
                    for (int kh = 0; kh < KH; ++kh)
                        tma_load_3d(smem + SM::OFF_K + s * SM::K_BLOCK + kh * (BN * 128), &mapK, &bar->k_full[s], kh * ROW_ELTS, (G % nblk) * BN, prob);
                    if (with_bias) tma_load_3d(smem + SM::OFF_X + s * SM::X_BLOCK, &mapX, &bar->k_full[s], 0, (G % nblk) * BN, prob);
                };
                auto load_v = [&](int G) {
                    const int s = G % STAGES, prob = prob_of(item_bh(G / nblk));
                    mbar_expect_tx(&bar->v_full[s], SM::V_BLOCK);
                    for (int hh = 0; hh < 2; ++hh)
                        tma_load_3d(smem + SM::OFF_V + s * SM::V_BLOCK + hh * (D * 128), &mapV, &bar->v_full[s], hh * 64, 0, prob * nblk + G % nblk);
                };
                // The queries of item k may replace those of item k - 1 once every S = Q K^T of item k - 1
                // has been computed (q_free); they are fetched right after the keys of the item's first block.
                int next_q = 1, k_loaded = -1;
                auto feed_q = [&]() {
                    while (ok && next_q < n_items && next_q * nblk <= k_loaded) {
                        ok = mbar_wait(&bar->q_free, (uint32_t)(next_q - 1) & 1u);
                        if (ok) load_q(next_q);
                        ++next_q;
                    }
                };
                load_q(0);
                // The issuer commits "event" i to kv_free[i % 2] after the prologue (i = 0: S = Q K^T of block
                // 0 issued) and after iteration i - 1 (O += P V of block i - 1 and S = Q K^T of block i issued).
                // Once event i is complete, K's stage i % 2 (block i) and V's stage (i + 1) % 2 (block i - 1)
                // have been read, so K(i + 2) and V(i + 1) may overwrite them.
                for (int G = 0; G < STAGES && G < total; ++G) { load_k(G); load_v(G); k_loaded = G; }
                feed_q();
                for (int i = 0; i + 2 < total && ok; ++i) {
                    ok = mbar_wait(&bar->kv_free[i % STAGES], (uint32_t)(i / STAGES) & 1u);
                    if (!ok) break;
                    load_k(i + 2);
                    k_loaded = i + 2;
                    if (i >= 1) load_v(i + 1);
                    feed_q();
                }
                // the last V block: freed by event total - 1
                if (ok && total > STAGES) {
                    const int i = total - 2;
                    ok = mbar_wait(&bar->kv_free[i % STAGES], (uint32_t)(i / STAGES) & 1u);
                    if (ok) load_v(i + 1);
                }
            } else {
                // (launch with block lists: the producer that walks them is a function of its own, not inlined - the
                // code of this kernel's other roles is sensitive to what is compiled in beside it)
                ProducerArgs pa;
                pa.mapQ = &mapQ; pa.mapK = &mapK; pa.mapV = &mapV; pa.mapX = &mapX;
                pa.smem = smem; pa.bar = bar;
                pa.nonuniform = nonuniform; pa.tile_cnt = tile_cnt; pa.tile_blk = tile_blk; pa.item_tab = item_tab;
                pa.n_items = n_items; pa.tiles_x = tiles_x; pa.tile_cap = tile_cap; pa.item_cap = item_cap;
                pa.q_heads = q_heads; pa.kv_heads = kv_heads; pa.q_row0 = q_row0; pa.nblk = nblk;
                pa.ragged_end = ragged_end ? 1 : 0;
                pa.wait_limit_ns = wait_limit_ns;
                ok = produce_block_lists<D, QKB>(&pa);
            }
            if (!ok) { atomicExch(status, 1); bar->abort_flag = 1; }
        }
    } else if (warp == MMA_WARP || warp == MMA_WARP + 1) {
        // ------------------------------ MMA issuers ------------------------------
        // One issuing thread per query tile.  A tcgen05.mma holds its issuing thread until the tensor pipe
        // takes it, and the waits and commits around a block cost that thread several hundred cycles in
        // which it feeds nothing: with one thread for both tiles the pipe idled a quarter of the time.
        // Each thread commits its own MMAs, so the barriers that release shared memory count two arrivals.
        if (lane == 0) {
            const int t = warp - MMA_WARP;
            constexpr uint32_t IDESC_QK = QKB == 1 ? umma_idesc_e4m3(BM, BN) : umma_idesc_bf16(BM, BN);
            constexpr uint32_t IDESC_BIAS = umma_idesc_bf16(BM, BN);     // the bias operands are bf16 whatever Q and K are
            constexpr uint32_t IDESC_PV = umma_idesc_bf16(BM, D);
            // descriptors differ only in the 14-bit start-address field (address / 16)
            const uint64_t dQ = umma_desc_k128(smem_u32(smem + SM::OFF_Q));
            const uint64_t dK = umma_desc_k128(smem_u32(smem + SM::OFF_K));
            const uint64_t dV = umma_desc_k128(smem_u32(smem + SM::OFF_V));
            const uint64_t dX = umma_desc_k32(smem_u32(smem + SM::OFF_X));
            const uint64_t dOnes = umma_desc_k32(smem_u32(smem + SM::OFF_ONES));
            auto issue_qk = [&](int t, int s, bool with_bias) {
                const uint64_t a0 = dQ + (uint64_t)(t * (SM::Q_TILE >> 4));
                const uint64_t b0 = dK + (uint64_t)(s * (SM::K_BLOCK >> 4));
#pragma unroll
                for (int kh = 0; kh < KH; ++kh)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        if constexpr (QKB == 1)
                            mma_ss_f8(tmem + t * 128, a0 + (uint64_t)(kh * (BM * 128 >> 4) + ks * 2),
                                      b0 + (uint64_t)(kh * (BN * 128 >> 4) + ks * 2), IDESC_QK, (kh | ks) != 0);
                        else
                            mma_ss(tmem + t * 128, a0 + (uint64_t)(kh * (BM * 128 >> 4) + ks * 2),
                                   b0 + (uint64_t)(kh * (BN * 128 >> 4) + ks * 2), IDESC_QK, (kh | ks) != 0);
                // S += ones x (log2 w / scale_log2 in three bf16 terms)^T
                if (with_bias) mma_ss(tmem + t * 128, dOnes, dX + (uint64_t)(s * (SM::X_BLOCK >> 4)), IDESC_BIAS, 1u);
            };
            auto issue_pv = [&](int t, int s, bool acc) {
                const uint64_t b0 = dV + (uint64_t)(s * (SM::V_BLOCK >> 4));
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_ts(tmem + 256 + t * 128, tmem + t * 128 + (hh * 2 + (ks >> 1)) * 32 + (ks & 1) * 8,
                               b0 + (uint64_t)(hh * (D * 128 >> 4) + ks * 2), IDESC_PV, (acc || (hh | ks) != 0) ? 1u : 0u);
            };
            const int total = count_blocks();
            int nb = n_items > 0 ? item_nblk(0) : 0;                           // blocks of item k
            bool ok = mbar_wait(&bar->q_full, 0) && mbar_wait(&bar->k_full[0], 0);
            if (ok) {
                tc_fence_after();
                const bool b0 = item_bias(0);
                issue_qk(t, 0, b0);
                tc_commit(&bar->s_full[t]);
                if (nb == 1) tc_commit(&bar->q_free);                          // item 0 needs its queries no more
                tc_commit(&bar->kv_free[0]);                                   // event 0
            }
            // Iteration G: O += P V of block G, then S = Q K^T of block G + 1 - which may be the first
            // block of the next item: the tensor pipe runs on while the softmax warps finish an item.
            int j = 0, k = 0;                                                  // block G = item k, block j
            bool bias_next = n_items > 0 && item_bias(0);                      // of the item block G + 1 belongs to
            bool bias_after = false;
            int nb_after = 0;                                                  // blocks of item k + 1
            for (int G = 0; G < total && ok; ++G) {
                const int s = G % STAGES;
                const bool more = G + 1 < total;
                const int sn = (G + 1) % STAGES;
                const bool last = j == nb - 1;                                 // last block of item k
                if (j == 0) {                                                  // fetched early, used at the item's last block
                    bias_after = k + 1 < n_items && item_bias(k + 1);
                    nb_after = k + 1 < n_items ? item_nblk(k + 1) : 0;
                }
                if (last) bias_next = bias_after;
                if (more) ok = mbar_wait(&bar->k_full[sn], (uint32_t)((G + 1) / STAGES) & 1u);
                ok = ok && mbar_wait(&bar->v_full[s], (uint32_t)(G / STAGES) & 1u);
                ok = ok && mbar_wait(&bar->p_ready[t], (uint32_t)G & 1u);
                // a new item overwrites the accumulator: the epilogue of the previous one must have read it
                if (ok && j == 0 && k > 0) ok = mbar_wait(&bar->o_free[t], (uint32_t)(k - 1) & 1u);
                if (!ok) break;
                tc_fence_after();
                issue_pv(t, s, j > 0);
                // s_full also tells the softmax warps that O += P V of block j is complete (a commit
                // covers every earlier MMA of this thread); the last block of an item signals the epilogue
                if (last) tc_commit(&bar->o_done[t]);
                if (more) {
                    // the next item's queries are needed only now, after this item's last O += P V went out
                    if (last) ok = mbar_wait(&bar->q_full, (uint32_t)(k + 1) & 1u);
                    if (!ok) break;
                    issue_qk(t, sn, bias_next);
                    tc_commit(&bar->s_full[t]);
                }
                if (!ok) break;
                // the logits just issued belong to block j + 1 of item k, or to block 0 of item k + 1
                const int jn = last ? 0 : j + 1;
                if (more && jn == (last ? nb_after : nb) - 1) tc_commit(&bar->q_free);
                tc_commit(&bar->kv_free[(G + 1) % STAGES]);                    // event G + 1
                j = jn;
                if (last) { ++k; nb = nb_after; }
            }
            if (!ok) { atomicExch(status, 2); bar->abort_flag = 1; }
        }
    } else {
        // ------------------------------ softmax + epilogue ------------------------------
        if constexpr (!MASKED) {
        // No mask: warps 0-7 own query tile 0, warps 8-15 tile 1, so the two tiles' passes run out of
        // phase - while one group waits for the tensor pipe, or is between its passes, the other keeps
        // the special-function unit busy (the exponentials of a block are what a pass mostly waits for).
        // Warps with the same (warp % 4) share 32 rows; a thread owns one row and half of the block's
        // columns (two quarters, the logits kept in registers between the passes); the two halves
        // exchange their row maxima through shared memory behind a 64-thread barrier of their own.
        const int t = warp >> 3, ch = (warp >> 2) & 1;
        const int row = (warp & 3) * 32 + lane;                    // row in the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_addr + t * 128 + ch * 64;  // this thread's 64 logit columns
        const uint32_t tO = tmem + lane_addr + 256 + t * 128 + ch * (D / 2);   // its half of the accumulator
        const int bar_id = 1 + t * 4 + (warp & 3);
        const uint64_t scale2 = pack2(scale_log2, scale_log2);
        bool ok = true;
        int G = 0, xc = 0;                                         // xc: exchanges so far (buffers alternate)
        for (int k = 0; k < n_items && ok; ++k) {
            const int bh = item_bh(k), q0 = item_q0(k);
            float m_ref = -INFINITY, l = 0.f;
            for (int j = 0; j < nblk && ok; ++j, ++G, ++xc) {
                ok = mbar_wait(&bar->s_full[t], (uint32_t)G & 1u);
                if (!ok) break;
                tc_fence_after();
                // ---- pass 1: row maximum over the two halves ----
                uint32_t a0[32], a1[32];
                tmem_ld32(tS, a0);
                tmem_ld32(tS + 32, a1);
                tmem_wait_ld();
                float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    m0 = max3(m0, __uint_as_float(a0[c]), __uint_as_float(a0[c + 1]));
                    m1 = max3(m1, __uint_as_float(a1[c]), __uint_as_float(a1[c + 1]));
                }
                bar->xchg[xc & 1][t * 2 + ch][row] = fmaxf(m0, m1) * scale_log2;
                asm volatile("bar.sync %0, 64;" ::"r"(bar_id) : "memory");
                const float mx = fmaxf(bar->xchg[xc & 1][t * 2][row], bar->xchg[xc & 1][t * 2 + 1][row]);
                // lazy rescale: keep the old reference unless the maximum grew by more than 2^TAU
                const bool grow = mx > m_ref + RESCALE_TAU;
                if (__any_sync(0xffffffffu, grow)) {
                    if (j > 0) {
                        // O += P V of block j-1 is complete: s_full of block j was committed after it
                        const float alpha = grow ? fast_exp2(m_ref - mx) : 1.f;
#pragma unroll 1
                        for (int c0 = 0; c0 < D / 2; c0 += 32) {
                            uint32_t o[32];
                            tmem_ld32(tO + c0, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                            tmem_st32(tO + c0, o);
                        }
                        l *= alpha;
                        // the logits are fetched again rather than kept alive across this (rare) path
                        tmem_ld32(tS, a0);
                        tmem_ld32(tS + 32, a1);
                        tmem_wait_ld();
                    }
                    if (grow) m_ref = mx;
                }
                // ---- pass 2: probabilities (bf16, over the first 16 columns of each quarter) and denominator ----
                const uint64_t negm2 = pack2(-m_ref, -m_ref);
                uint64_t sum2 = pack2(0.f, 0.f), sum2b = pack2(0.f, 0.f);
                auto chunk = [&](const uint32_t (&a)[32], uint32_t tP) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        const int c = 2 * i;
                        float x0, x1, x2, x3;
                        unpack2(fma2(pack2(__uint_as_float(a[c]), __uint_as_float(a[c + 1])), scale2, negm2), x0, x1);
                        unpack2(fma2(pack2(__uint_as_float(a[c + 2]), __uint_as_float(a[c + 3])), scale2, negm2), x2, x3);
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = fast_exp2(x3);
                        sum2 = add2(sum2, pack2(p0, p1));
                        sum2b = add2(sum2b, pack2(p2, p3));
                        pk[i] = pack_bf16x2(p0, p1);
                        pk[i + 1] = pack_bf16x2(p2, p3);
                    }
                    asm volatile(
                        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
                        ::"r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]),
                          "r"(pk[8]), "r"(pk[9]), "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15]),
                          "r"(tP)
                        : "memory");
                };
                chunk(a0, tS);
                chunk(a1, tS + 32);
                float s_lo, s_hi;
                unpack2(add2(sum2, sum2b), s_lo, s_hi);
                l += s_lo + s_hi;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&bar->p_ready[t]);
            }
            if (!ok) break;
            ok = mbar_wait(&bar->o_done[t], (uint32_t)k & 1u);
            if (!ok) break;
            tc_fence_after();
            bar->xchg[xc & 1][t * 2 + ch][row] = l;
            asm volatile("bar.sync %0, 64;" ::"r"(bar_id) : "memory");
            const float l_all = bar->xchg[xc & 1][t * 2][row] + bar->xchg[xc & 1][t * 2 + 1][row];
            ++xc;
            const float inv = 1.f / l_all;
            const int64_t qrow = (int64_t)q0 + t * BM + row;
            if (lse && ch == 0 && qrow < n_q) lse[(int64_t)bh * n_q_total + q_row0 + qrow] = m_ref + log2f(l_all);
            __nv_bfloat16 *dst = O + ((int64_t)bh * n_q_total + q_row0 + qrow) * D + ch * (D / 2);
#pragma unroll 1
            for (int c0 = 0; c0 < D / 2; c0 += 32) {
                uint32_t o[32];
                tmem_ld32(tO + c0, o);
                tmem_wait_ld();
                if (c0 + 32 >= D / 2) {
                    // the accumulator is in registers: the next item may overwrite it
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar->o_free[t]);
                }
                if (qrow < n_q) {
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
                        *reinterpret_cast<uint4 *>(dst + c0 + c) = v;
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicExch(status, 3);
        } else {
        // All 16 warps serve the query tile whose logits are ready, tile 0 and tile 1 in turn: while
        // they work on one tile the tensor pipe works on the other.  Warps with the same (warp % 4)
        // share 32 rows (TMEM lanes) and split the block's 128 columns in four quarters; the
        // quarters exchange their row maxima (and, at the end, their denominators) through shared
        // memory, in a buffer per tile so that a value is overwritten only two barriers later.
        const int cq = warp >> 2;                                  // column quarter
        const bool has_tail = tail_start != 0x7fffffff;
        const int row = (warp & 3) * 32 + lane;                    // row in the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        bool ok = true;
        int G = 0;
        for (int k = 0; k < n_items && ok; ++k) {
            const int bh = item_bh(k), q0 = item_q0(k);
            const int64_t life0 = (int64_t)prob_of(bh) * n_pad + cq * 32;     // this thread's first entry of the lifetime arrays
            const int64_t blk0 = (int64_t)prob_of(bh) * nblk;
            float m_ref[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
            const int nb = item_nblk(k);
            for (int j = 0; j < nb && ok; ++j, ++G) {
                // block of the list (j itself unless the launch has block lists); a list may say that the pair sees the
                // block whole - then no lifetime is looked at
                const int blk_entry = item_blk(k, j);
                const int blk = MASKED && tile_cnt ? (blk_entry & BLK_NUMBER) : blk_entry;
                const bool maybe_partly = !(MASKED && tile_cnt) || (blk_entry & BLK_PARTLY) != 0;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    // A row sees the list up to its own entry of the causal tail (if there is one), so
                    // the visible columns are a prefix of the list; of this thread's 32, `valid` exist.
                    // Without a tail every block takes the plain form: the bias MMA has added log2 w and
                    // hidden the columns beyond the list.
                    // `special` must be warp-uniform: both forms of the two passes contain warp-collective TMEM loads.
                    uint32_t vmask = 0xffffffffu;
                    bool special = false;
                    if constexpr (MASKED) {
                        if (birth && maybe_partly) {
                            // lifetimes: the block is seen whole by this warp's 32 rows unless an entry is born
                            // after the first or dies before the last of them
                            const int t_first = q_row0 + q0 + t * BM + (warp & 3) * 32;
                            // (with block lists, a block that comes here is one the list marks as possibly partly visible:
                            // its entries are fetched at once rather than behind the block's summaries)
                            if (tile_cnt) {
                                // Births and deaths do not decrease along a block of such a list (every piece of the
                                // round's list is in order of arrival and no block mixes pieces), so a row sees an
                                // interval of the columns: [entries that died by its token, entries born by it).  Lane c
                                // fetches entry c of this warp's 32 columns and each lane finds its row's two bounds by
                                // bisection over the lanes.
                                const int t_row = t_first + lane;
                                const int32_t b_mine = __ldg(birth + life0 + (int64_t)blk * BN + lane);
                                const int32_t d_mine = __ldg(death + life0 + (int64_t)blk * BN + lane);
                                int hi = 0, lo = 0;
#pragma unroll
                                for (int step = 16; step > 0; step >>= 1) {
                                    if (__shfl_sync(0xffffffffu, b_mine, hi + step - 1) <= t_row) hi += step;
                                    if (__shfl_sync(0xffffffffu, d_mine, lo + step - 1) <= t_row) lo += step;
                                }
                                if (__shfl_sync(0xffffffffu, b_mine, hi) <= t_row) ++hi;          // hi, lo <= 31 here
                                if (__shfl_sync(0xffffffffu, d_mine, lo) <= t_row) ++lo;
                                const uint32_t below_hi = hi >= 32 ? 0xffffffffu : (1u << hi) - 1u;
                                const uint32_t below_lo = lo >= 32 ? 0xffffffffu : (1u << lo) - 1u;
                                vmask = below_hi & ~below_lo;
                                special = __any_sync(0xffffffffu, vmask != 0xffffffffu);          // this warp's rows may see it whole
                            } else {
                            special = !(__ldg(blk_birth + blk0 + blk) <= t_first && __ldg(blk_death + blk0 + blk) > t_first + 31);
                            if (special) {
                                const int t_row = t_first + lane;
                                const int32_t *bp = birth + life0 + (int64_t)blk * BN, *dp = death + life0 + (int64_t)blk * BN;
                                vmask = 0u;
                                // 32 consecutive entries of each array, 128-byte aligned: vector loads
#pragma unroll
                                for (int c = 0; c < 32; c += 4) {
                                    const int4 b4 = __ldg(reinterpret_cast<const int4 *>(bp + c));
                                    const int4 d4 = __ldg(reinterpret_cast<const int4 *>(dp + c));
                                    vmask |= (uint32_t)(b4.x <= t_row && t_row < d4.x) << c;
                                    vmask |= (uint32_t)(b4.y <= t_row && t_row < d4.y) << (c + 1);
                                    vmask |= (uint32_t)(b4.z <= t_row && t_row < d4.z) << (c + 2);
                                    vmask |= (uint32_t)(b4.w <= t_row && t_row < d4.w) << (c + 3);
                                }
                            }
                            }
                        } else if (has_tail) {
                            int valid = n_core - blk * BN - cq * 32;
                            const int64_t seen = (int64_t)tail_start + q0 + t * BM + row + 1;
                            if (seen < n_core) valid = (int)seen - blk * BN - cq * 32;
                            special = __any_sync(0xffffffffu, valid < 32);
                            vmask = valid >= 32 ? 0xffffffffu : (valid <= 0 ? 0u : (1u << valid) - 1u);
                        }
                    }
                    const uint32_t tS = tmem + lane_addr + t * 128 + cq * 32;   // this thread's 32 logit columns
                    const uint32_t tP = tS;                 // their bf16 probabilities overwrite the first 16 of them
                    const uint32_t tO = tmem + lane_addr + 256 + t * 128 + cq * (D / 4);   // its quarter of the accumulator
                    ok = mbar_wait(&bar->s_full[t], (uint32_t)G & 1u);
                    if (!ok) break;
                    tc_fence_after();
                    // ---- pass 1: row maximum over the four quarters ----
                    float mh;
                    uint32_t kept[32];                               // plain form: the logits between the two passes
                    if constexpr (MASKED) mh = special ? row_max<true, 1>(tS, scale_log2, vmask) : row_max<false, 1>(tS, scale_log2, vmask);
                    else mh = row_max_keep(tS, scale_log2, kept);
                    bar->xchg[t][cq][row] = mh;
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + (warp & 3)) : "memory");
                    const float mx = fmaxf(fmaxf(bar->xchg[t][0][row], bar->xchg[t][1][row]),
                                           fmaxf(bar->xchg[t][2][row], bar->xchg[t][3][row]));
                    // lazy rescale: keep the old reference unless the maximum grew by more than 2^TAU
                    const bool grow = mx > m_ref[t] + RESCALE_TAU;
                    if (__any_sync(0xffffffffu, grow)) {
                        if (j > 0) {
                            // O += P V of block j-1 is complete: s_full of block j was committed after it
                            const float alpha = grow ? fast_exp2(m_ref[t] - mx) : 1.f;
                            uint32_t o[32];
                            if (D == 128) tmem_ld32(tO, o);
                            else tmem_ld16(tO, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < D / 4; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                            if (D == 128) tmem_st32(tO, o);
                            else tmem_st16(tO, o);
                            l[t] *= alpha;
                        }
                        if (grow) m_ref[t] = mx;
                    }
                    // ---- pass 2: probabilities and running denominator ----
                    if constexpr (MASKED)
                        l[t] += special ? exp_pass<true, 1>(tS, tP, scale_log2, -m_ref[t], vmask)
                                        : exp_pass<false, 1>(tS, tP, scale_log2, -m_ref[t], vmask);
                    else
                        l[t] += exp_pass_keep(tP, scale_log2, -m_ref[t], kept);
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(&bar->p_ready[t]);
                }
            }
            if (!ok) break;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const uint32_t tO = tmem + lane_addr + 256 + t * 128 + cq * (D / 4);
                ok = mbar_wait(&bar->o_done[t], (uint32_t)k & 1u);
                if (!ok) break;
                tc_fence_after();
                bar->xchg[t][cq][row] = l[t];
                asm volatile("bar.sync %0, 128;" ::"r"(1 + (warp & 3)) : "memory");
                const float l_all = (bar->xchg[t][0][row] + bar->xchg[t][1][row]) + (bar->xchg[t][2][row] + bar->xchg[t][3][row]);
                const float inv = 1.f / l_all;
                const int64_t qrow = (int64_t)q0 + t * BM + row;
                if (lse && cq == 0 && qrow < n_q) lse[(int64_t)bh * n_q_total + q_row0 + qrow] = m_ref[t] + log2f(l_all);
                __nv_bfloat16 *dst = O + ((int64_t)bh * n_q_total + q_row0 + qrow) * D + cq * (D / 4);
                uint32_t o[32];
                if (D == 128) tmem_ld32(tO, o);
                else tmem_ld16(tO, o);
                tmem_wait_ld();
                // the accumulator is in registers: the next item may overwrite it
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar->o_free[t]);
                if (qrow < n_q) {
#pragma unroll
                    for (int c = 0; c < D / 4; c += 8) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
                        *reinterpret_cast<uint4 *>(dst + c) = v;
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicExch(status, 3);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// 3-D bf16 tensor [d2][d1][d0] (d0 contiguous), box {64, box_rows, 1} with the 128-byte swizzle, or
// (narrow) box {16, box_rows, 1} with the 32-byte swizzle
static bool make_map(CUtensorMap *map, const void *base, uint64_t d0, uint64_t d1, uint64_t d2, uint32_t box_rows,
                     bool narrow = false, bool bytes = false)
{
    if (bytes) {
        // 8-bit elements: rows of d0 bytes, boxes of 128 bytes x box_rows, 128-byte swizzle
        sm100::EncodeTiledFn fn8 = sm100::tensor_map_encoder();
        if (!fn8) return false;
        cuuint64_t dims8[3] = {d0, d1, d2};
        cuuint64_t strides8[2] = {d0, d0 * d1};
        cuuint32_t box8[3] = {128u, box_rows, 1};
        cuuint32_t estr8[3] = {1, 1, 1};
        return fn8(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims8, strides8, box8, estr8,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    sm100::EncodeTiledFn fn = sm100::tensor_map_encoder();
    if (!fn) return false;
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {d0 * 2, d0 * d1 * 2};
    cuuint32_t box[3] = {narrow ? 16u : 64u, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, narrow ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int sm_count() { return device_sm_count(); }

// test hook (elm_debug_set): arrivals that the next launch expects on its "probabilities ready" barriers and that
// nobody makes, so that the issuing threads' bounded waits run out
static std::atomic<int> g_debug_extra_arrivals{0};
// test hook: the time limit of the kernel's bounded waits
static std::atomic<unsigned long long> g_debug_wait_limit_ns{sm100::WAIT_LIMIT_NS};

template <int D>
static int launch(const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V, const int32_t *idx,
                  const float *w, int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws,
                  cudaStream_t st, bool timed, const AttendWindow &win)
{
    const int64_t n_q_total = win.n_q_total ? win.n_q_total : (int64_t)p->n_q;
    const AttendLayout L = attend_layout(p, n_core);
    const int n_pad = (n_core + BN - 1) / BN * BN;
    const int problems = p->batch * p->kv_heads;
    __nv_bfloat16 *Kc = reinterpret_cast<__nv_bfloat16 *>(ws + L.Kc);
    __nv_bfloat16 *Vt = reinterpret_cast<__nv_bfloat16 *>(ws + L.Vc);
    __nv_bfloat16 *Bx = reinterpret_cast<__nv_bfloat16 *>(ws + L.bx);
    int *flags = reinterpret_cast<int *>(ws + L.flags);
    int *status = flags + problems;
    CUtensorMap mQ, mK, mV, mX;
    if (!make_map(&mQ, Q, D, (uint64_t)n_q_total, (uint64_t)p->batch * p->q_heads, BM) ||
        !make_map(&mK, Kc, D, (uint64_t)n_pad, (uint64_t)problems, BN) ||
        !make_map(&mV, Vt, BN, D, (uint64_t)problems * (uint64_t)(n_pad / BN), D) ||
        !make_map(&mX, Bx, 16, (uint64_t)n_pad, (uint64_t)problems, BN, true))
        return ELM_ERR_CUDA;
    const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)D));
    {
        StageTimer t(timed ? ELM_STAGE_GATHER : -1, st, 1);
        ELM_CUDA_TRY(cudaMemsetAsync(flags, 0, sizeof(int) * (size_t)(problems + 1), st));
        gather_tc_kernel<D><<<dim3((unsigned)(n_pad / GATHER_COLS), (unsigned)problems), 256, 0, st>>>(
            K, V, idx, w, p->n_kv, n_core, n_pad, Kc, Vt, Bx, 1.f / scale_log2, flags);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    StageTimer t(timed ? ELM_STAGE_ATTEND : -1, st, 1);
    const bool masked = win.birth != nullptr || win.tail_start != 0x7fffffff;
    auto kern = masked ? attend_tc_kernel<D, true> : attend_tc_kernel<D, false>;
    ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::TOTAL));
    // one persistent CTA per SM, each taking every gridDim.x-th pair of query tiles
    const int tiles_x = (p->n_q + 2 * BM - 1) / (2 * BM);
    const int64_t items = (int64_t)tiles_x * p->batch * p->q_heads;
    if (items > 0x7fffffff / 64 || (int64_t)problems * n_pad > 0x7fffffff - 256) return ELM_ERR_SHAPE;
    const int ctas = win.item_tab ? win.item_ctas : (int)(items < sm_count() ? items : sm_count());
    kern<<<ctas, NTHREADS, Smem<D>::TOTAL, st>>>(mQ, mK, mV, mX, flags, O, p->q_heads, p->kv_heads, p->n_q,
                                                 n_core, n_pad, scale_log2, tiles_x, (int)items, (int)win.q_row0,
                                                 (int)n_q_total, win.tail_start, win.birth, win.death, win.blk_birth,
                                                 win.blk_death, win.lse, status, g_debug_extra_arrivals.exchange(0),
                                                 g_debug_wait_limit_ns.load(), win.tile_cnt, win.tile_blk, win.tile_cap, win.item_tab, win.item_cnt, win.item_cap);
    count_launches(1);
    return cuda_status(cudaGetLastError());
}

// E4M3 inputs, d = 128, no mask: the same kernel with 8-bit Q and K tiles
static int launch_e4m3(const unsigned char *Q, const unsigned char *K, const unsigned char *V, const int32_t *idx, const float *w,
                       int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws, cudaStream_t st, bool timed)
{
    constexpr int D = 128;
    const AttendLayout L = attend_layout(p, n_core);
    const int n_pad = (n_core + BN - 1) / BN * BN;
    const int problems = p->batch * p->kv_heads;
    unsigned char *Kc = ws + L.Kc;                                  // [problems][n_pad][D] bytes
    __nv_bfloat16 *Vt = reinterpret_cast<__nv_bfloat16 *>(ws + L.Vc);
    __nv_bfloat16 *Bx = reinterpret_cast<__nv_bfloat16 *>(ws + L.bx);
    int *flags = reinterpret_cast<int *>(ws + L.flags);
    int *status = flags + problems;
    CUtensorMap mQ, mK, mV, mX;
    if (!make_map(&mQ, Q, D, (uint64_t)p->n_q, (uint64_t)p->batch * p->q_heads, BM, false, true) ||
        !make_map(&mK, Kc, D, (uint64_t)n_pad, (uint64_t)problems, BN, false, true) ||
        !make_map(&mV, Vt, BN, D, (uint64_t)problems * (uint64_t)(n_pad / BN), D) ||
        !make_map(&mX, Bx, 16, (uint64_t)n_pad, (uint64_t)problems, BN, true))
        return ELM_ERR_CUDA;
    const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)D));
    {
        StageTimer t(timed ? ELM_STAGE_GATHER : -1, st, 1);
        ELM_CUDA_TRY(cudaMemsetAsync(flags, 0, sizeof(int) * (size_t)(problems + 1), st));
        gather_tc_kernel<D, true><<<dim3((unsigned)(n_pad / GATHER_COLS), (unsigned)problems), 256, 0, st>>>(
            reinterpret_cast<const __nv_bfloat16 *>(K), reinterpret_cast<const __nv_bfloat16 *>(V), idx, w, p->n_kv, n_core, n_pad,
            reinterpret_cast<__nv_bfloat16 *>(Kc), Vt, Bx, 1.f / scale_log2, flags);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    StageTimer t(timed ? ELM_STAGE_ATTEND : -1, st, 1);
    auto kern = attend_tc_kernel<D, false, 1>;
    ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D, 1>::TOTAL));
    const int tiles_x = (p->n_q + 2 * BM - 1) / (2 * BM);
    const int64_t items = (int64_t)tiles_x * p->batch * p->q_heads;
    if (items > 0x7fffffff / 64) return ELM_ERR_SHAPE;
    const int ctas = (int)(items < sm_count() ? items : sm_count());
    kern<<<ctas, NTHREADS, Smem<D, 1>::TOTAL, st>>>(mQ, mK, mV, mX, flags, O, p->q_heads, p->kv_heads, p->n_q, n_core, n_pad,
                                                    scale_log2, tiles_x, (int)items, 0, p->n_q, 0x7fffffff, nullptr, nullptr, nullptr,
                                                    nullptr, nullptr, status, g_debug_extra_arrivals.exchange(0),
                                                    g_debug_wait_limit_ns.load(), nullptr, nullptr, 0, nullptr, nullptr, 0);
    count_launches(1);
    return cuda_status(cudaGetLastError());
}

}  // namespace tc

int attend_tc_e4m3(const unsigned char *Q, const unsigned char *K, const unsigned char *V, const int32_t *idx, const float *w,
                   int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws, cudaStream_t st, bool timed)
{
    return tc::launch_e4m3(Q, K, V, idx, w, n_core, p, O, ws, st, timed);
}

int debug_set_attend_tc(int32_t what, int64_t value)
{
    if (what == ELM_DEBUG_WAIT_LIMIT_NS) {
        if (value < 1000000) return ELM_ERR_SHAPE;              // at least a millisecond
        tc::g_debug_wait_limit_ns.store((unsigned long long)value);
        return ELM_OK;
    }
    if (what == ELM_DEBUG_ATTEND_MISSING_ARRIVALS) {
        if (value < 0 || value > 1024) return ELM_ERR_SHAPE;
        tc::g_debug_extra_arrivals.store((int)value);
        return ELM_OK;
    }
    return ELM_ERR_SHAPE;
}

int attend_tc(const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V, const int32_t *idx,
              const float *w, int n_core, const elm_params *p, __nv_bfloat16 *O, unsigned char *ws,
              cudaStream_t st, bool timed, const AttendWindow &win)
{
    if (p->d == 64) return tc::launch<64>(Q, K, V, idx, w, n_core, p, O, ws, st, timed, win);
    return tc::launch<128>(Q, K, V, idx, w, n_core, p, O, ws, st, timed, win);
}

}  // namespace elm

