// Kernel evaluation for one Compress2 level on the sm_100a tensor cores (bf16 inputs, fp32 mode).
//
// A CTA produces one 64 x 64 tile of the pair Gram F = P G P^T, i.e. a 128 x 128 tile of
//   G[a,b] = exp(<k_a,k_b>/sqrt(d) - M_pair(b)) * (<v_a,v_b> + v_max^2)                Eq. (katt), shifted
// The 128 row points and 128 column points are gathered through the level's index list straight
// into the 128-byte-swizzled K-major layout tcgen05.mma reads (rows are never copied in HBM).
// Two accumulators in TMEM hold K K^T and V V^T; the epilogue applies the exponential, the
// product and the +/- pair combination F[j,i] = G[2j,2i] - G[2j,2i+1] - G[2j+1,2i] + G[2j+1,2i+1]
// (Algorithm A.1's <f_j, f_i>) and stores only j <= i within one Halve call.
#include <math.h>

#include "elm_common.cuh"
#include "elm_compress.cuh"
#include "elm_sm100.cuh"
#include "elm_walk.cuh"

namespace elm {
namespace gramtc {

using namespace sm100;

constexpr int TP = 64;            // pairs per tile side
constexpr int TR = 128;           // points per tile side
constexpr int NTHREADS = 256;
constexpr uint32_t TMEM_COLS = 256;

// Shared memory holds ONE pair of operand tiles (row points, column points): the keys first, then,
// once K K^T has been consumed, the values in the same place.  64 KB (d = 128) lets two CTAs share
// an SM, so one CTA's gather overlaps the other's MMAs and epilogue.
template <int D> struct Smem {
    static constexpr int KH = D / 64;
    static constexpr int OPERAND = TR * D * 2;                 // one 128-row operand tile, bytes
    static constexpr int OFF_A = 0, OFF_B = OPERAND;
    static constexpr int OFF_MISC = 2 * OPERAND;
    static constexpr int TOTAL = OFF_MISC + 2048 + 1024;       // misc block + alignment slack
};

struct Misc {
    uint64_t mma_done[2];        // K K^T done, V V^T done
    uint32_t tmem_base;
    uint32_t pad;
    float colshift[TP];          // M of each pair column, in log2 units
    float rdec[TP], unif[TP];    // fused walk: decay factor and uniform of each pair of the tile
    int32_t rowsA[TR], rowsB[TR];
};

constexpr int FS_LD = 68;         // row stride of the shared-memory pair Gram of a fused tile (floats)

// Halving walk (Algorithm A.1) of the calls that lie inside one 64-pair tile, on the tile's pair
// Gram in shared memory: warp w walks call w of the tile (P = 16, 32 or 64 pairs per call) in blocks
// of 32 pairs with the warp-cooperative block walker; the first block of a 64-pair call folds its
// decisions into the second block's scores as it goes.
__device__ __forceinline__ void walk_in_tile(const float *Fs, const float *rdec, const float *unif, int p,
                                             int64_t JR, int P, int64_t Ptotal, int64_t n,
                                             const int32_t *__restrict__ cur, const WalkArgs &wk, int warp, int lane)
{
    const int calls = TP / P;
    if (warp >= calls) return;
    const int64_t J0 = JR + (int64_t)warp * P;                 // first pair of this call along the level's sequence
    if (J0 >= Ptotal) return;
    const float *Fc = Fs + (warp * P) * FS_LD + warp * P;      // the call's P x P block
    float bmax = 0.f, dn = 0.f;
    for (int blk = 0; blk * 32 < P; ++blk) {
        const int i = blk * 32 + lane;                         // pair within the call
        const bool live = i < P;
        const float dgn = live ? Fc[i * FS_LD + i] : 0.f;
        const float a = walk_block_thresholds(sqrtf(dgn > 0.f ? dgn : 0.f), live ? rdec[warp * P + i] : 1.f, bmax,
                                              wk.logfac, lane);
        // the previous block already folded its decisions into this block's scores (dn); pairs
        // past the end of a short call come after the live ones and decide nothing
        const float d = walk_sign_score(dn, a, live ? unif[warp * P + i] : 1.f);
        dn = 0.f;
        const uint32_t swaps = walk_block_warp(Fc + (blk * 32) * FS_LD + blk * 32, FS_LD, d, dn, lane);
        if (live) {
            const uint32_t sw = (swaps >> lane) & 1u;
            wk.out[(int64_t)p * wk.out_stride + J0 + i] = cur[(int64_t)p * n + 2 * (J0 + i) + sw];
        }
    }
}

// Gather 128 rows of X (row-major [n][D] bf16) into a swizzled K-major operand tile.
template <int D>
__device__ __forceinline__ void gather_operand(unsigned char *dst, const __nv_bfloat16 *__restrict__ X,
                                               const int32_t *rows, int tid)
{
    constexpr int CHUNKS = D / 8;                              // 16-byte chunks per row
    const uint32_t dst_s = smem_u32(dst);
#pragma unroll
    for (int q = tid; q < TR * CHUNKS; q += NTHREADS) {
        const int r = q / CHUNKS, ch = q % CHUNKS;
        const int kh = ch >> 3, c = ch & 7;
        // asynchronous 16-byte copies: all of a thread's chunks are in flight at once
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_s + kh * (TR * 128) + (r >> 3) * 1024 +
                                                                        (r & 7) * 128 + ((c ^ (r & 7)) << 4)),
                     "l"(X + (int64_t)rows[r] * D + ch * 8)
                     : "memory");
    }
}

template <int D>
__global__ void __launch_bounds__(NTHREADS, 2)
gram_tc_kernel(const __nv_bfloat16 *__restrict__ K, const __nv_bfloat16 *__restrict__ V,
               const int32_t *__restrict__ cur, const float *__restrict__ Mpair,
               const unsigned *__restrict__ vmax_bits, int64_t n, int P, int64_t Ptotal,
               float *__restrict__ F, int64_t F_stride, int *__restrict__ status, WalkArgs wk)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    using SM = Smem<D>;
    constexpr int KH = SM::KH;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    Misc *misc = reinterpret_cast<Misc *>(smem + SM::OFF_MISC);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int p = blockIdx.y;

    if (*reinterpret_cast<volatile int *>(status) != 0) return;

    int64_t JR, JC;
    if (P >= TP) {
        const int Tg = P / TP, ntri = Tg * (Tg + 1) / 2;
        const int g = blockIdx.x / ntri, local = blockIdx.x % ntri;
        int tc = (int)((sqrtf(8.f * (float)local + 1.f) - 1.f) * 0.5f);
        while ((tc + 1) * (tc + 2) / 2 <= local) ++tc;
        while (tc * (tc + 1) / 2 > local) --tc;
        const int tr = local - tc * (tc + 1) / 2;
        JR = (int64_t)g * P + tr * TP;
        JC = (int64_t)g * P + tc * TP;
    } else {
        JR = JC = (int64_t)blockIdx.x * TP;
    }
    const bool diagonal = JR == JC;
    const int32_t *curp = cur + (int64_t)p * n;
    const float LOG2E = 1.4426950408889634f;
    if (tid < TR) {
        const int64_t pt = 2 * JR + tid;
        misc->rowsA[tid] = pt < 2 * Ptotal ? curp[pt] : 0;
    } else {
        const int64_t pt = 2 * JC + (tid - TR);
        misc->rowsB[tid - TR] = pt < 2 * Ptotal ? curp[pt] : 0;
    }
    if (tid < TP) {
        const int64_t jc = JC + tid;
        misc->colshift[tid] = jc < Ptotal ? Mpair[(int64_t)p * (n / 2) + jc] * LOG2E : 0.f;
        if (wk.fused) {
            // everything the in-tile walk needs from global memory, fetched while the tile is built
            misc->rdec[tid] = jc < Ptotal ? wk.rdecay[(int64_t)p * (n / 2) + jc] : 1.f;
            uint32_t cgroup, ccode;
            call_counter((int)(jc / P), wk.level, cgroup, ccode);
            misc->unif[tid] = halving_uniform<float>(wk.seed, (uint32_t)(jc % P), cgroup, ccode, (uint32_t)p + wk.pbase);
        }
    }
    if (tid == 0) {
        mbar_init(&misc->mma_done[0], 1);
        mbar_init(&misc->mma_done[1], 1);
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&misc->tmem_base, TMEM_COLS);
    __syncthreads();

    const __nv_bfloat16 *Kp = K + (int64_t)p * n * D;
    const __nv_bfloat16 *Vp = V + (int64_t)p * n * D;
    constexpr uint32_t IDESC = umma_idesc_bf16(TR, TR);
    const uint32_t sA = smem_u32(smem + SM::OFF_A);
    const uint32_t sB = smem_u32(smem + SM::OFF_B);
    uint32_t tmem = 0;
    bool ok = true;
    auto issue = [&](int acc, uint32_t a_addr, uint32_t b_addr) {     // one 128 x 128 x D product into accumulator `acc`
#pragma unroll
        for (int kh = 0; kh < KH; ++kh)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                mma_ss(tmem + acc * 128, umma_desc_k128(a_addr + kh * (TR * 128) + ks * 32),
                       umma_desc_k128(b_addr + kh * (TR * 128) + ks * 32), IDESC, (kh | ks) != 0);
    };
    auto publish = [&]() {                                            // make the gathered tiles visible to the MMAs
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        tmem = misc->tmem_base;
    };
    if (diagonal) {
        // row points = column points: keys in the first slot, values in the second, one gather round
        gather_operand<D>(smem + SM::OFF_A, Kp, misc->rowsA, tid);
        gather_operand<D>(smem + SM::OFF_B, Vp, misc->rowsA, tid);
        publish();
        if (tid == 0) {
            const uint32_t sV = smem_u32(smem + SM::OFF_B);
            issue(0, sA, sA);
            issue(1, sV, sV);
            tc_commit(&misc->mma_done[1]);
        }
        ok = mbar_wait(&misc->mma_done[1], 0);
    } else {
#pragma unroll
        for (int phase = 0; phase < 2; ++phase) {              // 0: keys -> K K^T, 1: values -> V V^T
            const __nv_bfloat16 *X = phase == 0 ? Kp : Vp;
            gather_operand<D>(smem + SM::OFF_A, X, misc->rowsA, tid);
            gather_operand<D>(smem + SM::OFF_B, X, misc->rowsB, tid);
            publish();
            if (tid == 0) {
                issue(phase, sA, sB);
                tc_commit(&misc->mma_done[phase]);
            }
            // the operand tiles are reused by the next phase only after the MMAs have read them
            ok = ok && mbar_wait(&misc->mma_done[phase], 0);
        }
    }

    // epilogue: warp w owns TMEM lanes 32 (w % 4) .. +31 (tile rows) and the column half w / 4
    if (ok) {
        tc_fence_after();
        const int r = (warp & 3) * 32 + lane;                 // point row in the tile
        const int ch = warp >> 2;                             // columns [64 ch, 64 ch + 64)
        const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + ch * 64;
        const float vm = __uint_as_float(vmax_bits[p]);
        const float vm2 = vm * vm;
        const float qscale = LOG2E / sqrtf((float)D);
        float h[32];                                          // G[r,2i] - G[r,2i+1] for the 32 pair columns
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            uint32_t kk[32], vv[32];
            tmem_ld32(taddr + q * 32, kk);
            tmem_ld32(taddr + 128 + q * 32, vv);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
                const float sh = misc->colshift[ch * 32 + q * 16 + (c >> 1)];
                float e0 = fmaf(__uint_as_float(kk[c]), qscale, -sh);
                float e1 = fmaf(__uint_as_float(kk[c + 1]), qscale, -sh);
                float g0 = e0 < -115.f ? 0.f : fast_exp2(e0) * (__uint_as_float(vv[c]) + vm2);
                float g1 = e1 < -115.f ? 0.f : fast_exp2(e1) * (__uint_as_float(vv[c + 1]) + vm2);
                h[q * 16 + (c >> 1)] = g0 - g1;
            }
        }
        // pair rows are adjacent lanes: the even lane finishes pair columns 0..15 of its 32, the odd
        // lane columns 16..31
        const bool odd = lane & 1;
        float f[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float send = odd ? h[i] : h[i + 16];
            const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
            f[i] = odd ? recv - h[i + 16] : h[i] - recv;
        }
        const int64_t jr = JR + (r >> 1);
        const int64_t jc0 = JC + ch * 32 + (odd ? 16 : 0);
        if (wk.fused) {
            // calls of at most 64 pairs lie inside this (diagonal) tile: keep the pair Gram in shared
            // memory (over the operand tiles, which the MMAs have finished reading) and walk here
            float *Fs = reinterpret_cast<float *>(smem + SM::OFF_A);
#pragma unroll
            for (int i = 0; i < 16; ++i) Fs[(r >> 1) * FS_LD + ch * 32 + (odd ? 16 : 0) + i] = f[i];
        } else {
            float *Fp = F + (int64_t)p * F_stride;
            if (jr < Ptotal) {
                const int64_t gr = jr / P;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int64_t jc = jc0 + i;
                    if (jc < Ptotal && jr <= jc && jc / P == gr) Fp[jr * P + (jc - gr * P)] = f[i];
                }
            }
        }
    } else if (lane == 0) {
        atomicExch(status, 4);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
    if (wk.fused && ok) walk_in_tile(reinterpret_cast<float *>(smem + SM::OFF_A),
                                     misc->rdec, misc->unif, p, JR, P, Ptotal, n, cur, wk, warp, lane);
}

// ---------------------------------------------------------------------------------------------
// Persistent, pipelined variant for levels whose calls span several tiles (P > 64 pairs).
// One CTA per SM walks the level's tile list (tile, problem) round-robin.  Roles:
//   warps 0-3   loaders: gather the tile's row and column points with 16-byte cp.async into a ring
//               of three 64 KB operand buffers -- one "job" for the keys, one for the values of each
//               tile -- and let the copies' completion arrive on the job's mbarrier, so up to three
//               jobs are in flight while earlier ones are multiplied
//   warp 4      issues the tcgen05.mma of each job into one of two TMEM accumulator slots
//               (K K^T | V V^T, 256 columns each); its commits free the operand buffers
//   warps 5-12  epilogue of the previous tile (exp2, product, pair combination, stores) while the
//               next tile is gathered and multiplied
// ---------------------------------------------------------------------------------------------
constexpr int PNS = 3;                       // operand ring depth (jobs)
constexpr int PLOAD = 4;                      // loader warps (8 were slower: 0.76 against 0.71 ms per cfg5 step)
constexpr int PTHREADS = (PLOAD + 1 + 8) * 32;   // loaders, the MMA issuer, 8 epilogue warps
constexpr int PTAB = 256;                    // items of a CTA whose tiles are decoded up front

struct PBarriers {
    uint64_t full[PNS], empty[PNS], accfull[2], accempty[2];
    uint32_t tmem_base;
    uint32_t pad;
};

template <int D> struct PSmem {
    static constexpr int JOB = 2 * TR * D * 2;                // row tile + column tile of one operand type
    static constexpr int OFF_BAR = PNS * JOB;
    static constexpr int TOTAL = OFF_BAR + 1024 + 1024;
};

__device__ __forceinline__ void decode_tile(int tile, int P, int64_t &JR, int64_t &JC)
{
    const int Tg = P / TP, ntri = Tg * (Tg + 1) / 2;
    const int g = tile / ntri, local = tile % ntri;
    int tc = (int)((sqrtf(8.f * (float)local + 1.f) - 1.f) * 0.5f);
    while ((tc + 1) * (tc + 2) / 2 <= local) ++tc;
    while (tc * (tc + 1) / 2 > local) --tc;
    const int tr = local - tc * (tc + 1) / 2;
    JR = (int64_t)g * P + tr * TP;
    JC = (int64_t)g * P + tc * TP;
}

template <int D>
__global__ void __launch_bounds__(PTHREADS, 1)
gram_tc_persistent_kernel(const __nv_bfloat16 *__restrict__ K, const __nv_bfloat16 *__restrict__ V,
                          const int32_t *__restrict__ cur, const float *__restrict__ Mpair,
                          const unsigned *__restrict__ vmax_bits, int64_t n, int P, int tiles_per_problem,
                          int total_items, float *__restrict__ F, int64_t F_stride, int *__restrict__ status)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    using SM = PSmem<D>;
    constexpr int KH = D / 64;
    constexpr int CHUNKS = D / 8;                             // 16-byte chunks per row
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    PBarriers *bar = reinterpret_cast<PBarriers *>(smem + SM::OFF_BAR);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (*reinterpret_cast<volatile int *>(status) != 0) return;
    // Which tile is item k of this CTA?  Decoding a tile number (two divisions, a square root) costs a lone
    // thread about 900 cycles - a quarter of a tile's time on the MMA issuer - so all threads decode the CTA's
    // items once, in parallel, into a table.
    __shared__ int tab_p[PTAB], tab_jr[PTAB], tab_jc[PTAB];
    for (int i = tid; i < PTAB; i += PTHREADS) {
        const int it = blockIdx.x + i * gridDim.x;
        if (it < total_items) {
            int64_t jr, jc;
            decode_tile(it % tiles_per_problem, P, jr, jc);
            tab_p[i] = it / tiles_per_problem;
            tab_jr[i] = (int)jr;
            tab_jc[i] = (int)jc;
        }
    }
    auto item = [&](int k, int it, int &p, int64_t &JR, int64_t &JC) {
        if (k < PTAB) {
            p = tab_p[k]; JR = tab_jr[k]; JC = tab_jc[k];
        } else {
            p = it / tiles_per_problem;
            decode_tile(it % tiles_per_problem, P, JR, JC);
        }
    };
    if (tid == 0) {
        for (int b = 0; b < PNS; ++b) { mbar_init(&bar->full[b], PLOAD * 32); mbar_init(&bar->empty[b], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&bar->accfull[s], 1); mbar_init(&bar->accempty[s], 256); }
        fence_barrier_init();
    }
    if (warp == PLOAD) tmem_alloc(&bar->tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;
    bool ok = true;

    if (warp < PLOAD) {
        // ------------------------------ loaders ------------------------------
        int job = 0, lk = 0;
        for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x, ++lk) {
            int p;
            int64_t JR, JC;
            item(lk, it, p, JR, JC);
            const bool diagonal = JR == JC;
            const int32_t *curp = cur + (int64_t)p * n;
            // chunk q = tid + NL i of a 128-row tile lies in row tid / CHUNKS + (NL / CHUNKS) i, NL loader threads
            constexpr int NL = PLOAD * 32;
            constexpr int RPT = TR * CHUNKS / NL;            // chunks (= distinct rows) per thread and tile
            int32_t ra[RPT], rb[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int r = tid / CHUNKS + (NL / CHUNKS) * i;
                ra[i] = __ldg(curp + 2 * JR + r);
                rb[i] = diagonal ? 0 : __ldg(curp + 2 * JC + r);
            }
            const int ch = tid % CHUNKS, kh = ch >> 3, c = ch & 7;
            for (int op = 0; op < 2 && ok; ++op, ++job) {     // 0: keys, 1: values
                const int b = job % PNS;
                ok = mbar_wait(&bar->empty[b], ((uint32_t)(job / PNS) & 1u) ^ 1u);
                if (!ok) break;
                const __nv_bfloat16 *X = (op == 0 ? K : V) + (int64_t)p * n * D;
                const uint32_t dstA = smem_u32(smem + b * SM::JOB), dstB = dstA + TR * D * 2;
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    const int r = tid / CHUNKS + (NL / CHUNKS) * i;
                    const uint32_t off = kh * (TR * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4);
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dstA + off), "l"(X + (int64_t)ra[i] * D + ch * 8) : "memory");
                    if (!diagonal)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dstB + off), "l"(X + (int64_t)rb[i] * D + ch * 8) : "memory");
                }
                // the job's barrier completes when every loader thread's copies have landed
                asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&bar->full[b])) : "memory");
            }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        if (!ok && lane == 0) atomicExch(status, 5);
    } else if (warp == PLOAD) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr uint32_t IDESC = umma_idesc_bf16(TR, TR);
            int job = 0, k = 0;
            for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x, ++k) {
                int p;
                int64_t JR, JC;
                item(k, it, p, JR, JC);
                const bool diagonal = JR == JC;
                const int slot = k & 1;
                ok = mbar_wait(&bar->accempty[slot], ((uint32_t)(k >> 1) & 1u) ^ 1u);
                if (!ok) break;
                tc_fence_after();
                for (int op = 0; op < 2 && ok; ++op, ++job) {
                    const int b = job % PNS;
                    ok = mbar_wait(&bar->full[b], (uint32_t)(job / PNS) & 1u);
                    if (!ok) break;
                    fence_proxy_async();                       // the gathered bytes were written by generic-proxy copies
                    tc_fence_after();
                    const uint32_t sA = smem_u32(smem + b * SM::JOB), sB = diagonal ? sA : sA + TR * D * 2;
#pragma unroll
                    for (int kh = 0; kh < KH; ++kh)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_ss(tmem + slot * 256 + op * 128, umma_desc_k128(sA + kh * (TR * 128) + ks * 32),
                                   umma_desc_k128(sB + kh * (TR * 128) + ks * 32), IDESC, (kh | ks) != 0);
                    tc_commit(&bar->empty[b]);
                }
                if (ok) tc_commit(&bar->accfull[slot]);
            }
            if (!ok) atomicExch(status, 6);
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int e = warp - (PLOAD + 1);                     // 0..7
        const int q4 = warp & 3;                              // TMEM lane quarter this warp may access
        const int ch = e >> 2;                                // column half
        const int r = q4 * 32 + lane;                         // point row in the tile
        const float LOG2E = 1.4426950408889634f;
        const float qscale = LOG2E / sqrtf((float)D);
        int k = 0;
        for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x, ++k) {
            int p;
            int64_t JR, JC;
            item(k, it, p, JR, JC);
            const int slot = k & 1;
            const float vm = __uint_as_float(vmax_bits[p]);
            const float vm2 = vm * vm;
            // running shifts of this thread's 32 pair columns (in log2 units), fetched while the MMAs run
            float sh[32];
            {
                // 32 consecutive floats, 128-byte aligned (n / 2 and JC are multiples of 32)
                const float4 *mp = reinterpret_cast<const float4 *>(Mpair + (int64_t)p * (n / 2) + JC + ch * 32);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 v = __ldg(mp + i);
                    sh[4 * i] = v.x * LOG2E; sh[4 * i + 1] = v.y * LOG2E; sh[4 * i + 2] = v.z * LOG2E; sh[4 * i + 3] = v.w * LOG2E;
                }
            }
            ok = mbar_wait(&bar->accfull[slot], (uint32_t)(k >> 1) & 1u);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + slot * 256 + ch * 64;
            float h[32];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t kk[32], vv[32];
                tmem_ld32(taddr + q * 32, kk);
                tmem_ld32(taddr + 128 + q * 32, vv);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    const float shc = sh[q * 16 + (c >> 1)];
                    float e0 = fmaf(__uint_as_float(kk[c]), qscale, -shc);
                    float e1 = fmaf(__uint_as_float(kk[c + 1]), qscale, -shc);
                    float g0 = e0 < -115.f ? 0.f : fast_exp2(e0) * (__uint_as_float(vv[c]) + vm2);
                    float g1 = e1 < -115.f ? 0.f : fast_exp2(e1) * (__uint_as_float(vv[c + 1]) + vm2);
                    h[q * 16 + (c >> 1)] = g0 - g1;
                }
            }
            // the accumulator slot is free as soon as its values are in registers
            tc_fence_before();
            mbar_arrive(&bar->accempty[slot]);
            const bool odd = lane & 1;
            float f[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float send = odd ? h[i] : h[i + 16];
                const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
                f[i] = odd ? recv - h[i + 16] : h[i] - recv;
            }
            const int64_t jr = JR + (r >> 1);
            const int64_t jc0 = JC + ch * 32 + (odd ? 16 : 0);
            const int64_t gr = jr / P;
            float *Fp = F + (int64_t)p * F_stride + jr * P - gr * P;
            // 64 contiguous bytes per thread.  On a diagonal tile half of them lie below the diagonal of the
            // call's P x P block, which nothing reads: written all the same, four vector stores being
            // cheaper than sixteen predicated ones.
#pragma unroll
            for (int i = 0; i < 16; i += 4)
                *reinterpret_cast<float4 *>(Fp + jc0 + i) = make_float4(f[i], f[i + 1], f[i + 2], f[i + 3]);
        }
        if (!ok && lane == 0) atomicExch(status, 7);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == PLOAD) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

template <int D>
static int launch(const __nv_bfloat16 *K, const __nv_bfloat16 *V, const elm_params *p, const int32_t *cur,
                  const float *Mpair, const unsigned *vmax_bits, int P, int64_t Ptotal, int groups, float *F,
                  int64_t F_stride, int *status, const WalkArgs &wk, cudaStream_t st)
{
    const int BH = p->batch * p->kv_heads;
    int64_t tiles;
    if (P >= TP) {
        const int Tg = P / TP;
        tiles = (int64_t)groups * (Tg * (Tg + 1) / 2);
    } else {
        tiles = (Ptotal + TP - 1) / TP;
    }
    if (P > TP || (P == TP && !wk.fused)) {
        // calls that span several tiles: persistent, pipelined kernel, one CTA per SM
        const int sm_count = device_sm_count();
        const int64_t total = tiles * BH;
        const int grid = (int)(total < sm_count ? total : sm_count);
        auto pk = gram_tc_persistent_kernel<D>;
        ELM_CUDA_TRY(cudaFuncSetAttribute(pk, cudaFuncAttributeMaxDynamicSharedMemorySize, PSmem<D>::TOTAL));
        ELM_CUDA_TRY(launch_after(pk, dim3((unsigned)grid), dim3(PTHREADS), (size_t)PSmem<D>::TOTAL, st, K, V, cur, Mpair, vmax_bits,
                                  p->n_kv, P, (int)tiles, (int)total, F, F_stride, status));
        count_launches(1);
        return cuda_status(cudaGetLastError());
    }
    auto kern = gram_tc_kernel<D>;
    ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::TOTAL));
    ELM_CUDA_TRY(launch_after(kern, dim3((unsigned)tiles, (unsigned)BH), dim3(NTHREADS), (size_t)Smem<D>::TOTAL, st, K, V, cur, Mpair, vmax_bits,
                              p->n_kv, P, Ptotal, F, F_stride, status, wk));
    count_launches(1);
    return cuda_status(cudaGetLastError());
}

}  // namespace gramtc

int gram_tc(const __nv_bfloat16 *K, const __nv_bfloat16 *V, const elm_params *p, const int32_t *cur,
            const float *Mpair, const unsigned *vmax_bits, int P, int64_t Ptotal, int groups, float *F,
            int64_t F_stride, int *status, const WalkArgs &wk, cudaStream_t st)
{
    if (p->d == 64) return gramtc::launch<64>(K, V, p, cur, Mpair, vmax_bits, P, Ptotal, groups, F, F_stride, status, wk, st);
    return gramtc::launch<128>(K, V, p, cur, Mpair, vmax_bits, P, Ptotal, groups, F, F_stride, status, wk, st);
}

}  // namespace elm
