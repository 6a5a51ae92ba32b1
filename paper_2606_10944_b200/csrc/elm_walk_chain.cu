// The halving walk of Algorithm A.1 for calls of at least 32 pairs, as a chain of 32-pair blocks.
//
// The walk of one Halve call is a single serial chain over its P pairs; what can run beside the
// chain is everything that does not depend on the decisions:
//   - streaming the call's P x P pair Gram F (row j = earlier pair, column i = later pair),
//   - the thresholds a_i = b_i b_max,i (1/2 + ln(2s/delta)), which depend on F's diagonal only,
//   - folding DECIDED blocks into the scores alpha_i = -sum_j eta_j F[j,i] of later columns.
// One CTA, or for long calls one thread-block cluster, handles a call.  CTA k of a cluster of C owns
// the columns [k W, (k+1) W), W = P / C, and reads only the rows above the end of its own diagonal
// block, W columns wide, so no SM has to pull the whole Gram through itself.  Row panel R = rows
// [32 R, 32 R + 32) x own columns is fetched by bulk asynchronous copies into a ring of shared-memory
// buffers that runs ahead of the chain.  A CTA first folds the panels of earlier CTAs' blocks as
// their swap masks arrive (the owner writes each mask into every later CTA's shared memory and
// raises that CTA's progress word with a release), then walks its own W / 32 blocks.
//
// Warp roles: warp 0 walks, warp 1 issues copies and publishes masks, warp 2 prepares thresholds and
// next-block scores, warps 3.. fold decided panels into later columns.  One CTA barrier per block.
#include <math.h>
#include <stdlib.h>

#include <type_traits>

#include "elm_common.cuh"
#include "elm_compress.cuh"
#include "elm_sm100.cuh"
#include "elm_walk.cuh"

namespace elm {
namespace {

constexpr int MAX_CLUSTER = 16;          // above 8 the cluster size is "non-portable": opt-in, and checked for schedulability
constexpr int UPD_THREADS_MAX = 256;
constexpr uint32_t FULL = 0xffffffffu;

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of `local` (a shared-memory address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// progress words only grow; a maximum keeps them monotonic whichever CTA's update lands last
__device__ __forceinline__ void red_max_release_cluster_u32(uint32_t addr, uint32_t v)
{
    asm volatile("red.release.cluster.shared::cluster.max.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_cluster_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.cluster.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)) : "memory");
    return v;
}
// Bounded wait until *word > want (about 2 s)
__device__ __forceinline__ bool wait_progress(const uint32_t *word, uint32_t want)
{
    if (ld_acquire_cluster_u32(word) > want) return true;
    uint64_t t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (ld_acquire_cluster_u32(word) > want) return true;
        uint64_t t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > 2000000000ull) return false;
    }
}

// Shared-memory plan (byte offsets) for a call of P pairs split over C CTAs, element size es.
struct ChainSmem {
    size_t panels, alpha, a, U, ball, rall, xnext, mask, ctl, total;
    int NB;   // ring depth; < 3 means the call does not fit
};
__host__ __device__ inline ChainSmem chain_smem(int P, int C, int es, int nb_cap)
{
    ChainSmem s{};
    const int W = P / C;
    if (W < 32) return s;
    const size_t panel = (size_t)32 * W * es;
    const size_t fixed = (size_t)(3 * W + 2 * P + 64) * es + (size_t)(P / 32) * 4 + 16 + 16 + 8 * 8;
    const size_t budget = 227 * 1024;
    int NB = budget > fixed ? (int)((budget - fixed) / panel) : 0;
    const int blocks = P / 32;
    int want = blocks < 3 ? 3 : (blocks < nb_cap ? blocks : nb_cap);
    if (NB > want) NB = want;
    s.NB = NB;
    s.panels = 0;
    s.alpha = panel * (size_t)NB;
    s.a = s.alpha + (size_t)W * es;
    s.U = s.a + (size_t)W * es;
    s.ball = s.U + (size_t)W * es;
    s.rall = s.ball + (size_t)P * es;
    s.xnext = s.rall + (size_t)P * es;
    s.mask = s.xnext + (size_t)64 * es;
    s.ctl = (s.mask + (size_t)(P / 32) * 4 + 15) / 16 * 16;          // progress word, then the mbarriers
    s.total = s.ctl + 16 + 8 * 8;
    return s;
}

// sum over the 32 rows of a panel of eta_t F[t, column], eta = +1 for a swapped pair (bit set in pm):
// the decided block's contribution to alpha of that column.  All loads are issued before the sums.
template <typename T> __device__ __forceinline__ T fold32(const T *__restrict__ col, const int ld, const uint32_t pm)
{
    T f[32];
#pragma unroll
    for (int t = 0; t < 32; ++t) f[t] = col[t * ld];
    T acc0 = 0, acc1 = 0;
#pragma unroll
    for (int t = 0; t < 32; t += 2) {
        acc0 += ((pm >> t) & 1u) ? f[t] : -f[t];
        acc1 += ((pm >> (t + 1)) & 1u) ? f[t + 1] : -f[t + 1];
    }
    return acc0 + acc1;
}

// Generic-precision block walker (fp64 mode): one vote per pair.  Fd[t] = F[t, lane] of the block's
// diagonal tile; a = this lane's threshold.
template <typename T>
__device__ __forceinline__ uint32_t walk_block_vote(const T (&Fd)[32], T alpha, T a, T U, const int lane)
{
    uint32_t swaps = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        const bool mine = (lane == t) && swap_decision(alpha, a, U);
        const uint32_t sw = (__ballot_sync(FULL, mine) >> t) & 1u;
        swaps |= sw << t;
        const T f = t < lane ? Fd[t] : (T)0;
        alpha += sw ? f : -f;
    }
    return swaps;
}

template <typename T>
__global__ void __launch_bounds__(96 + UPD_THREADS_MAX)
walk_chain_kernel(const __grid_constant__ CUtensorMap mapF, const T *__restrict__ F, int64_t F_stride,
                  const T *__restrict__ rdecay,
                  const int32_t *__restrict__ cur, int32_t *__restrict__ out, int64_t out_stride,
                  int64_t n, int P, int64_t lvl, uint64_t seed, T logfac, uint32_t pbase, int nb_cap, int *status)
{
    using namespace sm100;
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization
    constexpr bool EAGER = std::is_same<T, float>::value;            // the fp32 walker also scores the next block
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int C = (int)cluster_nctarank(), k = (int)cluster_ctarank();
    const ChainSmem S = chain_smem(P, C, (int)sizeof(T), nb_cap);
    const int NB = S.NB;
    const int W = P / C, nbw = W / 32;
    T *panels = reinterpret_cast<T *>(smem_raw + S.panels);          // [NB][32][W]
    T *alpha_s = reinterpret_cast<T *>(smem_raw + S.alpha);          // [W] scores of the own columns from folded panels
    T *a_s = reinterpret_cast<T *>(smem_raw + S.a);                  // [W] thresholds a_i
    T *U_s = reinterpret_cast<T *>(smem_raw + S.U);                  // [W] uniforms
    T *ball_s = reinterpret_cast<T *>(smem_raw + S.ball);            // [(k+1) W] b_i of every pair up to the own ones
    T *rall_s = reinterpret_cast<T *>(smem_raw + S.rall);            // [(k+1) W] shift decay factors
    T *xnext_s = reinterpret_cast<T *>(smem_raw + S.xnext);          // [2][32] next block's scores without the current block
    uint32_t *mask_s = reinterpret_cast<uint32_t *>(smem_raw + S.mask);   // [P/32] swap masks of the whole call
    uint32_t *progress = reinterpret_cast<uint32_t *>(smem_raw + S.ctl);  // blocks of the call decided so far
    uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw + S.ctl + 16); // [NB]
    const int g = blockIdx.x / C, p = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nthr = blockDim.x, NU = nthr - 96, u = threadIdx.x - 96;
    const T *Fg = F + (int64_t)p * F_stride + (int64_t)g * P * P;
    const int64_t base = (int64_t)g * P;
    const int col0 = k * W;
    const int first_own = k * nbw, R_end = first_own + nbw;

    if (threadIdx.x == 0) {
        *progress = 0;
        for (int i = 0; i < NB; ++i) mbar_init(full + i, 1);
        fence_barrier_init();
    }
    __syncthreads();
    // one tiled copy per panel: box {W columns, 32 rows} of the level's Gram seen as [problem][row][column]
    auto issue_panel = [&](int R, int buf) {                         // warp 1
        if (lane == 0) {
            mbar_expect_tx(full + buf, (uint32_t)(32 * W * sizeof(T)));
            tma_load_3d(panels + (size_t)buf * 32 * W, &mapF, full + buf, col0, g * P + 32 * R, p);
        }
    };
    // Block R is decided: lane q of the calling warp tells CTA q.  The mask stores precede (through
    // the warp barrier) every progress update, so a CTA that learns of block R from any CTA also
    // sees the masks the other lanes wrote for it.
    auto publish = [&](int R) {
        const bool tell = lane > k && lane < C;
        if (tell) st_cluster_u32(cluster_map(smem_u32(mask_s + R), (uint32_t)lane), mask_s[R]);
        __syncwarp();
        if (tell) red_max_release_cluster_u32(cluster_map(smem_u32(progress), (uint32_t)lane), (uint32_t)R + 1u);
    };
    // b_max recurrence of Algorithm A.1 over block Rb (one thread, in pair order); thresholds of own pairs
    T hb = 0;
    auto prefix_block = [&](int Rb) {
#pragma unroll 1
        for (int t0 = 0; t0 < 32; t0 += 8) {
            T bt[8], rt[8], av[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                bt[t] = ball_s[32 * Rb + t0 + t];
                rt[t] = rall_s[32 * Rb + t0 + t];
            }
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const T carried = hb * rt[t];
                hb = bt[t] > carried ? bt[t] : carried;
                av[t] = bt[t] * hb * logfac;
            }
            if (Rb >= first_own) {
#pragma unroll
                for (int t = 0; t < 8; ++t) a_s[32 * Rb + t0 + t - col0] = av[t];
            }
        }
    };
    if (warp == 1)
        for (int R = 0; R < NB - 2 && R < R_end; ++R) issue_panel(R, R);
    // b_i = sqrt(F[i,i]) and the decay factors of every pair up to the own ones (the diagonal is a
    // strided read: keep eight loads in flight per thread), uniforms of the own pairs
    for (int i0 = threadIdx.x; i0 < col0 + W; i0 += 8 * nthr) {
        T dv[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + q * nthr;
            dv[q] = i < col0 + W ? Fg[(int64_t)i * P + i] : (T)0;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + q * nthr;
            if (i < col0 + W) ball_s[i] = sqrt(dv[q] > 0 ? dv[q] : (T)0);
        }
    }
    for (int i = threadIdx.x; i < col0 + W; i += nthr) rall_s[i] = rdecay[(int64_t)p * (n / 2) + base + i];
    uint32_t cgroup, ccode;
    call_counter(g, lvl, cgroup, ccode);
    for (int i = threadIdx.x; i < W; i += nthr) {
        alpha_s[i] = 0;
        U_s[i] = halving_uniform<T>(seed, (uint32_t)(col0 + i), cgroup, ccode, (uint32_t)p + pbase);
    }
    __syncthreads();
    if (C > 1) cluster_sync_all();                                   // every CTA's control words are initialised
    if (threadIdx.x == 64) prefix_block(0);
    if (!mbar_wait(full + 0, 0)) atomicExch(status, 8);              // a copy that never lands also fails the next wait
    __syncthreads();

    bool aborted = false;
    int R = 0;
    int cbuf = 0, pbuf = NB - 1, ibuf = NB - 2;                      // buffers of panel R, R-1 and R+NB-2
    uint32_t cpar = 0;
    T dn = 0;                                                        // walker: this block's decisions folded into the next block's column
    for (; R < R_end; ++R) {
        int bad = 0;
        const T *pan = panels + (size_t)cbuf * 32 * W;
        const T *prev = panels + (size_t)pbuf * 32 * W;
        if (warp == 1) {
            if (R > first_own) publish(R - 1);
            if (R + NB - 2 < R_end) issue_panel(R + NB - 2, ibuf);   // into the buffer of panel R-2
        }
        if (warp == 1 && R == R_end - 1 && C > 1) {
            // every mask leaves through this warp, so that a later CTA's view of them is ordered by
            // this warp's own program order
            asm volatile("bar.sync 2, 64;" ::: "memory");
            publish(R);
        }
        if (R < first_own) {
            // rows of an earlier CTA's block: fold them into every own column once its mask is known
            // (one warp polls; the barrier hands its view of the mask to the others)
            if (warp == 1 && !wait_progress(progress, (uint32_t)R)) {
                atomicExch(status, 9);
                bad = 1;
            }
            __syncthreads();
            if (warp >= 3) {
                const uint32_t pm = mask_s[R];
                for (int j = u; j < W; j += NU) alpha_s[j] += fold32(pan + j, W, pm);
            } else if (threadIdx.x == 64 && R + 1 < R_end) {
                prefix_block(R + 1);
            }
        } else {
            const int lb = R - first_own;                            // own block number
            const bool has_next = lb + 1 < nbw;
            if (warp == 0) {
                const int c = 32 * lb + lane;
                uint32_t swaps;
                if constexpr (EAGER) {
                    float d;
                    if (lb == 0) {
                        const float a = a_s[c], U = U_s[c];
                        d = (a > 0.f && isfinite(a)) ? alpha_s[c] - a * (1.f - 2.f * U) : (U < 0.5f ? -1.f : 1.f);
                    } else {
                        d = xnext_s[(lb & 1) * 32 + lane] + dn;          // warp 2 prepared all but this block's part
                    }
                    dn = 0.f;
                    swaps = walk_block_warp(pan + 32 * lb, W, d, dn, lane);
                } else {
                    T alpha = alpha_s[c];
                    if (lb > 0) alpha += fold32(prev + c, W, mask_s[R - 1]);
                    T Fd[32];
#pragma unroll
                    for (int t = 0; t < 32; ++t) Fd[t] = pan[t * W + c];
                    swaps = walk_block_vote<T>(Fd, alpha, a_s[c], U_s[c], lane);
                }
                if (lane == 0) mask_s[R] = swaps;
                // last own block: warp 1 is waiting to hand the chain to the next CTA right away
                if (!has_next && C > 1) asm volatile("bar.arrive 2, 64;" ::: "memory");
            } else if (warp == 2) {
                if (lane == 0 && has_next) prefix_block(R + 1);
                __syncwarp();
                if (EAGER && has_next) {
                    // next block's scores from everything decided before the current block
                    const int c = 32 * (lb + 1) + lane;
                    const T acc = lb > 0 ? fold32(prev + c, W, mask_s[R - 1]) : (T)0;
                    // d of the sign test, short of the current block's decisions.  A pair with a = 0
                    // has F[., pair] = 0, so what the walker still adds leaves its +-1 untouched.
                    const float a = a_s[c], U = U_s[c];
                    xnext_s[((lb + 1) & 1) * 32 + lane] = (a > 0.f && isfinite(a))
                        ? (alpha_s[c] + acc) - a * (1.f - 2.f * U) : (U < 0.5f ? -1.f : 1.f);
                }
            } else if (warp >= 3 && lb > 0) {
                // the previous own block into the own columns after the ones the walker warps cover
                const uint32_t pm = mask_s[R - 1];
                for (int j = 32 * (lb + (EAGER ? 2 : 1)) + u; j < W; j += NU) alpha_s[j] += fold32(prev + j, W, pm);
            }
        }
        pbuf = cbuf;
        if (++cbuf == NB) { cbuf = 0; cpar ^= 1u; }
        if (++ibuf == NB) ibuf = 0;
        // Panel R+1 has to be there before the next iteration.  The walker warp does not look at the
        // mbarrier itself: the other warps observe the completed copy and the CTA barrier orders that
        // observation before the walker's reads.
        if (warp != 0 && R + 1 < R_end && !mbar_wait(full + cbuf, cpar)) {
            atomicExch(status, 8);
            bad = 1;
        }
        if (__syncthreads_or(bad)) {
            aborted = true;
            break;
        }
    }
    if (aborted) {
        // let the later CTAs run through instead of timing out one after the other, and wait
        // (bounded) for the copies still in flight into this CTA's shared memory
        if ((int)threadIdx.x > k && (int)threadIdx.x < C)
            red_max_release_cluster_u32(cluster_map(smem_u32(progress), threadIdx.x), 0xffffffffu);
        if (threadIdx.x == 32)
            for (int Rp = R + 1; Rp < R_end && Rp <= R + NB - 2; ++Rp) mbar_wait(full + Rp % NB, (uint32_t)(Rp / NB) & 1u);
    } else {
        // survivors: pair i keeps its second point when it was swapped
        for (int i = threadIdx.x; i < W; i += nthr) {
            const int gi = col0 + i;
            const uint32_t sw = (mask_s[gi >> 5] >> (gi & 31)) & 1u;
            out[(int64_t)p * out_stride + base + gi] = cur[(int64_t)p * n + 2 * (base + gi) + sw];
        }
    }
    if (C > 1) cluster_sync_all();                                   // nobody leaves while a peer may still write here
}

// CTAs per call: columns per CTA capped at 256 (32 KB fp32 panels), at most MAX_CLUSTER CTAs
int chain_cluster_size(int P)
{
    int C = P / 256;
    if (C < 1) C = 1;
    if (C > MAX_CLUSTER) C = MAX_CLUSTER;
    return C;
}

}  // namespace

template <typename T> bool walk_chain_covers(int P)
{
    if (P < 32 || P % 32 != 0) return false;
    const int C = chain_cluster_size(P);
    if (P % (32 * C) != 0 || P / C > 256) return false;               // a copy box is at most 256 elements wide
    return chain_smem(P, C, (int)sizeof(T), 3).NB >= 3;
}

template <typename T>
int walk_chain(const T *F, int64_t F_stride, const T *rdecay, const int32_t *cur, int32_t *out, int64_t out_stride,
               int64_t n, int P, int groups, int problems, int64_t level, uint64_t seed, T logfac, uint32_t pbase,
               int *status, cudaStream_t st)
{
    const int C = chain_cluster_size(P);
    const int nb_cap = 6;                                            // four panels ahead of the chain are enough
    const ChainSmem S = chain_smem(P, C, (int)sizeof(T), nb_cap);
    const int W = P / C;
    const int threads = 96 + (W > UPD_THREADS_MAX ? UPD_THREADS_MAX : W);
    CUtensorMap mapF;
    {
        sm100::EncodeTiledFn enc = sm100::tensor_map_encoder();
        if (!enc) return ELM_ERR_CUDA;
        cuuint64_t dims[3] = {(cuuint64_t)P, (cuuint64_t)groups * P, (cuuint64_t)problems};
        cuuint64_t strides[2] = {(cuuint64_t)P * sizeof(T), (cuuint64_t)F_stride * sizeof(T)};
        cuuint32_t box[3] = {(cuuint32_t)W, 32, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&mapF, sizeof(T) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 3,
                const_cast<T *>(F), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return ELM_ERR_CUDA;
    }
    auto kern = walk_chain_kernel<T>;
    ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S.total));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(groups * C), (unsigned)problems, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = S.total;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // (the grid may become resident while the Gram kernel in front of it drains; the kernel waits on the device)
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (C > 8) {
        // clusters of 16 CTAs need the opt-in and a GPC with 16 free SMs; if none can be resident
        // the caller falls back to one CTA per call
        ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        int resident = 0;
        if (cudaOccupancyMaxActiveClusters(&resident, kern, &cfg) != cudaSuccess || resident < 1) {
            cudaGetLastError();
            return 1;
        }
    }
    ELM_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, mapF, F, F_stride, rdecay, cur, out, out_stride, n, P, level, seed, logfac,
                                    pbase, nb_cap, status));
    return ELM_OK;
}

template bool walk_chain_covers<float>(int);
template bool walk_chain_covers<double>(int);
template int walk_chain<float>(const float *, int64_t, const float *, const int32_t *, int32_t *, int64_t, int64_t, int,
                               int, int, int64_t, uint64_t, float, uint32_t, int *, cudaStream_t);
template int walk_chain<double>(const double *, int64_t, const double *, const int32_t *, int32_t *, int64_t, int64_t,
                                int, int, int, int64_t, uint64_t, double, uint32_t, int *, cudaStream_t);

}  // namespace elm

