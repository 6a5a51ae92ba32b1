// The level machinery shared by the compression entry points (elm_compress, the Express paths, ragged
// Compress2, the streaming cache): one Halve level is
//   (1) level_prep : running shifts M_i of the Halve calls of that level,
//   (2) gram       : kernel evaluation of Eq. (katt) reduced to the pair Gram F = P G P^T,
//   (3) walk       : the self-balancing signed walk of Algorithm A.1 on F.
// Here: the precision-generic SIMT kernels (fp64 deterministic mode, fp32 inputs), the host-side level
// scheduler run_halve_level, and the small kernels that make and copy point lists.  The tensor-core Gram for
// bf16 inputs lives in elm_gram_tc.cu, the cluster walk in elm_walk_chain.cu.  Everything is a template or has
// internal linkage: each translation unit that includes this header carries its own copy.
#pragma once
#include <math.h>
#include <stdlib.h>

#include <type_traits>

#include "elm_attend.cuh"
#include "elm_common.cuh"
#include "elm_compress.cuh"
#include "elm_walk.cuh"

namespace elm {

// ---------------------------------------------------------------------------------------------
// Stage S0: per attention problem v_max (Eq. katt), c_t = ||k_t||^2 / sqrt(d), identity index list
// ---------------------------------------------------------------------------------------------
// 16-byte row chunks: 8 bf16 or 4 fp32 elements
template <typename T> __device__ __forceinline__ void chunk_sq_absmax(const __nv_bfloat16 *kp, const __nv_bfloat16 *vp, T &sq, float &vm)
{
    const uint4 kq = __ldg(reinterpret_cast<const uint4 *>(kp));
    const uint4 vq = __ldg(reinterpret_cast<const uint4 *>(vp));
    const uint32_t kw[4] = {kq.x, kq.y, kq.z, kq.w}, vw[4] = {vq.x, vq.y, vq.z, vq.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const T a = (T)__uint_as_float(kw[i] << 16), b = (T)__uint_as_float(kw[i] & 0xffff0000u);
        sq += a * a;
        sq += b * b;
        vm = fmaxf(vm, fmaxf(fabsf(__uint_as_float(vw[i] << 16)), fabsf(__uint_as_float(vw[i] & 0xffff0000u))));
    }
}
template <typename T> __device__ __forceinline__ void chunk_sq_absmax(const float *kp, const float *vp, T &sq, float &vm)
{
    const float4 kq = __ldg(reinterpret_cast<const float4 *>(kp));
    const float4 vq = __ldg(reinterpret_cast<const float4 *>(vp));
    sq += (T)kq.x * (T)kq.x;
    sq += (T)kq.y * (T)kq.y;
    sq += (T)kq.z * (T)kq.z;
    sq += (T)kq.w * (T)kq.w;
    vm = fmaxf(vm, fmaxf(fmaxf(fabsf(vq.x), fabsf(vq.y)), fmaxf(fabsf(vq.z), fabsf(vq.w))));
}

// One pass over K and V with 16-byte loads: a group of (row bytes / 16) lanes owns a row.
template <typename Tin, typename T>
static __global__ void __launch_bounds__(256) prepass_kernel(const Tin *__restrict__ K,
                                                      const Tin *__restrict__ V, int64_t n, int d,
                                                      T *__restrict__ cnorm,
                                                      unsigned *__restrict__ vmax_bits,
                                                      int32_t *__restrict__ cur, int64_t first = 0,
                                                      int64_t last = -1 /* rows [first, last); -1: n */)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    if (last < 0) last = n;
    constexpr int EPC = 16 / sizeof(Tin);                 // elements per 16-byte chunk
    const int p = blockIdx.y;
    const int lpr = d / EPC;                              // lanes per row: 8, 16 or 32
    const int rows_per_pass = 256 / lpr;
    const int sub = threadIdx.x % lpr, rloc = threadIdx.x / lpr;
    const int64_t row0 = first + (int64_t)blockIdx.x * 256;   // 256 rows per CTA
    const Tin *Kp = K + (int64_t)p * n * d;
    const Tin *Vp = V + (int64_t)p * n * d;
    const T rsd = sqrt((T)d);
    float vm = 0.f;
    for (int r = rloc; r < 256; r += rows_per_pass) {
        const int64_t t = row0 + r;
        T s = 0;
        if (t < last) chunk_sq_absmax<T>(Kp + t * d + sub * EPC, Vp + t * d + sub * EPC, s, vm);
        for (int o = lpr >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (sub == 0 && t < last) {
            cnorm[(int64_t)p * n + t] = s / rsd;
            cur[(int64_t)p * n + t] = (int32_t)t;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, o));
    if ((threadIdx.x & 31) == 0) atomicMax(vmax_bits + p, __float_as_uint(vm));   // non-negative floats order as uints
}

// ---------------------------------------------------------------------------------------------
// Stage level_prep: for every Halve call of the level, M_i = max over the call's first 2i points
// of c, and the factor exp(-(M_i - M_{i-1})/2) that carries b_max from one shift to the next.
// One CTA per call.
// ---------------------------------------------------------------------------------------------
template <typename T>
static __global__ void __launch_bounds__(1024) level_prep_kernel(const T *__restrict__ cnorm,
                                                         const int32_t *__restrict__ cur, int64_t n,
                                                         int P, T *__restrict__ Mpair,
                                                         T *__restrict__ rdecay)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    __shared__ T warp_tot[32];
    const int p = blockIdx.y, g = blockIdx.x;
    const int nthr = blockDim.x, nwarp = nthr >> 5;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T *cp = cnorm + (int64_t)p * n;
    const int32_t *curp = cur + (int64_t)p * n;
    const int64_t base = (int64_t)g * P;
    T carry = 0;            // c >= 0, so 0 is the identity of the running max
    for (int c0 = 0; c0 < P; c0 += nthr) {
        int i = c0 + threadIdx.x;
        T v = 0;
        if (i < P) {
            T a = cp[curp[2 * (base + i)]], b = cp[curp[2 * (base + i) + 1]];
            v = a > b ? a : b;
        }
        T inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            T u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc = inc > u ? inc : u;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        T before = carry;
        for (int w = 0; w < warp; ++w) before = before > warp_tot[w] ? before : warp_tot[w];
        T prev_lane = __shfl_up_sync(0xffffffffu, inc, 1);
        T excl = lane == 0 ? before : (before > prev_lane ? before : prev_lane);
        T M = inc > before ? inc : before;
        if (i < P) {
            Mpair[(int64_t)p * (n / 2) + base + i] = M;
            rdecay[(int64_t)p * (n / 2) + base + i] = (i == 0) ? (T)1 : (T)exp(-(double)(M - excl) * 0.5);
        }
        T tot = carry;
        for (int w = 0; w < nwarp; ++w) tot = tot > warp_tot[w] ? tot : warp_tot[w];
        __syncthreads();
        carry = tot;
    }
}

// ---------------------------------------------------------------------------------------------
// Stage gram (SIMT): one CTA computes a 32 x 32 tile of pair-Gram entries (64 x 64 points).
//   G[a,b] = E(<k_a,k_b>/sqrt(d) - M_pair(b)) * (<v_a,v_b> + v_max^2)          Eq. (katt), shifted
//   F[j,i] = G[2j,2i] - G[2j,2i+1] - G[2j+1,2i] + G[2j+1,2i+1] = <f_j, f_i>   Algorithm A.1's f_i
// Only j <= i is produced (the walk needs j < i and the diagonal b_i^2 = F[i,i]).
// Pairs are numbered along the problem's current sequence (J = g*P + j); when a call has fewer
// than 32 pairs a tile holds several whole calls and only same-call entries are written.
// ---------------------------------------------------------------------------------------------
template <typename Tin, typename T, int D>
static __global__ void __launch_bounds__(256) gram_simt_kernel(const Tin *__restrict__ K,
                                                        const Tin *__restrict__ V,
                                                        const int32_t *__restrict__ cur,
                                                        const T *__restrict__ Mpair,
                                                        const unsigned *__restrict__ vmax_bits,
                                                        int64_t n, int P, int64_t Ptotal,
                                                        T *__restrict__ F, int64_t F_stride)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    constexpr int DC = 16, LD = 68;
    __shared__ T Ak[DC][LD], Bk[DC][LD], Av[DC][LD], Bv[DC][LD];
    __shared__ int32_t rowsA[64], rowsB[64];
    const int p = blockIdx.y;
    const int tid = threadIdx.x;
    int64_t JR, JC;
    if (P >= 32) {
        const int Tg = P / 32, ntri = Tg * (Tg + 1) / 2;
        const int g = blockIdx.x / ntri, local = blockIdx.x % ntri;
        int tc = (int)((sqrtf(8.f * (float)local + 1.f) - 1.f) * 0.5f);
        while ((tc + 1) * (tc + 2) / 2 <= local) ++tc;
        while (tc * (tc + 1) / 2 > local) --tc;
        const int tr = local - tc * (tc + 1) / 2;
        JR = (int64_t)g * P + tr * 32;
        JC = (int64_t)g * P + tc * 32;
    } else {
        JR = JC = (int64_t)blockIdx.x * 32;
    }
    const int32_t *curp = cur + (int64_t)p * n;
    if (tid < 64) {
        int64_t pt = 2 * JR + tid;
        rowsA[tid] = pt < 2 * Ptotal ? curp[pt] : 0;
    } else if (tid < 128) {
        int64_t pt = 2 * JC + (tid - 64);
        rowsB[tid - 64] = pt < 2 * Ptotal ? curp[pt] : 0;
    }
    __syncthreads();
    const Tin *Kp = K + (int64_t)p * n * D;
    const Tin *Vp = V + (int64_t)p * n * D;
    const int ty = tid >> 4, tx = tid & 15;
    T kk[4][4], vv[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) { kk[r][c] = 0; vv[r][c] = 0; }

    for (int k0 = 0; k0 < D; k0 += DC) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            int e = tid + 256 * r;
            int pt = e / DC, q = e % DC;
            int64_t ra = (int64_t)rowsA[pt] * D + k0 + q, rb = (int64_t)rowsB[pt] * D + k0 + q;
            Ak[q][pt] = load_as<T>(Kp, ra);
            Av[q][pt] = load_as<T>(Vp, ra);
            Bk[q][pt] = load_as<T>(Kp, rb);
            Bv[q][pt] = load_as<T>(Vp, rb);
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < DC; ++q) {
            T a[4], b[4], av[4], bv[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                a[r] = Ak[q][4 * ty + r];
                av[r] = Av[q][4 * ty + r];
                b[r] = Bk[q][4 * tx + r];
                bv[r] = Bv[q][4 * tx + r];
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    kk[r][c] += a[r] * b[c];
                    vv[r][c] += av[r] * bv[c];
                }
        }
        __syncthreads();
    }

    const T vm = (T)__uint_as_float(vmax_bits[p]);
    const T vm2 = vm * vm;
    const T rsd = sqrt((T)D);
    T *Fp = F + (int64_t)p * F_stride;
#pragma unroll
    for (int cp = 0; cp < 2; ++cp) {
        const int64_t jc = JC + 2 * tx + cp;
        if (jc >= Ptotal) continue;
        const T M = Mpair[(int64_t)p * (n / 2) + jc];
        const int64_t gc = jc / P;
#pragma unroll
        for (int rp = 0; rp < 2; ++rp) {
            const int64_t jr = JR + 2 * ty + rp;
            if (jr > jc || jr / P != gc) continue;
            T g00 = floored_exp(kk[2 * rp][2 * cp] / rsd - M) * (vv[2 * rp][2 * cp] + vm2);
            T g01 = floored_exp(kk[2 * rp][2 * cp + 1] / rsd - M) * (vv[2 * rp][2 * cp + 1] + vm2);
            T g10 = floored_exp(kk[2 * rp + 1][2 * cp] / rsd - M) * (vv[2 * rp + 1][2 * cp] + vm2);
            T g11 = floored_exp(kk[2 * rp + 1][2 * cp + 1] / rsd - M) * (vv[2 * rp + 1][2 * cp + 1] + vm2);
            Fp[jr * P + (jc - gc * P)] = (g00 - g01) - (g10 - g11);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Stage walk: Algorithm A.1 on the pair Gram.  With eta_j = +1 when x_{2j-1} stayed in S^(1) and
// -1 when the pair was swapped, the balancing score is alpha_i = -sum_{j<i} eta_j F[j,i].
// A warp resolves 32 consecutive pairs: lane i holds column i of the 32 x 32 diagonal tile and its
// running alpha_i; each step publishes one decision with a ballot and every later lane folds it in.
// ---------------------------------------------------------------------------------------------
template <typename T> struct WalkState {
    T bmax;   // b_{max,i-1} in the shift of the last pair seen (warp-uniform)
};

// Resolve pairs [i0, i0 + cnt) (cnt <= 32) of one call.  `alpha` is this lane's score from all
// earlier blocks; Fg points at the call's P x P pair Gram; returns the 32-bit swap mask.
template <typename T>
__device__ __forceinline__ uint32_t walk_block(const T *__restrict__ Fg, int P, int i0, int cnt,
                                               T alpha, T r, T U, T logfac, T &bmax, int lane)
{
    T Fd[32];
    T b2 = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        T v = 0;
        if (t <= lane && lane < cnt) v = Fg[(int64_t)(i0 + t) * P + i0 + lane];
        Fd[t] = v;
        if (t == lane) b2 = v;
    }
    T b = sqrt(b2 > 0 ? b2 : (T)0);
    // b_{max,i} for every lane (independent of the decisions)
    T my_bmax = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        T bt = __shfl_sync(0xffffffffu, b, t);
        T rt = __shfl_sync(0xffffffffu, r, t);
        if (t < cnt) {
            T carried = bmax * rt;
            bmax = bt > carried ? bt : carried;
        }
        if (t == lane) my_bmax = bmax;
    }
    const T a = b * my_bmax * logfac;
    uint32_t swaps = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        bool mine = (lane == t) && (t < cnt) && swap_decision(alpha, a, U);
        uint32_t sw = (__ballot_sync(0xffffffffu, mine) >> t) & 1u;
        swaps |= sw << t;
        // alpha_i = -sum_j eta_j F[j,i]: a kept pair (eta = +1) subtracts, a swapped one adds
        alpha += sw ? Fd[t] : -Fd[t];
    }
    return swaps;
}

// 16-byte asynchronous copy global -> shared
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}

__device__ __forceinline__ void load4(const float *p, float (&f)[4])
{
    const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void load4(const double *p, double (&f)[4])
{
    const double2 a = __ldg(reinterpret_cast<const double2 *>(p));
    const double2 b = __ldg(reinterpret_cast<const double2 *>(p) + 1);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}

// Calls with at least 32 pairs: one CTA per call.
//   setup      all threads: b_i = sqrt(F[i,i]), the decay factors and the uniforms of every pair
//              into shared memory; scores alpha = 0.
//   warp 0     the walker: the 32 serial steps of block c on a tile copied to shared memory during the
//              previous block.  fp32: the warp-cooperative walker on rows of block c x columns of
//              blocks c and c+1, so block c+1's scores are complete when block c ends; fp64: one
//              vote per pair on the diagonal tile (c, c) after adding block c-1's contribution
//              from the cross tile (c-1, c).
//   warp 1     copies the tiles the walker needs for block c+1 (asynchronous copies).
//   warps 2..  the updaters fold block c-1 into the scores of all columns from block c+1 on, one
//              block behind the walker.  The rows of a block are streamed through two shared-memory
//              panels with asynchronous copies; F does not depend on the decisions, so the first
//              panel of the next round is already in flight when its swap mask becomes known.
// One __syncthreads per block separates the iterations.
template <typename T>
static __global__ void __launch_bounds__(576) walk_cta_kernel(const T *__restrict__ F, int64_t F_stride,
                                                       const T *__restrict__ rdecay,
                                                       const int32_t *__restrict__ cur,
                                                       int32_t *__restrict__ out, int64_t out_stride,
                                                       int64_t n, int P, int64_t lvl, uint64_t seed,
                                                       T logfac, uint32_t pbase)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    constexpr int PW = 2048 / sizeof(T);                             // panel width in columns (64 KB / 2 buffers... per 32 rows)
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *tiles = reinterpret_cast<T *>(smem_raw);                      // [2][2][32][32]: buffer, (diag, cross)
    T *alpha_s = tiles + 4 * 1024;                                   // [P] scores from finished rounds
    T *b_s = alpha_s + P;                                            // [P]
    T *r_s = b_s + P;                                                // [P]
    T *U_s = r_s + P;                                                // [P]
    T *a32_s = U_s + P;                                              // [32] the walker's scores of the block
    T *panels = a32_s + 32;                                          // [2][32][pw_alloc]
    const int pw_alloc = P - 64 < PW ? (P - 64 > 0 ? P - 64 : 32) : PW;
    uint32_t *mask_s = reinterpret_cast<uint32_t *>(panels + 2 * 32 * pw_alloc);   // [P/32] swap masks
    const int p = blockIdx.y, g = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nthr = blockDim.x;
    const T *Fg = F + (int64_t)p * F_stride + (int64_t)g * P * P;
    const int64_t base = (int64_t)g * P;
    const int nb = P / 32;
    constexpr int CH = 16 / sizeof(T);                               // elements per 16-byte chunk
    constexpr int CPR = 32 / CH;                                     // chunks per 32-element tile row

    // copies tile (rows r0.., cols c0..) of the call's pair Gram into `dst` [32][32]
    auto copy_tile = [&](T *dst, int r0, int c0) {
        for (int q = lane; q < 32 * CPR; q += 32) {
            const int t = q / CPR, k = q % CPR;
            cp_async16(dst + t * 32 + k * CH, Fg + (int64_t)(r0 + t) * P + c0 + k * CH);
        }
    };
    // fp32: rows of a block x the columns of that block and of the next one, [32][64]
    auto copy_tile64 = [&](T *dst, int r0) {
        const int ncols = P - r0 < 64 ? P - r0 : 64, cpr = ncols / CH;
        for (int q = lane; q < 32 * cpr; q += 32) {
            const int t = q / cpr, k = q % cpr;
            cp_async16(dst + t * 64 + k * CH, Fg + (int64_t)(r0 + t) * P + r0 + k * CH);
        }
    };
    constexpr bool WARP_WALK = std::is_same<T, float>::value;
    if (warp == (nthr > 32 ? 1 : 0)) {
        if constexpr (WARP_WALK) copy_tile64(tiles, 0);
        else copy_tile(tiles, 0, 0);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    uint32_t cgroup, ccode;
    call_counter(g, lvl, cgroup, ccode);
    for (int i = threadIdx.x; i < P; i += nthr) {
        alpha_s[i] = 0;
        const T d = Fg[(int64_t)i * P + i];
        b_s[i] = sqrt(d > 0 ? d : (T)0);
        r_s[i] = rdecay[(int64_t)p * (n / 2) + base + i];
        U_s[i] = halving_uniform<T>(seed, (uint32_t)i, cgroup, ccode, (uint32_t)p + pbase);
    }
    if (warp <= 1) asm volatile("cp.async.wait_group 0;" ::: "memory");

    // ---- updater streaming state ----
    const int NU = nthr - 64;                                        // updater threads (warps 2..)
    const int u = threadIdx.x - 64;
    // panel `pi` of round `r` (rows of block r): columns [32 (r + 2) + pi * PW, ...)
    auto panels_of = [&](int r) { const int cols = P - 32 * (r + 2); return cols > 0 ? (cols + PW - 1) / PW : 0; };
    auto issue_panel = [&](int r, int pi, int buf) {
        const int col0 = 32 * (r + 2) + pi * PW;
        const int pw = P - col0 < PW ? P - col0 : PW;
        const int cpr = pw / CH;
        const T *rows = Fg + (int64_t)(32 * r) * P + col0;
        T *dst = panels + (size_t)buf * 32 * pw_alloc;
        for (int q = u; q < 32 * cpr; q += NU) {
            const int t = q / cpr, k = q % cpr;
            cp_async16(dst + t * pw_alloc + k * CH, rows + (int64_t)t * P + k * CH);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int stream = 0;                                                  // panels consumed so far (buffer parity)
    if (warp >= 2 && panels_of(0) > 0) issue_panel(0, 0, 0);
    __syncthreads();

    T bmax = 0;
    float dn = 0.f;                                                  // fp32 walker: the next block's scores from the current block
    for (int c = 0; c < nb; ++c) {
        const int i0 = 32 * c;
        T *tdiag = tiles + (c & 1) * 2048, *tcross = tdiag + 1024;
        T *ndiag = tiles + ((c + 1) & 1) * 2048, *ncross = ndiag + 1024;
        if (warp == 0) {
            if constexpr (WARP_WALK) {
                // the previous block folded its decisions into this block's scores as it went (dn)
                const float a = walk_block_thresholds(b_s[i0 + lane], r_s[i0 + lane], bmax, logfac, lane);
                const float d = walk_sign_score(alpha_s[i0 + lane] + dn, a, U_s[i0 + lane]);
                dn = 0.f;
                const uint32_t swaps = walk_block_warp(tiles + (c & 1) * 2048, 64, d, dn, lane);
                if (lane == 0) mask_s[c] = swaps;
            } else {
                T alpha = alpha_s[i0 + lane];
                if (c > 0) {
                    const uint32_t pm = mask_s[c - 1];
#pragma unroll
                    for (int t = 0; t < 32; ++t) {
                        const T f = tcross[t * 32 + lane];
                        alpha += ((pm >> t) & 1u) ? f : -f;
                    }
                }
                T Fd[32];
#pragma unroll
                for (int t = 0; t < 32; ++t) Fd[t] = tdiag[t * 32 + lane];
                const uint32_t swaps = walk_block_regs<T>(Fd, b_s[i0 + lane], alpha, r_s[i0 + lane], U_s[i0 + lane],
                                                          logfac, bmax, lane);
                if (lane == 0) mask_s[c] = swaps;
            }
        } else if (warp == 1) {
            if (c + 1 < nb) {
                if constexpr (WARP_WALK) {
                    copy_tile64(tiles + ((c + 1) & 1) * 2048, i0 + 32);
                } else {
                    copy_tile(ndiag, i0 + 32, i0 + 32);
                    copy_tile(ncross, i0, i0 + 32);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
        } else if (c > 0) {
            // round r = c-1: rows of block r into every column from block r+2 on
            const int r = c - 1;
            const uint32_t pm = mask_s[r];
            const int np = panels_of(r);
            for (int pi = 0; pi < np; ++pi, ++stream) {
                const int buf = stream & 1;
                bool issued = true;
                if (pi + 1 < np) issue_panel(r, pi + 1, buf ^ 1);
                else if (panels_of(c) > 0) issue_panel(c, 0, buf ^ 1);       // first panel of the next round
                else issued = false;
                if (issued) asm volatile("cp.async.wait_group 1;" ::: "memory");
                else asm volatile("cp.async.wait_group 0;" ::: "memory");
                asm volatile("bar.sync 1, %0;" ::"r"(NU) : "memory");
                const int col0 = 32 * (r + 2) + pi * PW;
                const int pw = P - col0 < PW ? P - col0 : PW;
                const T *src = panels + (size_t)buf * 32 * pw_alloc;
                for (int j = u; j < pw; j += NU) {
                    T acc = 0;
#pragma unroll
                    for (int t = 0; t < 32; ++t) {
                        const T f = src[t * pw_alloc + j];
                        acc += ((pm >> t) & 1u) ? f : -f;
                    }
                    alpha_s[col0 + j] += acc;
                }
                asm volatile("bar.sync 1, %0;" ::"r"(NU) : "memory");
            }
        }
        __syncthreads();
    }
    // survivors: pair i keeps its second point when it was swapped (kept out of the walker's loop,
    // where a dependent global load would stall the one warp everything waits for)
    for (int i = threadIdx.x; i < P; i += nthr) {
        const uint32_t sw = (mask_s[i >> 5] >> (i & 31)) & 1u;
        out[(int64_t)p * out_stride + base + i] = cur[(int64_t)p * n + 2 * (base + i) + sw];
    }
}

// Smallest call (in pairs) that goes to the chain kernel of elm_walk_chain.cu.  From about a
// thousand pairs on, a call is worth a cluster of CTAs; below that one CTA per call (walk_cta_kernel)
// already fills the GPU with calls.  The environment variable exists for tests, which push small
// calls through the chain kernel.
static int walk_chain_min_pairs()
{
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("ELM_WALK_CHAIN_MIN_PAIRS");
        v = e ? atoi(e) : 1024;
        if (v < 32) v = 32;
    }
    return v;
}

// Calls with fewer than 32 pairs: one warp per call, 8 calls per CTA.
template <typename T>
static __global__ void __launch_bounds__(256) walk_warp_kernel(const T *__restrict__ F, int64_t F_stride,
                                                        const T *__restrict__ rdecay,
                                                        const int32_t *__restrict__ cur,
                                                        int32_t *__restrict__ out, int64_t out_stride,
                                                        int64_t n, int P, int groups, int64_t lvl,
                                                        uint64_t seed, T logfac, uint32_t pbase)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    const int p = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.x * 8 + warp;
    if (g >= groups) return;
    const T *Fg = F + (int64_t)p * F_stride + (int64_t)g * P * P;
    const int64_t base = (int64_t)g * P;
    T bmax = 0;
    const bool live = lane < P;
    const T r = live ? rdecay[(int64_t)p * (n / 2) + base + lane] : (T)1;
    uint32_t cgroup, ccode;
    call_counter(g, lvl, cgroup, ccode);
    const T U = halving_uniform<T>(seed, (uint32_t)lane, cgroup, ccode, (uint32_t)p + pbase);
    uint32_t swaps = walk_block<T>(Fg, P, 0, P, (T)0, r, U, logfac, bmax, lane);
    if (live) {
        const uint32_t sw = (swaps >> lane) & 1u;
        out[(int64_t)p * out_stride + base + lane] = cur[(int64_t)p * n + 2 * (base + lane) + sw];
    }
}

// ---------------------------------------------------------------------------------------------
// Stage emit: weights 1/n_out (Definition 1: positive, summing to 1); identity list when m = 0
// ---------------------------------------------------------------------------------------------
static __global__ void emit_kernel(float *__restrict__ w, int32_t *__restrict__ idx, int64_t total,
                            int64_t n_out, int write_identity)
{
    cudaGridDependencySynchronize();           // launched with programmatic stream serialization (launch_after)
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    w[i] = 1.0f / (float)n_out;
    if (write_identity) idx[i] = (int32_t)(i % n_out);
}

// ---------------------------------------------------------------------------------------------
// the level scheduler
// ---------------------------------------------------------------------------------------------
template <typename Tin, typename T>
static int run_gram_simt(const Tin *K, const Tin *V, const elm_params *p, const int32_t *cur,
                         const T *Mpair, const unsigned *vmax_bits, int P, int64_t Ptotal, int groups,
                         T *F, int64_t F_stride, cudaStream_t st)
{
    const int BH = p->batch * p->kv_heads;
    int64_t tiles;
    if (P >= 32) {
        const int Tg = P / 32;
        tiles = (int64_t)groups * (Tg * (Tg + 1) / 2);
    } else {
        tiles = (Ptotal + 31) / 32;
    }
    dim3 grid((unsigned)tiles, (unsigned)BH);
    if (p->d == 64)
        ELM_CUDA_TRY(launch_after(gram_simt_kernel<Tin, T, 64>, grid, dim3(256), 0, st, K, V, cur, Mpair, vmax_bits, p->n_kv, P, Ptotal, F, F_stride));
    else
        ELM_CUDA_TRY(launch_after(gram_simt_kernel<Tin, T, 128>, grid, dim3(256), 0, st, K, V, cur, Mpair, vmax_bits, p->n_kv, P, Ptotal, F, F_stride));
    count_launches(1);
    return cuda_status(cudaGetLastError());
}

// Everything one level needs besides its point lists.
template <typename Tin, typename T> struct LevelCtx {
    const Tin *K, *V;
    const elm_params *p;
    unsigned *vmax_bits;        // [BH] v_max bits (the workspace keeps the device status word behind them)
    int *status;                // that status word
    T *cnorm, *Mpair, *rdecay, *F;
    int64_t F_stride;
    uint64_t seed;
    uint32_t pbase;
    cudaStream_t st;
};

// One level: `groups` Halve calls KH(delta_call) of P pairs each per attention problem, on the point
// lists `cur` ([BH][n_kv]-strided, the level's 2 P groups points at the front); survivors go to
// `out` (stride out_stride) in call order.  `code` is the third word of the uniforms' counter; with
// calls_per_sibling > 0 the level holds the calls of several sibling segments (see call_counter).
template <typename Tin, typename T>
static int run_halve_level(const LevelCtx<Tin, T> &c, const int32_t *cur, int32_t *out, int64_t out_stride, int groups,
                           int P, int code, double delta_call, int calls_per_sibling = 0, int64_t first_call = 0)
{
    const int64_t lvl = pack_level(code, first_call, calls_per_sibling);
    const elm_params *p = c.p;
    const int BH = p->batch * p->kv_heads;
    const int64_t n = p->n_kv;
    const int64_t Ptotal = (int64_t)groups * P;
    const T logfac = (T)(0.5 + log(2.0 * (double)(2 * P) / delta_call));
    cudaStream_t st = c.st;
    int *status = c.status;
    {
        StageTimer t(ELM_STAGE_LEVEL_PREP, st, 1);
        const int lp_threads = P >= 1024 ? 1024 : (P <= 32 ? 32 : (P + 31) / 32 * 32);
        ELM_CUDA_TRY(launch_after(level_prep_kernel<T>, dim3((unsigned)groups, (unsigned)BH), dim3(lp_threads), 0, st, c.cnorm, cur, n, P, c.Mpair, c.rdecay));
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    bool walked = false;                                       // the Gram kernel walked the level itself
    {
        StageTimer t(ELM_STAGE_GRAM, st, 1);
        int rc;
        if constexpr (std::is_same<Tin, __nv_bfloat16>::value && std::is_same<T, float>::value) {
            // tensor cores once a Halve call fills at least a quarter of a 64-pair tile side; calls
            // that share a tile (< 64 pairs) are also walked inside the Gram kernel.  Calls of exactly 64
            // pairs - level 0 of the large workloads, one tile per call - go through the persistent
            // kernel and a walk launch of their own: 0.61 + 0.32 ms of Gram + walk per cfg5 step against
            // 0.70 + 0.27 with the walk inside the (one CTA per tile) Gram kernel
            if (P >= 16) {
                WalkArgs wk;
                wk.fused = P < 64;
                wk.level = lvl;
                wk.seed = c.seed;
                wk.logfac = logfac;
                wk.rdecay = c.rdecay;
                wk.out = out;
                wk.out_stride = out_stride;
                wk.pbase = c.pbase;
                walked = wk.fused;
                rc = gram_tc(c.K, c.V, p, cur, c.Mpair, c.vmax_bits, P, Ptotal, groups, c.F, c.F_stride, status, wk, st);
            } else {
                rc = run_gram_simt<Tin, T>(c.K, c.V, p, cur, c.Mpair, c.vmax_bits, P, Ptotal, groups, c.F, c.F_stride, st);
            }
        } else {
            rc = run_gram_simt<Tin, T>(c.K, c.V, p, cur, c.Mpair, c.vmax_bits, P, Ptotal, groups, c.F, c.F_stride, st);
        }
        if (rc != ELM_OK) return rc;
    }
    if (!walked) {
        StageTimer t(ELM_STAGE_WALK, st, 1);
        int chain_rc = 1;                                          // 1 = not taken
        if (P >= walk_chain_min_pairs() && walk_chain_covers<T>(P)) {
            chain_rc = walk_chain<T>(c.F, c.F_stride, c.rdecay, cur, out, out_stride, n, P, groups, (int)BH, lvl, c.seed,
                                     logfac, c.pbase, status, st);
            if (chain_rc < 0) return chain_rc;
        }
        if (chain_rc == ELM_OK) {
            // launched by walk_chain
        } else if (P >= 32) {
            // walker warp + tile-copy warp + updaters (one per two pairs, at most 512 threads)
            int upd = P / 2;
            upd = upd < 32 ? 32 : (upd > 512 ? 512 : upd);
            const int threads = P == 32 ? 32 : 64 + upd;
            constexpr int PW = 2048 / sizeof(T);
            const int pw_alloc = P - 64 < PW ? (P - 64 > 0 ? P - 64 : 32) : PW;
            const size_t smem = (size_t)(4 * 1024 + 4 * P + 32 + 2 * 32 * pw_alloc) * sizeof(T) + (size_t)(P / 32) * 4;
            if (smem > 227 * 1024) return ELM_ERR_SHAPE;               // a call this long needs the chain kernel
            auto kern = walk_cta_kernel<T>;
            ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            ELM_CUDA_TRY(launch_after(kern, dim3((unsigned)groups, (unsigned)BH), dim3(threads), smem, st,
                                      c.F, c.F_stride, c.rdecay, cur, out, out_stride, n, P, lvl, c.seed, logfac, c.pbase));
        } else {
            ELM_CUDA_TRY(launch_after(walk_warp_kernel<T>, dim3((unsigned)((groups + 7) / 8), (unsigned)BH), dim3(256), 0, st,
                                      c.F, c.F_stride, c.rdecay, cur, out, out_stride, n, P, groups, lvl, c.seed, logfac, c.pbase));
        }
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}

// n_kv = n_out 4^R ?  Returns R or -1.
static int express_rounds(const elm_params *p)
{
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    int64_t v = n_out;
    for (int R = 0; R <= 15; ++R, v *= 4)
        if (v == (int64_t)p->n_kv) return R;
    return -1;
}
static int validate_express(const elm_params *p, int32_t mbar)
{
    if (p->batch < 1 || p->kv_heads < 1) return ELM_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return ELM_ERR_SHAPE;
    if (p->log2_nout < 1 || p->log2_nout > 24 || mbar < 0 || mbar > 30) return ELM_ERR_SHAPE;
    if (p->n_kv < 1 || express_rounds(p) < 0) return ELM_ERR_SHAPE;
    if ((int64_t)p->batch * p->kv_heads > 65535) return ELM_ERR_SHAPE;
    if (p->dtype != ELM_F32 && p->dtype != ELM_BF16) return ELM_ERR_DTYPE;
    if (p->precision != ELM_PREC_FP64_DET && p->precision != ELM_PREC_FP32) return ELM_ERR_DTYPE;
    if (!(p->delta > 0.0 && p->delta < 1.0)) return ELM_ERR_DELTA;
    return ELM_OK;
}

// list[p][dst + i] = start + i
static __global__ void range_kernel(int32_t *__restrict__ list, int64_t stride, int64_t dst, int64_t start, int64_t count)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) list[(int64_t)blockIdx.y * stride + dst + i] = (int32_t)(start + i);
}
// dst[p][dst_off + i] = src[p][i]
static __global__ void copy_list_kernel(int32_t *__restrict__ dstl, int64_t dst_off, const int32_t *__restrict__ src, int64_t stride,
                                 int64_t count)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) dstl[(int64_t)blockIdx.y * stride + dst_off + i] = src[(int64_t)blockIdx.y * stride + i];
}
// Subsample (Algorithm 3) of three consecutive sibling segments of `seg` points, the first starting at
// `start`: stratum s of width 2^wlog of sibling j keeps point (segment start) + s 2^wlog + floor(U 2^wlog),
// U the 24-bit uniform of counter (s, 0, code + 64 j, problem); `per` strata per sibling.
static __global__ void subsample_kernel(int32_t *__restrict__ list, int64_t stride, int64_t start, int64_t seg, int wlog,
                                 int64_t per, uint64_t seed, uint32_t code, uint32_t pbase)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= 3 * per) return;
    const int64_t j = t / per, s = t % per;
    const double U = halving_uniform<double>(seed, (uint32_t)s, 0u, code + 64u * (uint32_t)j, (uint32_t)blockIdx.y + pbase);
    list[(int64_t)blockIdx.y * stride + t] =
        (int32_t)(start + j * seg + (s << wlog) + (int64_t)floor(U * (double)((int64_t)1 << wlog)));
}

static double kh_express_delta(double delta, int m)
{
    // Corollary 2: delta_m = (delta / 2) (1 / log2(m/2 + 2) - 1 / log2(m/2 + 3))
    return 0.5 * delta * (1.0 / log2(0.5 * m + 2.0) - 1.0 / log2(0.5 * m + 3.0));
}

// One epoch's cache list: up to 16 pieces laid end to end, each either a run of a point list
// (src != NULL: entries src[problem * src_stride + src_off ...]) or a run of consecutive tokens.
struct ListPieces {
    const int32_t *src[16];
    int64_t src_off[16];        // offset into the list, or the first token of a run
    int32_t dst_off[17];        // dst_off[k+1] - dst_off[k] entries
    float w[16];
    int n;
};
static __global__ void build_list_kernel(ListPieces pc, int64_t src_stride, int32_t *__restrict__ idx, float *__restrict__ w,
                                  int64_t cap)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= pc.dst_off[pc.n]) return;
    int k = 0;
    while (i >= pc.dst_off[k + 1]) ++k;
    const int64_t o = i - pc.dst_off[k];
    const int64_t pr = blockIdx.y;
    idx[pr * cap + i] = pc.src[k] ? pc.src[k][pr * src_stride + pc.src_off[k] + o] : (int32_t)(pc.src_off[k] + o);
    w[pr * cap + i] = pc.w[k];
}

}  // namespace elm
