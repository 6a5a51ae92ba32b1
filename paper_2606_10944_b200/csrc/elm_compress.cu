// Kernel-halving compression: Offline-Compress2 scheduled level by level, each level being
//   (1) level_prep : running shifts M_i of the Halve calls of that level,
//   (2) gram       : kernel evaluation of Eq. (katt) reduced to the pair Gram F = P G P^T,
//   (3) walk       : the self-balancing signed walk of Algorithm A.1 on F.
// This file holds the precision-generic SIMT kernels (fp64 deterministic mode, fp32 inputs) and
// the host-side level scheduler.  The tensor-core Gram for bf16 inputs lives in elm_gram_tc.cu.
#include <math.h>
#include <stdlib.h>

#include <type_traits>

#include "elm_attend.cuh"
#include "elm_common.cuh"
#include "elm_prefill_round.cuh"
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
__global__ void __launch_bounds__(256) prepass_kernel(const Tin *__restrict__ K,
                                                      const Tin *__restrict__ V, int64_t n, int d,
                                                      T *__restrict__ cnorm,
                                                      unsigned *__restrict__ vmax_bits,
                                                      int32_t *__restrict__ cur, int64_t first = 0,
                                                      int64_t last = -1 /* rows [first, last); -1: n */)
{
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
__global__ void __launch_bounds__(1024) level_prep_kernel(const T *__restrict__ cnorm,
                                                         const int32_t *__restrict__ cur, int64_t n,
                                                         int P, T *__restrict__ Mpair,
                                                         T *__restrict__ rdecay)
{
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
__global__ void __launch_bounds__(256) gram_simt_kernel(const Tin *__restrict__ K,
                                                        const Tin *__restrict__ V,
                                                        const int32_t *__restrict__ cur,
                                                        const T *__restrict__ Mpair,
                                                        const unsigned *__restrict__ vmax_bits,
                                                        int64_t n, int P, int64_t Ptotal,
                                                        T *__restrict__ F, int64_t F_stride)
{
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
__global__ void __launch_bounds__(576) walk_cta_kernel(const T *__restrict__ F, int64_t F_stride,
                                                       const T *__restrict__ rdecay,
                                                       const int32_t *__restrict__ cur,
                                                       int32_t *__restrict__ out, int64_t out_stride,
                                                       int64_t n, int P, int64_t lvl, uint64_t seed,
                                                       T logfac, uint32_t pbase)
{
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
__global__ void __launch_bounds__(256) walk_warp_kernel(const T *__restrict__ F, int64_t F_stride,
                                                        const T *__restrict__ rdecay,
                                                        const int32_t *__restrict__ cur,
                                                        int32_t *__restrict__ out, int64_t out_stride,
                                                        int64_t n, int P, int groups, int64_t lvl,
                                                        uint64_t seed, T logfac, uint32_t pbase)
{
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
__global__ void emit_kernel(float *__restrict__ w, int32_t *__restrict__ idx, int64_t total,
                            int64_t n_out, int write_identity)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    w[i] = 1.0f / (float)n_out;
    if (write_identity) idx[i] = (int32_t)(i % n_out);
}

// ---------------------------------------------------------------------------------------------
// workspace layout and the level scheduler
// ---------------------------------------------------------------------------------------------
CompressLayout compress_layout(const elm_params *p)
{
    CompressLayout L;
    const size_t ts = p->precision == ELM_PREC_FP64_DET ? 8 : 4;
    const size_t BH = (size_t)p->batch * p->kv_heads;
    const size_t n = (size_t)p->n_kv;
    const size_t n_out = (size_t)1 << p->log2_nout;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.vmax_bits = take((BH + 1) * 4);      // + one device status word
    L.cnorm = take(BH * n * ts);
    L.cur = take(BH * n * 4);
    L.nxt = take(BH * n * 4);
    L.Mpair = take(BH * (n / 2 + 1) * ts);
    L.rdecay = take(BH * (n / 2 + 1) * ts);
    L.F_stride = n_out * n_out;
    L.F = take(p->m > 0 ? BH * L.F_stride * ts : 0);
    L.wide = take(p->dtype == ELM_E4M3 ? 2 * BH * n * (size_t)p->d * 2 : 0);
    L.total = off;
    return L;
}

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
        gram_simt_kernel<Tin, T, 64><<<grid, 256, 0, st>>>(K, V, cur, Mpair, vmax_bits, p->n_kv, P, Ptotal, F, F_stride);
    else
        gram_simt_kernel<Tin, T, 128><<<grid, 256, 0, st>>>(K, V, cur, Mpair, vmax_bits, p->n_kv, P, Ptotal, F, F_stride);
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
        level_prep_kernel<T><<<dim3((unsigned)groups, (unsigned)BH), lp_threads, 0, st>>>(c.cnorm, cur, n, P, c.Mpair, c.rdecay);
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
            kern<<<dim3((unsigned)groups, (unsigned)BH), threads, smem, st>>>(
                c.F, c.F_stride, c.rdecay, cur, out, out_stride, n, P, lvl, c.seed, logfac, c.pbase);
        } else {
            walk_warp_kernel<T><<<dim3((unsigned)((groups + 7) / 8), (unsigned)BH), 256, 0, st>>>(
                c.F, c.F_stride, c.rdecay, cur, out, out_stride, n, P, groups, lvl, c.seed, logfac, c.pbase);
        }
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}

template <typename Tin, typename T>
static int compress_impl(const Tin *K, const Tin *V, const elm_params *p, uint64_t seed,
                         int32_t *idx_out, float *w_out, unsigned char *ws, cudaStream_t st, uint32_t pbase)
{
    const CompressLayout L = compress_layout(p);
    const int BH = p->batch * p->kv_heads;
    const int64_t n = p->n_kv;
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    const int m = p->m;
    LevelCtx<Tin, T> c;
    c.K = K; c.V = V; c.p = p;
    c.vmax_bits = reinterpret_cast<unsigned *>(ws + L.vmax_bits);
    c.status = reinterpret_cast<int *>(c.vmax_bits + BH);
    c.cnorm = reinterpret_cast<T *>(ws + L.cnorm);
    c.Mpair = reinterpret_cast<T *>(ws + L.Mpair);
    c.rdecay = reinterpret_cast<T *>(ws + L.rdecay);
    c.F = reinterpret_cast<T *>(ws + L.F);
    c.F_stride = (int64_t)L.F_stride;
    c.seed = seed; c.pbase = pbase; c.st = st;
    int32_t *cur = reinterpret_cast<int32_t *>(ws + L.cur);
    int32_t *nxt = reinterpret_cast<int32_t *>(ws + L.nxt);

    double dl[32];
    if (p->delta_level) {
        for (int i = 0; i < m; ++i) dl[i] = p->delta_level[i];
    } else {
        elm_default_delta_levels(m, p->delta, dl);
    }

    if (m > 0) {
        StageTimer t(ELM_STAGE_PREPASS, st, 1);
        ELM_CUDA_TRY(cudaMemsetAsync(c.vmax_bits, 0, (size_t)(BH + 1) * 4, st));
        dim3 grid((unsigned)((n + 255) / 256), (unsigned)BH);
        prepass_kernel<Tin, T><<<grid, 256, 0, st>>>(K, V, n, p->d, c.cnorm, c.vmax_bits, cur);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    for (int level = 0; level < m; ++level) {
        const int64_t len = n >> level;                            // points alive
        const int groups = 1 << (2 * (m - 1 - level));             // 4^(m-1-level) Halve calls
        const int P = (int)(len / groups / 2);
        const bool last = level == m - 1;
        const int rc = run_halve_level<Tin, T>(c, cur, last ? idx_out : nxt, last ? n_out : n, groups, P, level, dl[level]);
        if (rc != ELM_OK) return rc;
        int32_t *tmp = cur; cur = nxt; nxt = tmp;
    }
    {
        StageTimer t(ELM_STAGE_EMIT, st, 1);
        const int64_t total = (int64_t)BH * n_out;
        emit_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w_out, idx_out, total, n_out, m == 0);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}

// ---------------------------------------------------------------------------------------------
// Offline-Express: the cache a streaming Express run (Algorithm 1, with Subsample, Algorithm 3, and
// Compress2, Algorithm 2, inside, Halve = KH with the failure parameters of Corollary 2) holds after
// n = n_out 4^R points, computed by the equivalent recursion: E = first n_out points; round r
// (thinning factor m = 2r) thins the next three segments of n_out 2^m points each - one stratified
// draw per 2^(m - mbar) points when m > mbar, then Compress2 of depth min(m, mbar) - appends the three
// results to E and halves E twice.  Every Halve call runs through the same level machinery as
// elm_compress; the uniforms' counter words follow the call structure of the streaming run:
//   third word = level i + 64 (4 r + j)    Halve_i inside sibling j in {1, 2, 3} of round r,
//                62 / 63 + 64 (4 r)        the two halvings of E,
//                61 + 64 (4 r + j)         the stratified draws of sibling j (first word = stratum).
// v_max is taken over the whole sequence.
// ---------------------------------------------------------------------------------------------
constexpr int EXPRESS_LANES = 6;       // side streams of the prefill: two per sibling segment
struct ExpressLayout {
    size_t vmax_bits, cnorm, listA, listB, E, T1, Mpair, rdecay, F, F_stride, total;
    // prefill only: the output lists of every Compress2 level of a round; per side stream the cache list
    // of one launch with its weights and lifetimes and the workspace of elm_attend for that list; log2 of
    // the softmax denominators (rounds with Subsample: the tokens that were not kept are merged in afterwards)
    size_t levels, ep_idx, ep_w, ep_birth, ep_death, ep_blk, ws_attend, ep_cap, ep_pad, ep_stride, ws_attend_stride, lse;
    int n_levels;
    // prefill, rounds that take one attention launch: the round's universe and tile table (elm_prefill_round.cuh)
    size_t round;
    RoundBufferLayout rbl;
};
// Tokens per attention launch of the prefill: windows of about 512 tokens (whole strata, at most a segment).
static int64_t prefill_window(const RoundGeom &g)
{
    static const int64_t target = []() {
        const char *e = getenv("ELM_PREFILL_WINDOW");           // tuning aid: a power of two
        const long v = e ? atol(e) : 0;
        return (int64_t)(v >= 64 && (v & (v - 1)) == 0 ? v : 512);
    }();
    int64_t W = (int64_t)1 << g.wlog;
    if (W < target) W = target;
    return W < g.seg ? W : g.seg;
}

// The cache entries some token of a window can see, as runs of the round's point lists, each entry with
// the span of tokens that see it.  In terms of G = the number of kept points of the sibling segment
// that have arrived (a window covers G in [G0, G1)):
//   kind 0   E and the finished siblings: always
//   kind 1   S_i, 1 <= i < q: the output of call c of level i - 1 (u entries) exists from G = (c + 1) A,
//            A = s0 4^(i-1), until the level-i call that consumes it completes at G = (c / 4 + 1) 4 A
//   kind 2   S_0: kept point g exists from its own token (which sees itself) until G = (g / s0 + 1) s0
//   kind 3   S_q: the output of the segment's last call, from G = len0 on
// G = X is reached right after the X-th kept point: at token kept[X - 1] + 1.
struct WindowPieces {
    const int32_t *src[16];
    int64_t src_off[16];
    int64_t first[16];          // kind 1: index of the run's first entry within the sibling's part of the list; kind 2: its g
    int64_t per_call[16];       // kind 1: A
    int32_t dst_off[17];
    int32_t unit[16];           // kind 1: u; kind 2: s0
    float w[16];
    int8_t kind[16];
    int n;
    const int32_t *kept;        // kept points of the round's three siblings (the level-0 input list)
    int64_t kept_off, len0;
    int32_t q;
};
static int32_t window_pieces(const RoundGeom &g, int64_t n_out, int jj, int64_t G0, int64_t G1, const int32_t *E,
                             const int32_t *levels, size_t level_stride, const int32_t *kept, WindowPieces &pc)
{
    int k = 0;
    int32_t at = 0;
    auto piece = [&](const int32_t *src, int64_t off, int64_t count, double wgt, int kind, int64_t first, int64_t unit,
                     int64_t per_call) {
        if (count <= 0) return;
        pc.src[k] = src; pc.src_off[k] = off; pc.w[k] = (float)wgt; pc.dst_off[k] = at;
        pc.kind[k] = (int8_t)kind; pc.first[k] = first; pc.unit[k] = (int32_t)unit; pc.per_call[k] = per_call;
        at += (int32_t)count;
        ++k;
    };
    const int q = g.q;
    piece(E, 0, (1 + jj) * n_out, 1.0, 0, 0, 1, 1);
    for (int i = q - 1; i >= 1; --i) {
        const int64_t A = g.s0 << (2 * (i - 1)), u = (g.s0 << (i - 1)) >> 1;
        const int64_t c_lo = 4 * (G0 / (4 * A)), c_end = G1 / A;
        piece(levels ? levels + (size_t)(i - 1) * level_stride : nullptr, jj * (g.len0 >> i) + c_lo * u, (c_end - c_lo) * u,
              ldexp(1.0, i - q), 1, c_lo * u, u, A);
    }
    if (q >= 1 && g.sub && G1 >= g.len0) piece(E, (1 + jj) * n_out, n_out, 1.0, 3, 0, 1, 1);
    const int64_t g_lo = q >= 1 ? (G0 / g.s0) * g.s0 : 0;
    piece(kept, jj * g.len0 + g_lo, G1 - g_lo, ldexp(1.0, -q), 2, g_lo, g.s0, 1);
    pc.dst_off[k] = at;
    pc.n = k;
    pc.kept = kept;
    pc.kept_off = jj * g.len0;
    pc.len0 = g.len0;
    pc.q = q;
    return at;
}
// Longest cache list any launch of the prefill attends over.
static size_t express_list_cap(const elm_params *p, int mbar)
{
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    size_t cap = (size_t)(4 * n_out);                         // the exact start: causal attention over 4 n_out tokens
    const int R = [&]() { int64_t v = n_out; int r = 0; while (v < (int64_t)p->n_kv) { v *= 4; ++r; } return r; }();
    for (int r = 1; r < R; ++r) {
        const RoundGeom g = round_geom(p, mbar, r);
        const int64_t Wg = prefill_window(g) >> g.wlog;
        for (int jj = 0; jj < 3; ++jj)
            for (int64_t G0 = 0; G0 < g.len0; G0 += Wg) {
                WindowPieces pc;
                const size_t len = (size_t)window_pieces(g, n_out, jj, G0, G0 + Wg, nullptr, nullptr, 0, nullptr, pc);
                if (len > cap) cap = len;
            }
    }
    return cap;
}
static ExpressLayout express_layout(const elm_params *p, int mbar = 0, bool prefill = false)
{
    ExpressLayout L;
    const size_t ts = p->precision == ELM_PREC_FP64_DET ? 8 : 4;
    const size_t BH = (size_t)p->batch * p->kv_heads;
    const size_t n = (size_t)p->n_kv;
    const size_t n_out = (size_t)1 << p->log2_nout;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.vmax_bits = take((BH + 1) * 4);      // + one device status word
    L.cnorm = take(BH * n * ts);
    L.listA = take(BH * n * 4);
    L.listB = take(BH * n * 4);
    L.E = take(BH * n * 4);                // every point list is [BH][n]-strided, like the lists of elm_compress
    L.T1 = take(BH * n * 4);
    L.Mpair = take(BH * (n / 2 + 1) * ts);
    L.rdecay = take(BH * (n / 2 + 1) * ts);
    L.F_stride = 4 * n_out * n_out;        // the first halving of E is one call of 2 n_out pairs
    L.F = take(BH * L.F_stride * ts);
    L.levels = L.ep_idx = L.ep_w = L.ep_birth = L.ep_death = L.ep_blk = L.ws_attend = L.ep_cap = L.ep_pad = L.ep_stride = 0;
    L.ws_attend_stride = L.lse = 0;
    L.n_levels = 0;
    L.round = 0;
    L.rbl = RoundBufferLayout();
    if (prefill) {
        L.n_levels = mbar < 30 ? mbar : 30;
        L.levels = take((size_t)L.n_levels * BH * n * 4);
        L.ep_cap = express_list_cap(p, mbar);
        L.ep_pad = (L.ep_cap + 127) / 128 * 128;
        // one set per side stream: the launches of a round are spread over EXPRESS_LANES streams
        L.ep_stride = align_up(BH * L.ep_pad * 4, 256);
        L.ep_idx = take(EXPRESS_LANES * L.ep_stride);
        L.ep_w = take(EXPRESS_LANES * L.ep_stride);
        L.ep_birth = take(EXPRESS_LANES * L.ep_stride);
        L.ep_death = take(EXPRESS_LANES * L.ep_stride);
        L.ep_blk = take(EXPRESS_LANES * L.ep_stride);          // two arrays of [BH][ep_pad / 128]
        L.lse = take((size_t)p->batch * p->q_heads * n * 4);
        L.ws_attend_stride = align_up(attend_layout(p, (int32_t)L.ep_cap).total, 256);
        L.ws_attend = take(EXPRESS_LANES * L.ws_attend_stride);
        int R = 0;
        for (size_t v = n_out; v < n; v *= 4) ++R;
        L.rbl = round_buffer_layout(p, mbar, R);
        L.round = take(L.rbl.total);
    }
    L.total = off;
    return L;
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
__global__ void range_kernel(int32_t *__restrict__ list, int64_t stride, int64_t dst, int64_t start, int64_t count)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) list[(int64_t)blockIdx.y * stride + dst + i] = (int32_t)(start + i);
}
// dst[p][dst_off + i] = src[p][i]
__global__ void copy_list_kernel(int32_t *__restrict__ dstl, int64_t dst_off, const int32_t *__restrict__ src, int64_t stride,
                                 int64_t count)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) dstl[(int64_t)blockIdx.y * stride + dst_off + i] = src[(int64_t)blockIdx.y * stride + i];
}
// Subsample (Algorithm 3) of three consecutive sibling segments of `seg` points, the first starting at
// `start`: stratum s of width 2^wlog of sibling j keeps point (segment start) + s 2^wlog + floor(U 2^wlog),
// U the 24-bit uniform of counter (s, 0, code + 64 j, problem); `per` strata per sibling.
__global__ void subsample_kernel(int32_t *__restrict__ list, int64_t stride, int64_t start, int64_t seg, int wlog,
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
__global__ void build_list_kernel(ListPieces pc, int64_t src_stride, int32_t *__restrict__ idx, float *__restrict__ w,
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

// The list of one prefill window (see WindowPieces): indices, weights, and for every entry the first
// token that sees it (birth) and the first that does not any more (death); per block of 128 entries the
// largest birth and the smallest death.  Entries beyond the list (up to n_pad) are given the lifetime
// "always": the attention kernel hides them by other means.
__global__ void __launch_bounds__(256) build_window_kernel(WindowPieces pc, int64_t src_stride, int32_t *__restrict__ idx,
                                                           float *__restrict__ w, int n_core, int n_pad,
                                                           int32_t *__restrict__ birth, int32_t *__restrict__ death,
                                                           int32_t *__restrict__ blk_birth, int32_t *__restrict__ blk_death)
{
    __shared__ int32_t sb[8], sd[8];
    const int i = blockIdx.x * 256 + threadIdx.x;
    const int64_t pr = blockIdx.y;
    int32_t bt = 0, dt = 0x7fffffff;
    if (i < n_core) {
        int k = 0;
        while (i >= pc.dst_off[k + 1]) ++k;
        const int64_t o = i - pc.dst_off[k];
        const int32_t *kept = pc.kept + pr * src_stride + pc.kept_off;
        auto token_after = [&](int64_t X) { return X > pc.len0 ? 0x7fffffff : kept[X - 1] + 1; };   // G = X is reached
        idx[pr * n_core + i] = pc.src[k][pr * src_stride + pc.src_off[k] + o];
        w[pr * n_core + i] = pc.w[k];
        if (pc.kind[k] == 1) {
            const int64_t c = (pc.first[k] + o) / pc.unit[k];
            bt = token_after((c + 1) * pc.per_call[k]);
            dt = token_after((c / 4 + 1) * 4 * pc.per_call[k]);
        } else if (pc.kind[k] == 2) {
            const int64_t g = pc.first[k] + o;
            bt = kept[g];
            if (pc.q >= 1) dt = token_after((g / pc.unit[k] + 1) * pc.unit[k]);
        } else if (pc.kind[k] == 3) {
            bt = token_after(pc.len0);
        }
    }
    if (i < n_pad) {
        birth[pr * n_pad + i] = bt;
        death[pr * n_pad + i] = dt;
    }
    int32_t bm = bt, dm = dt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        bm = max(bm, __shfl_xor_sync(0xffffffffu, bm, o));
        dm = min(dm, __shfl_xor_sync(0xffffffffu, dm, o));
    }
    if ((threadIdx.x & 31) == 0) { sb[threadIdx.x >> 5] = bm; sd[threadIdx.x >> 5] = dm; }
    __syncthreads();
    if (threadIdx.x < 2) {
        const int blk = blockIdx.x * 2 + threadIdx.x, h = threadIdx.x * 4;
        if (blk < n_pad / 128) {
            blk_birth[pr * (n_pad / 128) + blk] = max(max(sb[h], sb[h + 1]), max(sb[h + 2], sb[h + 3]));
            blk_death[pr * (n_pad / 128) + blk] = min(min(sd[h], sd[h + 1]), min(sd[h + 2], sd[h + 3]));
        }
    }
}

// Rounds with Subsample: a token that was not kept is in no list, but Algorithm 5 still lets it attend to
// itself with the weight of a point of S_0.  One warp per (head, token): merges that single term into the
// output row, given log2 of the row's denominator over the cache.
template <typename Tin, typename T>
__global__ void __launch_bounds__(256) self_merge_kernel(const Tin *__restrict__ Q, const Tin *__restrict__ K,
                                                         const Tin *__restrict__ V, Tin *__restrict__ O,
                                                         const float *__restrict__ lse, const int32_t *__restrict__ kept,
                                                         int q_heads, int kv_heads, int64_t n, int d, int64_t seg,
                                                         int64_t len0, int wlog, T log2w)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t rel = (int64_t)blockIdx.x * 8 + warp;                   // token within the round's 3 segments
    if (rel >= 3 * seg) return;
    const int bh = blockIdx.y;
    const int64_t prob = (int64_t)(bh / q_heads) * kv_heads + ((int64_t)(bh % q_heads) * kv_heads) / q_heads;
    const int64_t t = seg + rel, jj = rel / seg, stratum = (rel % seg) >> wlog;
    if (kept[prob * n + jj * len0 + stratum] == (int32_t)t) return;        // a kept token is an entry of S_0
    const Tin *q = Q + ((int64_t)bh * n + t) * d, *k = K + (prob * n + t) * d, *v = V + (prob * n + t) * d;
    Tin *o = O + ((int64_t)bh * n + t) * d;
    T dot = 0;
    for (int e = lane; e < d; e += 32) dot += load_as<T>(q, e) * load_as<T>(k, e);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
    const T sc = dot * (T)(1.4426950408889634 / sqrt((double)d)) + log2w;
    const T L = (T)lse[(int64_t)bh * n + t];
    const T M = sc > L ? sc : L;
    const T a = (T)exp2((T)(L - M)), b = (T)exp2((T)(sc - M));
    const T inv = (T)1 / (a + b);
    for (int e = lane; e < d; e += 32) store_from(o, e, (a * load_as<T>(o, e) + b * load_as<T>(v, e)) * inv);
}

// Launch-side state of one side stream of the prefill.
struct PrefillLane {
    int32_t *idx, *birth, *death, *blk_birth, *blk_death;
    float *w;
    unsigned char *ws_attend;
};
static PrefillLane prefill_lane(const ExpressLayout &L, unsigned char *ws, int BH, int lane)
{
    PrefillLane pl;
    pl.idx = reinterpret_cast<int32_t *>(ws + L.ep_idx + lane * L.ep_stride);
    pl.w = reinterpret_cast<float *>(ws + L.ep_w + lane * L.ep_stride);
    pl.birth = reinterpret_cast<int32_t *>(ws + L.ep_birth + lane * L.ep_stride);
    pl.death = reinterpret_cast<int32_t *>(ws + L.ep_death + lane * L.ep_stride);
    pl.blk_birth = reinterpret_cast<int32_t *>(ws + L.ep_blk + lane * L.ep_stride);
    pl.blk_death = pl.blk_birth + (size_t)BH * (L.ep_pad / 128);
    pl.ws_attend = ws + L.ws_attend + lane * L.ws_attend_stride;
    return pl;
}

static RoundBuffers round_buffers(const ExpressLayout &L, unsigned char *ws, int BH, int64_t n_univ)
{
    unsigned char *rw = ws + L.round;
    RoundBuffers rb;
    rb.idx = reinterpret_cast<int32_t *>(rw + L.rbl.idx);
    rb.w = reinterpret_cast<float *>(rw + L.rbl.w);
    rb.birth = reinterpret_cast<int32_t *>(rw + L.rbl.birth);
    rb.death = reinterpret_cast<int32_t *>(rw + L.rbl.death);
    rb.blk_birth = reinterpret_cast<int32_t *>(rw + L.rbl.blk);
    rb.blk_death = rb.blk_birth + (size_t)BH * (n_univ / 128);
    rb.tile_cnt = reinterpret_cast<int32_t *>(rw + L.rbl.tile_cnt);
    rb.tile_blk = reinterpret_cast<int32_t *>(rw + L.rbl.tile_blk);
    rb.item_tab = reinterpret_cast<int32_t *>(rw + L.rbl.item_tab);
    rb.item_cnt = reinterpret_cast<int32_t *>(rw + L.rbl.item_cnt);
    rb.item_cap = L.rbl.item_cap;
    rb.item_ctas = L.rbl.item_ctas;
    rb.ws_attend = rw + L.rbl.ws_attend;
    return rb;
}

// The exact start of Thinformer Express (Algorithm 5) in prefill: token t < rows attends over the tokens 0 .. t.
static int express_attend_start(const void *Q, const void *K, const void *V, void *O, const elm_params *p, const ExpressLayout &L,
                                unsigned char *ws, int rows, cudaStream_t st)
{
    const int BH = p->batch * p->kv_heads;
    const PrefillLane pl = prefill_lane(L, ws, BH, 0);
    if ((size_t)rows > L.ep_cap) return ELM_ERR_WORKSPACE;
    ListPieces pc = {};
    pc.n = 1;
    pc.src[0] = nullptr; pc.src_off[0] = 0; pc.w[0] = 1.f;
    pc.dst_off[0] = 0; pc.dst_off[1] = rows;
    build_list_kernel<<<dim3((unsigned)((rows + 255) / 256), (unsigned)BH), 256, 0, st>>>(pc, p->n_kv, pl.idx, pl.w, rows);
    count_launches(1);
    ELM_CUDA_TRY(cudaGetLastError());
    elm_params pe = *p;
    pe.n_q = rows;
    AttendWindow win;
    win.q_row0 = 0;
    win.n_q_total = p->n_kv;
    win.tail_start = 0;                  // the whole list is the causal tail
    if (L.rbl.total) {
        // (the run has the tile table of the one-launch rounds: pairs of query tiles stop at their own last token)
        const int rc = causal_tile_table(rows, p->batch * p->q_heads, round_buffers(L, ws, BH, 0), win, st);
        if (rc != ELM_OK) return rc;
    }
    return attend_enqueue(Q, K, V, pl.idx, pl.w, rows, &pe, O, pl.ws_attend, st, win);
}

// Attention of the tokens [t0, t0 + rows) over the entries of `pc`, each seen by the tokens of its lifetime.
static int express_attend_window(const void *Q, const void *K, const void *V, void *O, const elm_params *p,
                                 const ExpressLayout &L, unsigned char *ws, const WindowPieces &pc, int64_t t0, int rows,
                                 float *lse, cudaStream_t st, int lane)
{
    const int BH = p->batch * p->kv_heads;
    const int total = pc.dst_off[pc.n];
    const int n_pad = (total + 127) / 128 * 128;
    if ((size_t)total > L.ep_cap) return ELM_ERR_WORKSPACE;
    const PrefillLane pl = prefill_lane(L, ws, BH, lane);
    int32_t *blk_death = pl.blk_birth + (size_t)BH * (n_pad / 128);
    build_window_kernel<<<dim3((unsigned)((n_pad + 255) / 256), (unsigned)BH), 256, 0, st>>>(
        pc, p->n_kv, pl.idx, pl.w, total, n_pad, pl.birth, pl.death, pl.blk_birth, blk_death);
    count_launches(1);
    ELM_CUDA_TRY(cudaGetLastError());
    elm_params pe = *p;
    pe.n_q = rows;
    AttendWindow win;
    win.q_row0 = t0;
    win.n_q_total = p->n_kv;
    win.birth = pl.birth;
    win.death = pl.death;
    win.blk_birth = pl.blk_birth;
    win.blk_death = blk_death;
    win.lse = lse;
    return attend_enqueue(Q, K, V, pl.idx, pl.w, total, &pe, O, pl.ws_attend, st, win);
}

template <typename Tin, typename T>
static int express_impl(const Tin *K, const Tin *V, const elm_params *p, int mbar, uint64_t seed, int32_t *idx_out,
                        float *w_out, unsigned char *ws, cudaStream_t st, uint32_t pbase, const Tin *Q = nullptr,
                        Tin *O = nullptr)
{
    const bool prefill = Q != nullptr;
    const ExpressLayout L = express_layout(p, mbar, prefill);
    const int BH = p->batch * p->kv_heads;
    const int64_t n = p->n_kv;
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    const int R = express_rounds(p);
    LevelCtx<Tin, T> c;
    c.K = K; c.V = V; c.p = p;
    c.vmax_bits = reinterpret_cast<unsigned *>(ws + L.vmax_bits);
    c.status = reinterpret_cast<int *>(c.vmax_bits + BH);
    c.cnorm = reinterpret_cast<T *>(ws + L.cnorm);
    c.Mpair = reinterpret_cast<T *>(ws + L.Mpair);
    c.rdecay = reinterpret_cast<T *>(ws + L.rdecay);
    c.F = reinterpret_cast<T *>(ws + L.F);
    c.F_stride = (int64_t)L.F_stride;
    c.seed = seed; c.pbase = pbase; c.st = st;
    int32_t *listA = reinterpret_cast<int32_t *>(ws + L.listA);
    int32_t *listB = reinterpret_cast<int32_t *>(ws + L.listB);
    int32_t *E = reinterpret_cast<int32_t *>(ws + L.E);
    int32_t *T1 = reinterpret_cast<int32_t *>(ws + L.T1);
    auto blocks = [](int64_t count) { return (unsigned)((count + 255) / 256); };
    {
        StageTimer t(ELM_STAGE_PREPASS, st, 2);
        ELM_CUDA_TRY(cudaMemsetAsync(c.vmax_bits, 0, (size_t)(BH + 1) * 4, st));
        prepass_kernel<Tin, T><<<dim3(blocks(n), (unsigned)BH), 256, 0, st>>>(K, V, n, p->d, c.cnorm, c.vmax_bits, listA);
        range_kernel<<<dim3(blocks(n_out), (unsigned)BH), 256, 0, st>>>(E, n, 0, 0, n_out);      // exact phase
        count_launches(2);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    int32_t *levels = reinterpret_cast<int32_t *>(ws + L.levels);
    struct SideStreams {                                             // released on every return path
        cudaStream_t s[EXPRESS_LANES] = {};
        cudaEvent_t fork = nullptr, join[EXPRESS_LANES] = {};
        ~SideStreams()
        {
            for (int i = 0; i < EXPRESS_LANES; ++i) {
                if (s[i]) cudaStreamDestroy(s[i]);                   // work already enqueued still completes
                if (join[i]) cudaEventDestroy(join[i]);
            }
            if (fork) cudaEventDestroy(fork);
        }
    } sides;
    cudaStream_t *side = sides.s;
    cudaEvent_t &fork = sides.fork;
    cudaEvent_t *join = sides.join;
    if (prefill && R >= 2) {
        ELM_CUDA_TRY(cudaEventCreateWithFlags(&fork, cudaEventDisableTiming));
        for (int i = 0; i < EXPRESS_LANES; ++i) {
            ELM_CUDA_TRY(cudaStreamCreateWithFlags(&side[i], cudaStreamNonBlocking));
            ELM_CUDA_TRY(cudaEventCreateWithFlags(&join[i], cudaEventDisableTiming));
        }
    }
    if (prefill) {
        // Exact phase and round 0 (thinning factor 1: nothing is dropped): each of the first 4 n_out
        // tokens attends over all tokens up to itself (Theorem 3's exact regime).
        const int rc = express_attend_start(Q, K, V, O, p, L, ws, (int)(n < 4 * n_out ? n : 4 * n_out), st);
        if (rc != ELM_OK) return rc;
    }
    for (int r = 0; r < R; ++r) {
        const int m = 2 * r, q = m < mbar ? m : mbar;
        const int64_t seg = n_out << m, len0 = n_out << q;
        const double dm = kh_express_delta(p->delta, m);
        // The three sibling segments of the round are thinned together: their point lists are laid
        // side by side, every level holds the calls of all three (call_counter keeps their uniforms
        // apart), and the last level leaves their 3 n_out survivors behind the n_out points of E.
        const int code1 = 64 * (4 * r + 1);                                   // sibling 1; siblings 2, 3 are 64 apart
        if (m > mbar)
            subsample_kernel<<<dim3(blocks(3 * len0), (unsigned)BH), 256, 0, st>>>(listA, n, seg, seg, m - mbar, len0, seed,
                                                                                   (uint32_t)(61 + code1), pbase);
        else
            range_kernel<<<dim3(blocks(3 * seg), (unsigned)BH), 256, 0, st>>>(listA, n, 0, seg, 3 * seg);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
        if (q == 0) {
            copy_list_kernel<<<dim3(blocks(3 * n_out), (unsigned)BH), 256, 0, st>>>(E, n_out, listA, n, 3 * n_out);
            count_launches(1);
            ELM_CUDA_TRY(cudaGetLastError());
        } else {
            // level i reads list i and writes list i + 1; the prefill keeps every list of the round
            // (the cache of an epoch is made of runs of them), compression alone alternates two
            int32_t *cur = listA, *nxt = listB;
            for (int i = 0; i < q; ++i) {
                const int per = 1 << (2 * (q - 1 - i));                       // calls per sibling
                const int P = (int)((len0 >> i) / per / 2);
                const double dlt = ldexp(dm, 2 * (i + 1 - q)) / (3.0 * (double)q);
                if (prefill) nxt = levels + (size_t)i * BH * n;
                const int rc = run_halve_level<Tin, T>(c, cur, i == q - 1 ? E + n_out : nxt, n, 3 * per, P, i + code1, dlt, per);
                if (rc != ELM_OK) return rc;
                int32_t *tmp = cur; cur = nxt; nxt = tmp;
            }
        }
        if (prefill && r >= 1) {
            // Thinformer Express (Algorithm 5) for the 3 n_out 2^m tokens of this round.  The cache a token
            // sees is E with the finished siblings (weight 1), in every S_i the outputs of level-(i-1)
            // Halve calls that level i has not consumed yet (weight 2^(i-q)), and in S_0 the kept points
            // since the last level-0 call, itself included (weight 2^-q).  It changes with every level-0
            // call, so the tokens are taken in windows: one attention launch per window over every entry
            // that some token of the window sees, each entry carrying the span of tokens that see it.
            // The launches are independent given the round's lists; they are dealt to EXPRESS_LANES
            // streams (each with its own list buffers) between two events.
            const RoundGeom g = round_geom(p, mbar, r);
            float *lse = g.sub ? reinterpret_cast<float *>(ws + L.lse) : nullptr;
            RoundUniverse u;
            if (round_universe(p, mbar, r, u)) {
                // one launch for the round: every entry the round's tokens ever see is gathered once, each pair of
                // query tiles streams the blocks its own tokens see
                const RoundBuffers rb = round_buffers(L, ws, BH, u.n_univ);
                const int rc = express_attend_round(Q, K, V, O, p, u, E, levels, (size_t)BH * n, listA, n, rb, lse, st);
                if (rc != ELM_OK) return rc;
            } else {
            const int64_t W = prefill_window(g), Wg = W >> g.wlog;
            ELM_CUDA_TRY(cudaEventRecord(fork, st));
            for (int i = 0; i < EXPRESS_LANES; ++i) ELM_CUDA_TRY(cudaStreamWaitEvent(side[i], fork, 0));
            int launch = 0;
            for (int jj = 0; jj < 3; ++jj) {
                for (int64_t G0 = 0; G0 < g.len0; G0 += Wg, ++launch) {
                    const int lane_id = launch % EXPRESS_LANES;
                    WindowPieces pc;
                    window_pieces(g, n_out, jj, G0, G0 + Wg, E, levels, (size_t)BH * n, listA, pc);
                    const int64_t t0 = (jj + 1) * seg + (G0 << g.wlog);
                    const int rc = express_attend_window(Q, K, V, O, p, L, ws, pc, t0, (int)W, lse, side[lane_id], lane_id);
                    if (rc != ELM_OK) return rc;
                }
            }
            for (int i = 0; i < EXPRESS_LANES; ++i) {
                ELM_CUDA_TRY(cudaEventRecord(join[i], side[i]));
                ELM_CUDA_TRY(cudaStreamWaitEvent(st, join[i], 0));             // the halvings overwrite E
            }
            }
            if (g.sub) {
                // the tokens Subsample dropped still attend to themselves
                const dim3 grid((unsigned)((3 * seg + 7) / 8), (unsigned)(p->batch * p->q_heads));
                self_merge_kernel<Tin, T><<<grid, 256, 0, st>>>(Q, K, V, O, lse, listA, p->q_heads, p->kv_heads, n, p->d, seg,
                                                                g.len0, g.wlog, (T)(-g.q));
                count_launches(1);
                ELM_CUDA_TRY(cudaGetLastError());
            }
        }
        // halve phase: 4 n_out -> 2 n_out -> n_out
        const bool last_round = r == R - 1;
        int rc = run_halve_level<Tin, T>(c, E, T1, n, 1, (int)(2 * n_out), (int)(62 + 64 * 4 * r), 0.5 * dm);
        if (rc != ELM_OK) return rc;
        rc = run_halve_level<Tin, T>(c, T1, last_round ? idx_out : E, last_round ? n_out : n, 1, (int)n_out,
                                     (int)(63 + 64 * 4 * r), 0.5 * dm);
        if (rc != ELM_OK) return rc;
    }
    {
        StageTimer t(ELM_STAGE_EMIT, st, 1);
        const int64_t total = (int64_t)BH * n_out;
        emit_kernel<<<blocks(total), 256, 0, st>>>(w_out, idx_out, total, n_out, R == 0);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}

}  // namespace elm

namespace elm {
// Validated arguments -> launches.  `pbase` numbers the call's first attention problem in the
// uniforms' counter, so that a batch processed in several slices draws the same uniforms as one call.
int compress_enqueue(const void *K, const void *V, const elm_params *params, uint64_t seed, int32_t *idx_out,
                     float *w_out, void *workspace, cudaStream_t st, uint32_t pbase)
{
    unsigned char *ws = (unsigned char *)workspace;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    if (params->dtype == ELM_E4M3) {
        // every E4M3 value is a bf16 value: widen K and V (exactly) and run the bf16 kernels on the copies
        typedef __nv_bfloat16 bf;
        const int64_t count = (int64_t)params->batch * params->kv_heads * params->n_kv * params->d;
        bf *Kw = reinterpret_cast<bf *>(ws + compress_layout(params).wide), *Vw = Kw + count;
        int rc = widen_e4m3(K, Kw, count, st);
        if (rc == ELM_OK) rc = widen_e4m3(V, Vw, count, st);
        if (rc != ELM_OK) return rc;
        return det ? compress_impl<bf, double>(Kw, Vw, params, seed, idx_out, w_out, ws, st, pbase)
                   : compress_impl<bf, float>(Kw, Vw, params, seed, idx_out, w_out, ws, st, pbase);
    }
    if (params->dtype == ELM_F32) {
        return det ? compress_impl<float, double>((const float *)K, (const float *)V, params, seed, idx_out, w_out, ws, st, pbase)
                   : compress_impl<float, float>((const float *)K, (const float *)V, params, seed, idx_out, w_out, ws, st, pbase);
    }
    return det ? compress_impl<__nv_bfloat16, double>((const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, params, seed, idx_out, w_out, ws, st, pbase)
               : compress_impl<__nv_bfloat16, float>((const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, params, seed, idx_out, w_out, ws, st, pbase);
}
}  // namespace elm

extern "C" int elm_compress(const void *K, const void *V, const elm_params *params, uint64_t seed,
                            int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes,
                            void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    int rc = validate_params(params, true);
    if (rc != ELM_OK) return rc;
    if (!K || !V || !idx_out || !w_out || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)idx_out | (uintptr_t)w_out) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < compress_layout(params).total) return ELM_ERR_WORKSPACE;
    return compress_enqueue(K, V, params, seed, idx_out, w_out, workspace, (cudaStream_t)stream, 0u);
}

extern "C" int elm_express_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes)
{
    using namespace elm;
    if (!params || !bytes) return ELM_ERR_NULL;
    const int rc = validate_express(params, mbar);
    if (rc != ELM_OK) return rc;
    *bytes = express_layout(params).total;
    return ELM_OK;
}

extern "C" int elm_express_compress(const void *K, const void *V, const elm_params *params, int32_t mbar, uint64_t seed,
                                    int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    const int rc = validate_express(params, mbar);
    if (rc != ELM_OK) return rc;
    if (!K || !V || !idx_out || !w_out || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)idx_out | (uintptr_t)w_out) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < express_layout(params).total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    if (params->dtype == ELM_F32) {
        return det ? express_impl<float, double>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u)
                   : express_impl<float, float>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u);
    }
    return det ? express_impl<__nv_bfloat16, double>((const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u)
               : express_impl<__nv_bfloat16, float>((const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u);
}

namespace elm {
// what the prefill needs on top of validate_express
static int validate_prefill(const elm_params *p, int32_t mbar)
{
    int rc = validate_express(p, mbar);
    if (rc != ELM_OK) return rc;
    if (p->q_heads < 1 || p->q_heads % p->kv_heads != 0 || (int64_t)p->batch * p->q_heads > 65535) return ELM_ERR_SHAPE;
    if (p->n_q != p->n_kv) return ELM_ERR_SHAPE;                       // one query per token
    const int R = express_rounds(p);
    const int qmax = 2 * (R - 1) < mbar ? 2 * (R - 1) : mbar;            // deepest Compress2 of the run
    if (R >= 2 && qmax > p->log2_nout + 1) return ELM_ERR_SHAPE;          // level-0 calls of at least 2 points
    return ELM_OK;
}
}  // namespace elm

extern "C" int elm_express_prefill_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes)
{
    using namespace elm;
    if (!params || !bytes) return ELM_ERR_NULL;
    const int rc = validate_prefill(params, mbar);
    if (rc != ELM_OK) return rc;
    *bytes = express_layout(params, mbar, true).total;
    return ELM_OK;
}

extern "C" int elm_express_prefill(const void *Q, const void *K, const void *V, const elm_params *params, int32_t mbar,
                                   uint64_t seed, void *O, int32_t *idx_out, float *w_out, void *workspace,
                                   size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    const int rc = validate_prefill(params, mbar);
    if (rc != ELM_OK) return rc;
    if (!Q || !K || !V || !O || !idx_out || !w_out || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O | (uintptr_t)idx_out | (uintptr_t)w_out) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < express_layout(params, mbar, true).total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    typedef __nv_bfloat16 bf;
    if (params->dtype == ELM_F32) {
        return det ? express_impl<float, double>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const float *)Q, (float *)O)
                   : express_impl<float, float>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const float *)Q, (float *)O);
    }
    return det ? express_impl<bf, double>((const bf *)K, (const bf *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const bf *)Q, (bf *)O)
               : express_impl<bf, float>((const bf *)K, (const bf *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const bf *)Q, (bf *)O);
}

// ---------------------------------------------------------------------------------------------
// Compress2 on a sequence of any length (Algorithm 2 after n_mid updates), the first n_sink and the
// last n_window rows kept exactly.  Level i makes floor(a_i / thresh_i) Halve calls on consecutive
// stretches of thresh_i = n_out 2^(i - m + 2) points (a_0 = n_mid, a_(i+1) = calls_i thresh_i / 2);
// what is left over stays in S_i with weight 2^(i - m).  The output is wtd_cache() between the
// sink and the window rows, all weights divided by their sum n 2^-m.
// ---------------------------------------------------------------------------------------------
namespace elm {
struct RaggedPlan {
    int64_t thresh[16], calls[16], left[16];     // per level 0..m-1
    int64_t top;                                 // points in S_m
    int64_t n_mid, count;
};
static int ragged_plan(const elm_params *p, int32_t n_sink, int32_t n_window, RaggedPlan &pl)
{
    if (p->batch < 1 || p->kv_heads < 1) return ELM_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return ELM_ERR_SHAPE;
    if (p->log2_nout < 0 || p->log2_nout > 24 || p->m < 0 || p->m > 12 || p->log2_nout + p->m > 30) return ELM_ERR_SHAPE;
    if (p->m >= 1 && p->log2_nout - p->m + 2 < 1) return ELM_ERR_SHAPE;       // level-0 calls of at least one pair
    if ((int64_t)p->batch * p->kv_heads > 65535) return ELM_ERR_SHAPE;
    if (p->n_kv < 1 || n_sink < 0 || n_window < 0) return ELM_ERR_SHAPE;
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    pl.n_mid = (int64_t)p->n_kv - n_sink - n_window;
    if (pl.n_mid < 0 || pl.n_mid > (n_out << p->m)) return ELM_ERR_SHAPE;
    if (p->dtype != ELM_F32 && p->dtype != ELM_BF16) return ELM_ERR_DTYPE;
    if (p->precision != ELM_PREC_FP64_DET && p->precision != ELM_PREC_FP32) return ELM_ERR_DTYPE;
    if (!(p->delta > 0.0 && p->delta < 1.0)) return ELM_ERR_DELTA;
    if (p->delta_level)
        for (int i = 0; i < p->m; ++i)
            if (!(p->delta_level[i] > 0.0 && p->delta_level[i] < 1.0)) return ELM_ERR_DELTA;
    int64_t a = pl.n_mid;
    pl.count = (int64_t)n_sink + n_window;
    for (int i = 0; i < p->m; ++i) {
        pl.thresh[i] = (n_out << (i + 2)) >> p->m;
        pl.calls[i] = a / pl.thresh[i];
        pl.left[i] = a - pl.calls[i] * pl.thresh[i];
        pl.count += pl.left[i];
        a = pl.calls[i] * (pl.thresh[i] / 2);
    }
    pl.top = a;
    pl.count += a;
    return ELM_OK;
}

template <typename Tin, typename T>
static int ragged_impl(const Tin *K, const Tin *V, const elm_params *p, const RaggedPlan &pl, int32_t n_sink,
                       int32_t n_window, uint64_t seed, int32_t *idx_out, float *w_out, unsigned char *ws, cudaStream_t st)
{
    const CompressLayout L = compress_layout(p);
    const int BH = p->batch * p->kv_heads;
    const int64_t n = p->n_kv;
    const int m = p->m;
    LevelCtx<Tin, T> c;
    c.K = K; c.V = V; c.p = p;
    c.vmax_bits = reinterpret_cast<unsigned *>(ws + L.vmax_bits);
    c.status = reinterpret_cast<int *>(c.vmax_bits + BH);
    c.cnorm = reinterpret_cast<T *>(ws + L.cnorm);
    c.Mpair = reinterpret_cast<T *>(ws + L.Mpair);
    c.rdecay = reinterpret_cast<T *>(ws + L.rdecay);
    c.F = reinterpret_cast<T *>(ws + L.F);
    c.F_stride = (int64_t)L.F_stride;
    c.seed = seed; c.pbase = 0; c.st = st;
    int32_t *list[2] = {reinterpret_cast<int32_t *>(ws + L.cur), reinterpret_cast<int32_t *>(ws + L.nxt)};
    double dl[32];
    if (p->delta_level) {
        for (int i = 0; i < m; ++i) dl[i] = p->delta_level[i];
    } else {
        elm_default_delta_levels(m, p->delta, dl);
    }
    auto blocks = [](int64_t count) { return (unsigned)((count + 255) / 256); };
    {
        // key norms and v_max over every row of the problem; level 0 starts as the middle rows in order
        StageTimer t(ELM_STAGE_PREPASS, st, 2);
        ELM_CUDA_TRY(cudaMemsetAsync(c.vmax_bits, 0, (size_t)(BH + 1) * 4, st));
        prepass_kernel<Tin, T><<<dim3(blocks(n), (unsigned)BH), 256, 0, st>>>(K, V, n, p->d, c.cnorm, c.vmax_bits, list[1]);
        count_launches(1);
        if (pl.n_mid > 0) {
            range_kernel<<<dim3(blocks(pl.n_mid), (unsigned)BH), 256, 0, st>>>(list[0], n, 0, n_sink, pl.n_mid);
            count_launches(1);
        }
        ELM_CUDA_TRY(cudaGetLastError());
    }
    // Level i reads list[i & 1] and writes its survivors to the front of the other list.  What it
    // leaves over sits behind the stretches it consumed, at offset calls_i thresh_i; every later
    // level writes fewer than a quarter as many entries to that list, so the leftovers stay intact
    // until the output is assembled.
    ListPieces pc = {};
    int k = 0;
    int32_t at = 0;
    auto piece = [&](const int32_t *src, int64_t off, int64_t count, double wgt) {
        if (count <= 0) return;
        pc.src[k] = src; pc.src_off[k] = off; pc.w[k] = (float)wgt; pc.dst_off[k] = at;
        at += (int32_t)count;
        ++k;
    };
    piece(nullptr, 0, n_sink, 1.0 / (double)n);
    for (int i = 0; i < m; ++i) {
        if (pl.calls[i] > 0) {
            const int rc = run_halve_level<Tin, T>(c, list[i & 1], list[(i + 1) & 1], n, (int)pl.calls[i],
                                                   (int)(pl.thresh[i] / 2), i, dl[i]);
            if (rc != ELM_OK) return rc;
        }
        piece(list[i & 1], pl.calls[i] * pl.thresh[i], pl.left[i], ldexp(1.0, i) / (double)n);
    }
    piece(list[m & 1], 0, pl.top, ldexp(1.0, m) / (double)n);
    piece(nullptr, n - n_window, n_window, 1.0 / (double)n);
    pc.dst_off[k] = at;
    pc.n = k;
    {
        StageTimer t(ELM_STAGE_EMIT, st, 1);
        build_list_kernel<<<dim3(blocks(at), (unsigned)BH), 256, 0, st>>>(pc, n, idx_out, w_out, at);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}
}  // namespace elm

extern "C" int elm_compress_ragged_count(const elm_params *params, int32_t n_sink, int32_t n_window, int32_t *count,
                                         size_t *workspace_bytes)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    RaggedPlan pl;
    const int rc = ragged_plan(params, n_sink, n_window, pl);
    if (rc != ELM_OK) return rc;
    if (count) *count = (int32_t)pl.count;
    if (workspace_bytes) *workspace_bytes = compress_layout(params).total;
    return ELM_OK;
}

extern "C" int elm_compress_ragged(const void *K, const void *V, const elm_params *params, int32_t n_sink, int32_t n_window,
                                   uint64_t seed, int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes,
                                   void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    RaggedPlan pl;
    const int rc = ragged_plan(params, n_sink, n_window, pl);
    if (rc != ELM_OK) return rc;
    if (!K || !V || !idx_out || !w_out || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)idx_out | (uintptr_t)w_out) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < compress_layout(params).total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    typedef __nv_bfloat16 bf;
    if (params->dtype == ELM_F32) {
        return det ? ragged_impl<float, double>((const float *)K, (const float *)V, params, pl, n_sink, n_window, seed, idx_out, w_out, ws, st)
                   : ragged_impl<float, float>((const float *)K, (const float *)V, params, pl, n_sink, n_window, seed, idx_out, w_out, ws, st);
    }
    return det ? ragged_impl<bf, double>((const bf *)K, (const bf *)V, params, pl, n_sink, n_window, seed, idx_out, w_out, ws, st)
               : ragged_impl<bf, float>((const bf *)K, (const bf *)V, params, pl, n_sink, n_window, seed, idx_out, w_out, ws, st);
}

// ---------------------------------------------------------------------------------------------
// Streaming Thinformer Express: the host struct elm_stream carries the counters of Algorithms 1-2
// (they depend on the token count alone), the device workspace the point lists E, S_0..S_mbar.
// ---------------------------------------------------------------------------------------------
namespace elm {
struct StreamLayout {
    size_t vmax_bits, cnorm, E, T1, S, Mpair, rdecay, F, F_stride, ep_idx, ep_w, ws_attend, ep_cap, total;
};
static StreamLayout stream_layout(const elm_params *p, int mbar)
{
    StreamLayout L;
    const size_t ts = p->precision == ELM_PREC_FP64_DET ? 8 : 4;
    const size_t BH = (size_t)p->batch * p->kv_heads;
    const size_t n = (size_t)p->n_kv;
    const size_t n_out = (size_t)1 << p->log2_nout;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.vmax_bits = take((BH + 1) * 4);
    L.cnorm = take(BH * n * ts);
    L.E = take(BH * n * 4);                    // every point list is [BH][n_kv]-strided, like the lists of elm_compress
    L.T1 = take(BH * n * 4);
    L.S = take((size_t)(mbar + 1) * BH * n * 4);
    L.Mpair = take(BH * (n / 2 + 1) * ts);
    L.rdecay = take(BH * (n / 2 + 1) * ts);
    L.F_stride = 4 * n_out * n_out;
    L.F = take(BH * L.F_stride * ts);
    L.ep_cap = 6 * n_out + 1;                  // Theorem 1's cache bound, plus the token itself
    L.ep_idx = take(BH * L.ep_cap * 4);
    L.ep_w = take(BH * L.ep_cap * 4);
    elm_params one = *p;
    one.n_q = 1;
    L.ws_attend = take(attend_layout(&one, (int32_t)L.ep_cap).total);
    L.total = off;
    return L;
}
static int validate_stream(const elm_params *p, int32_t mbar)
{
    if (p->batch < 1 || p->kv_heads < 1 || p->q_heads < 1 || p->q_heads % p->kv_heads != 0) return ELM_ERR_SHAPE;
    if ((int64_t)p->batch * p->q_heads > 65535) return ELM_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return ELM_ERR_SHAPE;
    if (p->log2_nout < 1 || p->log2_nout > 24 || mbar < 0 || mbar > 12) return ELM_ERR_SHAPE;
    if (p->n_kv < 2 || p->n_q != 1) return ELM_ERR_SHAPE;
    if (p->dtype != ELM_F32 && p->dtype != ELM_BF16) return ELM_ERR_DTYPE;
    if (p->precision != ELM_PREC_FP64_DET && p->precision != ELM_PREC_FP32) return ELM_ERR_DTYPE;
    if (!(p->delta > 0.0 && p->delta < 1.0)) return ELM_ERR_DELTA;
    return ELM_OK;
}
__global__ void append_kernel(int32_t *__restrict__ list, int64_t stride, int64_t pos, int32_t value, int problems)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < problems) list[(int64_t)p * stride + pos] = value;
}

// wtd_cache() of Algorithm 1 (+ the token t itself when t >= 0) as list pieces
static void stream_pieces(const elm_stream *s, const int64_t *n_S, const StreamLayout &L, unsigned char *ws,
                          const elm_params *p, int64_t t, ListPieces &pc)
{
    const size_t BH = (size_t)p->batch * p->kv_heads;
    int32_t *S = reinterpret_cast<int32_t *>(ws + L.S);
    int k = 0;
    int32_t at = 0;
    auto piece = [&](const int32_t *src, int64_t off, int64_t count, float wgt) {
        if (count <= 0) return;
        pc.src[k] = src; pc.src_off[k] = off; pc.w[k] = wgt; pc.dst_off[k] = at;
        at += (int32_t)count;
        ++k;
    };
    for (int i = 0; i <= s->q; ++i) piece(S + (size_t)i * BH * p->n_kv, 0, n_S[i], (float)ldexp(1.0, i - s->q));
    piece(reinterpret_cast<int32_t *>(ws + L.E), 0, s->n_E, 1.f);
    if (t >= 0) piece(nullptr, t, 1, (float)ldexp(1.0, -s->q));          // the token enters S_0
    pc.dst_off[k] = at;
    pc.n = k;
}

// Subsample (Algorithm 3) in a streaming run.  Inside a stratum of 2^wlog tokens problem p keeps the token
// at offset floor(U 2^wlog), U the uniform of counter (stratum, 0, code, p): the problems take their
// Compress2.update at different tokens of the stratum, so at the token with offset o a problem is either
// still in the state the stratum began with (`a`) or already in the state it ends with (`b`: kept offset
// < o).  The two states differ only in how many entries of the same lists count.
struct StratumDraw {
    uint64_t seed;
    uint32_t stratum, code;
    int32_t wlog;
    int64_t o;
};
__host__ __device__ __forceinline__ int64_t kept_offset(const StratumDraw &d, uint32_t problem)
{
    return (int64_t)floor(halving_uniform<double>(d.seed, d.stratum, 0u, d.code, problem) * (double)((int64_t)1 << d.wlog));
}
// Like build_list_kernel with the list chosen per problem.  The two lists may differ in length; a list
// shorter than `total` repeats its last entry over the remaining slots with that entry's weight divided
// among the copies, which leaves every weighted sum over the list unchanged.
__global__ void build_list_choice_kernel(ListPieces a, ListPieces b, StratumDraw dr, int64_t src_stride,
                                         int32_t *__restrict__ idx, float *__restrict__ w, int total)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int64_t pr = blockIdx.y;
    const ListPieces &pc = kept_offset(dr, (uint32_t)pr) < dr.o ? b : a;
    const int len = pc.dst_off[pc.n];
    const int ii = i < len ? i : len - 1;
    int k = 0;
    while (ii >= pc.dst_off[k + 1]) ++k;
    const int64_t o = ii - pc.dst_off[k];
    idx[pr * total + i] = pc.src[k] ? pc.src[k][pr * src_stride + pc.src_off[k] + o] : (int32_t)(pc.src_off[k] + o);
    w[pr * total + i] = ii == len - 1 ? pc.w[k] / (float)(total - len + 1) : pc.w[k];
}
// S_0 of every problem that keeps the token gets it at position `pos`.
__global__ void append_kept_kernel(int32_t *__restrict__ list, int64_t stride, int64_t pos, int32_t value, int problems,
                                   StratumDraw dr)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < problems && kept_offset(dr, (uint32_t)p) == dr.o) list[(int64_t)p * stride + pos] = value;
}

// The stratum the next token of a subsampled thin phase falls in, and the level counters a problem has after
// it took the stratum's update (n_S plus one point in S_0, then the Halve calls that come due).
// Returns false when Subsample is not active.
static bool stratum_state(const elm_stream *s, int64_t n_out, StratumDraw &dr, int64_t nS_after[16], bool call_due[16])
{
    for (int i = 0; i < 16; ++i) { nS_after[i] = s->n_S[i]; call_due[i] = false; }
    if (!(s->m > s->mbar && s->n >= n_out)) return false;                  // thin phase with thinning factor above mbar
    dr.seed = s->seed;
    dr.wlog = s->m - s->mbar;
    dr.stratum = (uint32_t)(s->ell >> dr.wlog);
    dr.o = s->ell & (((int64_t)1 << dr.wlog) - 1);
    dr.code = (uint32_t)(61 + 64 * (4 * (s->m / 2) + s->b + 1));
    nS_after[0] += 1;
    for (int i = 0; i < s->q; ++i) {
        const int64_t thresh = ((n_out << s->q) << i) >> (2 * (s->q - 1));
        if (nS_after[i] != thresh) continue;
        call_due[i] = true;
        nS_after[i + 1] += thresh / 2;
        nS_after[i] = 0;
    }
    return true;
}

template <typename Tin, typename T>
static int stream_step_impl(elm_stream *s, const Tin *Q, const Tin *K, const Tin *V, const elm_params *p, Tin *O,
                            unsigned char *ws, cudaStream_t st)
{
    const StreamLayout L = stream_layout(p, s->mbar);
    const int BH = p->batch * p->kv_heads;
    const int64_t n = p->n_kv, n_out = (int64_t)1 << p->log2_nout;
    const int64_t t = s->n;
    if (t >= n) return ELM_ERR_SHAPE;                                      // capacity
    if (s->q >= 1 && p->log2_nout + 2 - s->q < 1) return ELM_ERR_SHAPE;     // level-0 calls of at least 2 points
    LevelCtx<Tin, T> c;
    c.K = K; c.V = V; c.p = p;
    c.vmax_bits = reinterpret_cast<unsigned *>(ws + L.vmax_bits);
    c.status = reinterpret_cast<int *>(c.vmax_bits + BH);
    c.cnorm = reinterpret_cast<T *>(ws + L.cnorm);
    c.Mpair = reinterpret_cast<T *>(ws + L.Mpair);
    c.rdecay = reinterpret_cast<T *>(ws + L.rdecay);
    c.F = reinterpret_cast<T *>(ws + L.F);
    c.F_stride = (int64_t)L.F_stride;
    c.seed = s->seed; c.pbase = 0; c.st = st;
    int32_t *E = reinterpret_cast<int32_t *>(ws + L.E);
    int32_t *T1 = reinterpret_cast<int32_t *>(ws + L.T1);
    int32_t *S = reinterpret_cast<int32_t *>(ws + L.S);
    auto Slist = [&](int i) { return S + (size_t)i * BH * n; };
    auto blocks = [](int64_t count) { return (unsigned)((count + 255) / 256); };
    if (t >= s->n_known) {
        // a token that was not there at init: its key norm, and v_max grows with it
        prepass_kernel<Tin, T><<<dim3(1, (unsigned)BH), 256, 0, st>>>(K, V, n, p->d, c.cnorm, c.vmax_bits, T1, t, t + 1);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    // ---- Subsample bookkeeping: the stratum of this token and the state a problem is in after its update ----
    StratumDraw dr = {};
    int64_t nS_after[16];
    bool call_due[16];
    const bool sub = stratum_state(s, n_out, dr, nS_after, call_due);
    // ---- Algorithm 5: attend over wtd_cache() plus the token ----
    {
        ListPieces pc = {};
        stream_pieces(s, s->n_S, L, ws, p, t, pc);
        int total = pc.dst_off[pc.n];
        int32_t *ep_idx = reinterpret_cast<int32_t *>(ws + L.ep_idx);
        float *ep_w = reinterpret_cast<float *>(ws + L.ep_w);
        if (sub && dr.o > 0) {
            // some problems have taken this stratum's update already
            ListPieces pb = {};
            stream_pieces(s, nS_after, L, ws, p, t, pb);
            if (pb.dst_off[pb.n] > total) total = pb.dst_off[pb.n];
            if ((size_t)total > L.ep_cap) return ELM_ERR_WORKSPACE;
            build_list_choice_kernel<<<dim3(blocks(total), (unsigned)BH), 256, 0, st>>>(pc, pb, dr, n, ep_idx, ep_w, total);
        } else {
            build_list_kernel<<<dim3(blocks(total), (unsigned)BH), 256, 0, st>>>(pc, n, ep_idx, ep_w, total);
        }
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
        const int rc = attend_enqueue(Q, K, V, ep_idx, ep_w, total, p, O, ws + L.ws_attend, st);
        if (rc != ELM_OK) return rc;
    }
    // ---- Algorithm 1: Express.update ----
    auto append = [&](int32_t *list, int64_t pos) {
        append_kernel<<<(BH + 127) / 128, 128, 0, st>>>(list, n, pos, (int32_t)t, BH);
        count_launches(1);
        return cuda_status(cudaGetLastError());
    };
    s->n += 1;
    if (s->n <= n_out) {                                                   // exact phase
        const int rc = append(E, s->n_E);
        s->n_E += 1;
        return rc;
    }
    s->ell += 1;                                                           // thin phase: Compress2.update
    if (sub) {
        // Subsample: only the problems whose draw is this token take the update now; the counters in *s
        // move on when the stratum ends
        append_kept_kernel<<<(BH + 127) / 128, 128, 0, st>>>(Slist(0), n, s->n_S[0], (int32_t)t, BH, dr);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
        if (call_due[0]) {
            const double dm = kh_express_delta(p->delta, s->m);
            const int q = s->q;
            for (int pi = 0; pi < BH; ++pi) {
                if (kept_offset(dr, (uint32_t)pi) != dr.o) continue;
                // the Halve calls of this one problem: the level machinery on its slice of every array
                elm_params p1 = *p;
                p1.batch = 1; p1.kv_heads = 1; p1.q_heads = 1;
                LevelCtx<Tin, T> c1 = c;
                c1.p = &p1;
                c1.K = K + (int64_t)pi * n * p->d;
                c1.V = V + (int64_t)pi * n * p->d;
                c1.vmax_bits = c.vmax_bits + pi;
                c1.cnorm = c.cnorm + (int64_t)pi * n;
                c1.Mpair = c.Mpair + (int64_t)pi * (n / 2);
                c1.rdecay = c.rdecay + (int64_t)pi * (n / 2);
                c1.F = c.F + (int64_t)pi * c.F_stride;
                c1.pbase = (uint32_t)pi;
                for (int i = 0; i < q && call_due[i]; ++i) {
                    const int64_t thresh = ((n_out << q) << i) >> (2 * (q - 1));
                    const double dlt = ldexp(dm, 2 * (i + 1 - q)) / (3.0 * (double)q);
                    const int code = i + 64 * (4 * (s->m / 2) + s->b + 1);
                    const int rc = run_halve_level<Tin, T>(c1, Slist(i) + (int64_t)pi * n,
                                                           Slist(i + 1) + (int64_t)pi * n + s->n_S[i + 1], n, 1,
                                                           (int)(thresh / 2), code, dlt, 0, s->calls[i]);
                    if (rc != ELM_OK) return rc;
                }
            }
        }
        if (dr.o == ((int64_t)1 << dr.wlog) - 1) {                         // the stratum ends: every problem has updated
            for (int i = 0; i < 16; ++i) {
                s->n_S[i] = nS_after[i];
                if (call_due[i]) s->calls[i] += 1;
            }
        }
    } else {
        const int q = s->q;
        int rc = append(Slist(0), s->n_S[0]);
        if (rc != ELM_OK) return rc;
        s->n_S[0] += 1;
        const double dm = kh_express_delta(p->delta, s->m);
        for (int i = 0; i < q; ++i) {
            const int64_t thresh = ((n_out << q) << i) >> (2 * (q - 1));  // n_in 2^i / 4^(q-1)
            if (s->n_S[i] != thresh) continue;
            const double dlt = ldexp(dm, 2 * (i + 1 - q)) / (3.0 * (double)q);
            const int code = i + 64 * (4 * (s->m / 2) + s->b + 1);
            rc = run_halve_level<Tin, T>(c, Slist(i), Slist(i + 1) + s->n_S[i + 1], n, 1, (int)(thresh / 2), code, dlt, 0,
                                         s->calls[i]);
            if (rc != ELM_OK) return rc;
            s->calls[i] += 1;
            s->n_S[i + 1] += thresh / 2;
            s->n_S[i] = 0;
        }
    }
    if (s->ell == (n_out << s->m)) {                                       // the segment is done: S_q joins E
        copy_list_kernel<<<dim3(blocks(s->n_S[s->q]), (unsigned)BH), 256, 0, st>>>(E, s->n_E, Slist(s->q), n, s->n_S[s->q]);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
        s->n_E += s->n_S[s->q];
        s->n_S[s->q] = 0;
        s->ell = 0;
        s->b += 1;
    }
    if (s->n == 4 * (n_out << s->m)) {                                     // halve phase
        const double dm = kh_express_delta(p->delta, s->m);
        int rc = run_halve_level<Tin, T>(c, E, T1, n, 1, (int)(2 * n_out), 62 + 64 * 4 * (s->m / 2), 0.5 * dm);
        if (rc != ELM_OK) return rc;
        rc = run_halve_level<Tin, T>(c, T1, E, n, 1, (int)n_out, 63 + 64 * 4 * (s->m / 2), 0.5 * dm);
        if (rc != ELM_OK) return rc;
        s->n_E = n_out;
        s->m += 2;
        s->b = 0;
    }
    if (s->ell == 0) {                                                     // a new Compress2 instance
        s->q = s->m < s->mbar ? s->m : s->mbar;
        for (int i = 0; i < 16; ++i) { s->n_S[i] = 0; s->calls[i] = 0; }
    }
    return ELM_OK;
}
}  // namespace elm

extern "C" int elm_stream_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes)
{
    using namespace elm;
    if (!params || !bytes) return ELM_ERR_NULL;
    const int rc = validate_stream(params, mbar);
    if (rc != ELM_OK) return rc;
    *bytes = stream_layout(params, mbar).total;
    return ELM_OK;
}

extern "C" int elm_stream_init(elm_stream *s, const void *K, const void *V, int64_t n_known, const elm_params *params,
                               int32_t mbar, uint64_t seed, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!s || !params || !workspace) return ELM_ERR_NULL;
    const int rc = validate_stream(params, mbar);
    if (rc != ELM_OK) return rc;
    if (n_known < 0 || n_known > params->n_kv || (n_known > 0 && (!K || !V))) return ELM_ERR_SHAPE;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    const StreamLayout L = stream_layout(params, mbar);
    if (workspace_bytes < L.total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const int BH = params->batch * params->kv_heads;
    *s = elm_stream{};
    s->mbar = mbar;
    s->seed = seed;
    s->n_known = n_known;
    ELM_CUDA_TRY(cudaMemsetAsync(ws + L.vmax_bits, 0, (size_t)(BH + 1) * 4, st));
    if (n_known > 0) {
        const dim3 grid((unsigned)((n_known + 255) / 256), (unsigned)BH);
        unsigned *vb = reinterpret_cast<unsigned *>(ws + L.vmax_bits);
        int32_t *scratch = reinterpret_cast<int32_t *>(ws + L.T1);
        const int64_t n = params->n_kv;
        typedef __nv_bfloat16 bf;
        if (params->dtype == ELM_F32) {
            if (params->precision == ELM_PREC_FP64_DET)
                prepass_kernel<float, double><<<grid, 256, 0, st>>>((const float *)K, (const float *)V, n, params->d, reinterpret_cast<double *>(ws + L.cnorm), vb, scratch, 0, n_known);
            else
                prepass_kernel<float, float><<<grid, 256, 0, st>>>((const float *)K, (const float *)V, n, params->d, reinterpret_cast<float *>(ws + L.cnorm), vb, scratch, 0, n_known);
        } else {
            if (params->precision == ELM_PREC_FP64_DET)
                prepass_kernel<bf, double><<<grid, 256, 0, st>>>((const bf *)K, (const bf *)V, n, params->d, reinterpret_cast<double *>(ws + L.cnorm), vb, scratch, 0, n_known);
            else
                prepass_kernel<bf, float><<<grid, 256, 0, st>>>((const bf *)K, (const bf *)V, n, params->d, reinterpret_cast<float *>(ws + L.cnorm), vb, scratch, 0, n_known);
        }
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}

extern "C" int elm_stream_step(elm_stream *s, const void *Q_t, const void *K, const void *V, const elm_params *params,
                               void *O_t, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!s || !params) return ELM_ERR_NULL;
    const int rc = validate_stream(params, s->mbar);
    if (rc != ELM_OK) return rc;
    if (!Q_t || !K || !V || !O_t || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)Q_t | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O_t) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < stream_layout(params, s->mbar).total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    typedef __nv_bfloat16 bf;
    if (params->dtype == ELM_F32) {
        return det ? stream_step_impl<float, double>(s, (const float *)Q_t, (const float *)K, (const float *)V, params, (float *)O_t, ws, st)
                   : stream_step_impl<float, float>(s, (const float *)Q_t, (const float *)K, (const float *)V, params, (float *)O_t, ws, st);
    }
    return det ? stream_step_impl<bf, double>(s, (const bf *)Q_t, (const bf *)K, (const bf *)V, params, (bf *)O_t, ws, st)
               : stream_step_impl<bf, float>(s, (const bf *)Q_t, (const bf *)K, (const bf *)V, params, (bf *)O_t, ws, st);
}

extern "C" int elm_stream_steps(elm_stream *s, int32_t n_tokens, const void *Q_T, const void *K, const void *V,
                                const elm_params *params, void *O_T, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!s || !params) return ELM_ERR_NULL;
    if (n_tokens < 0) return ELM_ERR_SHAPE;
    if (n_tokens > 0 && (!Q_T || !O_T)) return ELM_ERR_NULL;
    const size_t per_token = (size_t)params->batch * params->q_heads * params->d * elm::elt_bytes(params->dtype);
    if (per_token & 15) return ELM_ERR_ALIGN;
    for (int32_t i = 0; i < n_tokens; ++i) {
        const int rc = elm_stream_step(s, (const unsigned char *)Q_T + (size_t)i * per_token, K, V, params,
                                       (unsigned char *)O_T + (size_t)i * per_token, workspace, workspace_bytes, stream);
        if (rc != ELM_OK) return rc;
    }
    return ELM_OK;
}

extern "C" int elm_stream_cache(const elm_stream *s, const elm_params *params, int32_t *idx_out, float *w_out,
                                int32_t *count_host, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!s || !params || !idx_out || !w_out || !count_host || !workspace) return ELM_ERR_NULL;
    const int rc = validate_stream(params, s->mbar);
    if (rc != ELM_OK) return rc;
    const StreamLayout L = stream_layout(params, s->mbar);
    if (workspace_bytes < L.total) return ELM_ERR_WORKSPACE;
    ListPieces pc = {};
    stream_pieces(s, s->n_S, L, (unsigned char *)workspace, params, -1, pc);
    int total = pc.dst_off[pc.n];
    // Inside a stratum of a subsampled phase the problems that have kept their point hold one update more
    // than the others; a shorter list is padded by repeating its last entry with the weight split.
    StratumDraw dr = {};
    int64_t nS_after[16];
    bool call_due[16];
    const bool mixed = stratum_state(s, (int64_t)1 << params->log2_nout, dr, nS_after, call_due) && dr.o > 0;
    ListPieces pb = {};
    if (mixed) {
        stream_pieces(s, nS_after, L, (unsigned char *)workspace, params, -1, pb);
        if (pb.dst_off[pb.n] > total) total = pb.dst_off[pb.n];
    }
    *count_host = total;
    if (total > 0) {
        const dim3 grid((unsigned)((total + 255) / 256), (unsigned)(params->batch * params->kv_heads));
        if (mixed)
            build_list_choice_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(pc, pb, dr, params->n_kv, idx_out, w_out, total);
        else
            build_list_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(pc, params->n_kv, idx_out, w_out, total);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}
