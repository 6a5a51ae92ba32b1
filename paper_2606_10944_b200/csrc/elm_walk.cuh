// Device-side pieces of the halving walk (Algorithm A.1) shared by the walk kernels and by the
// Gram kernel that walks small calls in its own epilogue.
#pragma once
#include <math.h>
#include <stdint.h>

namespace elm {

// swap iff U < min(1, (1/2)(1 - alpha/a)_+);  a == 0 (or not finite) => probability 1/2
__device__ __forceinline__ bool swap_decision(double alpha, double a, double U)
{
    double p = 0.5;
    if (a > 0.0 && isfinite(a)) {
        double t = 1.0 - alpha / a;
        t = t < 0.0 ? 0.0 : t;
        p = 0.5 * t;
        p = p > 1.0 ? 1.0 : p;
    }
    return U < p;
}
// fp32 mode: the same test with the division cleared, alpha < a (1 - 2U)
__device__ __forceinline__ bool swap_decision(float alpha, float a, float U)
{
    if (a > 0.f && isfinite(a)) return alpha < a * (1.f - 2.f * U);
    return U < 0.5f;
}

// fp32 walker: the 32 serial steps of a block run in ONE thread with the diagonal tile in shared
// memory (row stride LD floats, a multiple of 4).  Thread-local state d[u] = alpha_u - a_u (1 - 2 U_u) makes "swap pair u" the sign test
// d[u] < 0; a decision then updates the later d[u] with independent FMAs, so a step costs one
// compare-select-FMA chain instead of a warp vote.  b_u = 0 (a_u = 0) needs no special case in the
// updates because then F[., u] = 0 (Cauchy-Schwarz in the RKHS); its decision is U_u < 1/2.
__device__ __forceinline__ uint32_t walk_block_thread_ld(const float *__restrict__ tile, const int LD,
                                                         const float *__restrict__ alpha32,
                                                         const float *__restrict__ b32, const float *__restrict__ r32,
                                                         const float *__restrict__ U32, float logfac, float &bmax)
{
    float d[32];
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        const float bt = b32[t], carried = bmax * r32[t];
        bmax = bt > carried ? bt : carried;
        const float a = bt * bmax * logfac;
        const float U = U32[t];
        d[t] = (a > 0.f && isfinite(a)) ? alpha32[t] - a * (1.f - 2.f * U) : (U < 0.5f ? -1.f : 1.f);
    }
    uint32_t swaps = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        const bool sw = d[t] < 0.f;
        swaps |= (sw ? 1u : 0u) << t;
        const float s = sw ? 1.f : -1.f;          // alpha_u = -sum_j eta_j F[j,u]: kept pair subtracts
        const float4 *row = reinterpret_cast<const float4 *>(tile + t * LD);
#pragma unroll
        for (int g4 = (t + 1) / 4; g4 < 8; ++g4) {
            const float4 v = row[g4];
            if (4 * g4 + 0 > t) d[4 * g4 + 0] = fmaf(s, v.x, d[4 * g4 + 0]);
            if (4 * g4 + 1 > t) d[4 * g4 + 1] = fmaf(s, v.y, d[4 * g4 + 1]);
            if (4 * g4 + 2 > t) d[4 * g4 + 2] = fmaf(s, v.z, d[4 * g4 + 2]);
            if (4 * g4 + 3 > t) d[4 * g4 + 3] = fmaf(s, v.w, d[4 * g4 + 3]);
        }
    }
    return swaps;
}
template <int LD>
__device__ __forceinline__ uint32_t walk_block_thread(const float *__restrict__ tile, const float *__restrict__ alpha32,
                                                      const float *__restrict__ b32, const float *__restrict__ r32,
                                                      const float *__restrict__ U32, float logfac, float &bmax)
{
    return walk_block_thread_ld(tile, LD, alpha32, b32, r32, U32, logfac, bmax);
}

// The serial part of a 32-pair block with everything in registers: Fd[t] = F[i0 + t, i0 + lane]
// (used for t < lane), b = b_i of this lane's pair.  No memory operation inside.
template <typename T>
__device__ __forceinline__ uint32_t walk_block_regs(const T (&Fd)[32], T b, T alpha, T r, T U, T logfac,
                                                    T &bmax, int lane)
{
    T my_bmax = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        T bt = __shfl_sync(0xffffffffu, b, t);
        T rt = __shfl_sync(0xffffffffu, r, t);
        T carried = bmax * rt;
        bmax = bt > carried ? bt : carried;
        if (t == lane) my_bmax = bmax;
    }
    const T a = b * my_bmax * logfac;
    uint32_t swaps = 0;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        bool mine = (lane == t) && swap_decision(alpha, a, U);
        uint32_t sw = (__ballot_sync(0xffffffffu, mine) >> t) & 1u;
        swaps |= sw << t;
        T f = t < lane ? Fd[t] : (T)0;
        alpha += sw ? f : -f;
    }
    return swaps;
}

}  // namespace elm
