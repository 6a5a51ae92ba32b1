// Device-side pieces of the halving walk (Algorithm A.1) shared by the walk kernels and by the
// Gram kernel that walks small calls in its own epilogue.
#pragma once
#include <math.h>
#include <stdint.h>

#include "elm_sm100.cuh"

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

// ---------------------------------------------------------------------------------------------
// fp32 block walker: the serial chain itself, run redundantly by every lane so that
// nothing is communicated inside it.  Every lane keeps broadcast copies x[0..8) of the scores of the
// eight pairs being decided (as four packed pairs); a decision is one sign-bit operation on x[t],
// followed by packed fused multiply-adds that fold it into the later x and into the lane's own
// column d and (NEXT) the same column of the next block, dn.  The scores of the next eight pairs
// are fetched from the lanes that own those columns two decisions before they are needed - hiding
// the shuffle latency - and the two decisions taken meanwhile are folded into the copies.
// A score of -0.0 counts as negative (the test reads the sign bit).  A single warp issues roughly
// one instruction every third cycle on this part, so the instruction count per pair is what this
// form keeps low.  The rows of F are fetched from shared memory three pairs ahead of their use.
struct WalkRow {
    float4 lo, hi, g0, g1;   // columns [t0, t0+4), [t0+4, t0+8) of the current eight, [t0+8, t0+16) of the next eight
    float own, nxt;          // the lane's own column, and the same column of the next block
};
__device__ __forceinline__ void walk_row_load(const float *__restrict__ tile, const int ld, const int r, const int lane,
                                              WalkRow &q)
{
    const float *row = tile + r * ld;
    const int t0 = r & ~7, t = r & 7;
    if (t < 3) q.lo = *reinterpret_cast<const float4 *>(row + t0);
    if (t < 7) q.hi = *reinterpret_cast<const float4 *>(row + t0 + 4);
    if (t0 < 24 && t >= 6) {
        q.g0 = *reinterpret_cast<const float4 *>(row + t0 + 8);
        q.g1 = *reinterpret_cast<const float4 *>(row + t0 + 12);
    }
    q.own = row[lane];
    q.nxt = row[32 + lane];
}
// dn is meaningful only when the tile has 32 further columns of the same rows (otherwise the
// loads read neighbouring shared memory and the caller ignores dn).
__device__ __forceinline__ uint32_t walk_block_warp(const float *__restrict__ tile, const int ld, float d, float &dn,
                                                    const int lane)
{
    using sm100::fma2;
    using sm100::pack2;
    using sm100::unpack2;
    uint32_t mask = 0;
    uint64_t X[4], XN[4];
    uint64_t DD = pack2(d, dn);
    WalkRow q[4];
    walk_row_load(tile, ld, 0, lane, q[0]);
    walk_row_load(tile, ld, 1, lane, q[1]);
    walk_row_load(tile, ld, 2, lane, q[2]);
#pragma unroll
    for (int j = 0; j < 4; ++j)
        X[j] = pack2(__shfl_sync(0xffffffffu, d, 2 * j), __shfl_sync(0xffffffffu, d, 2 * j + 1));
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const int t0 = r & ~7, t = r & 7;
        const bool more = t0 < 24;
        if (r + 3 < 32) walk_row_load(tile, ld, r + 3, lane, q[(r + 3) & 3]);
        if (t == 6 && more) {
            // the lanes' own scores hold every decision before pair t0 + 6
            float dcur, dnx;
            unpack2(DD, dcur, dnx);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                XN[j] = pack2(__shfl_sync(0xffffffffu, dcur, t0 + 8 + 2 * j), __shfl_sync(0xffffffffu, dcur, t0 + 9 + 2 * j));
        }
        const WalkRow &c = q[r & 3];
        float xlo, xhi;
        unpack2(X[t >> 1], xlo, xhi);
        const uint32_t xb = __float_as_uint((t & 1) ? xhi : xlo);
        const float s = __uint_as_float((~xb & 0x80000000u) | 0x3f800000u);   // swapped (negative) +1, kept -1
        const uint64_t S2 = pack2(s, s);
        mask = __funnelshift_l(xb, mask, 1);                         // decisions enter at bit 0, first one ends at bit 31
        const uint64_t F2[4] = {pack2(c.lo.x, c.lo.y), pack2(c.lo.z, c.lo.w), pack2(c.hi.x, c.hi.y), pack2(c.hi.z, c.hi.w)};
#pragma unroll
        for (int v = (t + 1) >> 1; v < 4; ++v) X[v] = fma2(S2, F2[v], X[v]);
        DD = fma2(S2, pack2(c.own, c.nxt), DD);
        if (more && t >= 6) {
            const uint64_t G2[4] = {pack2(c.g0.x, c.g0.y), pack2(c.g0.z, c.g0.w), pack2(c.g1.x, c.g1.y), pack2(c.g1.z, c.g1.w)};
#pragma unroll
            for (int j = 0; j < 4; ++j) XN[j] = fma2(S2, G2[j], XN[j]);
        }
        if (t == 7 && more) {
#pragma unroll
            for (int j = 0; j < 4; ++j) X[j] = XN[j];
        }
    }
    float dcur;
    unpack2(DD, dcur, dn);
    return __brev(mask);
}

// Thresholds a_u = b_u b_max,u (1/2 + ln(2s/delta)) of a 32-pair block in fp32, lane u = pair u.
// b_max,u = max(b_u, r_u b_max,u-1) is the composition of the maps x -> max(b_u, r_u x); a warp scan
// composes them in five steps ((m2, c2) o (m1, c1) = (max(m2, c2 m1), c2 c1)), which differs from
// the pair-by-pair recurrence only in the rounding of the products of decay factors.  `bmax` is
// b_max before the block on entry and after it on return (warp-uniform).
__device__ __forceinline__ float walk_block_thresholds(const float b, const float r, float &bmax, const float logfac,
                                                       const int lane)
{
    float m = b, c = r;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float mo = __shfl_up_sync(0xffffffffu, m, o), co = __shfl_up_sync(0xffffffffu, c, o);
        if (lane >= o) {
            m = fmaxf(m, c * mo);
            c = c * co;
        }
    }
    const float bm = fmaxf(m, c * bmax);
    bmax = __shfl_sync(0xffffffffu, bm, 31);
    return b * bm * logfac;
}
// d of the sign test: alpha - a (1 - 2U), or +-1 by U alone when a is zero (probability 1/2)
__device__ __forceinline__ float walk_sign_score(const float alpha, const float a, const float U)
{
    return (a > 0.f && isfinite(a)) ? alpha - a * (1.f - 2.f * U) : (U < 0.5f ? -1.f : 1.f);
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
