// Weighted attention over a coreset for a few queries per head (decode: one new token, or a handful):
//   O[j,:] = sum_c w_c exp(<q_j,k_c>/sqrt(d)) v_c / sum_c w_c exp(<q_j,k_c>/sqrt(d))      Eq. (def:att_approx)
// With so few queries the work is reading each coreset row of K and V once: HBM-bound, and far too
// small for the tile kernels.  The list of an attention problem is split over `splits` CTAs; all
// query heads that share the KV head (and all their query rows: G vectors in total, G <= 8) are
// processed together, so a row is read once for the whole group.  Rows are read through the index
// list straight from K and V (no gathered copy).  A warp takes one list entry at a time, a lane owns
// D/32 consecutive dimensions: the dot products are finished with warp shuffles, the softmax is kept
// online per query (running maximum, denominator, accumulator), the warps of a CTA and then the
// CTAs of a problem are combined through the usual (max, denominator, accumulator) merge.
// fp32 arithmetic on fp32 or bf16 inputs.
#include <math.h>

#include "elm_attend.cuh"
#include "elm_common.cuh"

namespace elm {
namespace {

constexpr int DEC_WARPS = 8;
constexpr int DEC_GMAX = 8;
constexpr int DEC_UNR = 4;             // list entries a warp has in flight

template <int DPL> __device__ __forceinline__ void load_dims(const float *p, float (&x)[DPL])
{
    if constexpr (DPL == 4) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
        const float2 v = __ldg(reinterpret_cast<const float2 *>(p));
        x[0] = v.x; x[1] = v.y;
    }
}
template <int DPL> __device__ __forceinline__ void load_dims(const __nv_bfloat16 *p, float (&x)[DPL])
{
    if constexpr (DPL == 4) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(p));
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    } else {
        const uint32_t v = __ldg(reinterpret_cast<const uint32_t *>(p));
        x[0] = __uint_as_float(v << 16); x[1] = __uint_as_float(v & 0xffff0000u);
    }
}

// partial results: part[problem][split][g][D + 2] = accumulator (D), running maximum, denominator
template <typename Tin, int D, int G>
__global__ void __launch_bounds__(DEC_WARPS * 32)
decode_partial_kernel(const Tin *__restrict__ Q, const Tin *__restrict__ K, const Tin *__restrict__ V,
                      const int32_t *__restrict__ idx, const float *__restrict__ w, int64_t n, int n_core, int q_heads,
                      int kv_heads, int n_q, int groups /* live query vectors <= G */, int chunk, float *__restrict__ part,
                      int *__restrict__ status)
{
    constexpr int DPL = D / 32;
    __shared__ float sm_o[DEC_WARPS][G][D];
    __shared__ float sm_ml[DEC_WARPS][G][2];
    // (launched with programmatic stream serialization: resident before the kernel in front of it has finished;
    // nothing is read before this point)
    cudaGridDependencySynchronize();
    const int prob = blockIdx.y, split = blockIdx.x, splits = gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = prob / kv_heads, kvh = prob % kv_heads, rep = q_heads / kv_heads;
    const float scale = 1.4426950408889634f / sqrtf((float)D);

    // query vector g = (head within the group) * n_q + row
    float q[G][DPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) q[g][i] = 0.f;
        if (g < groups) {
            const int h = kvh * rep + g / n_q, r = g % n_q;
            load_dims<DPL>(Q + (((int64_t)b * q_heads + h) * n_q + r) * D + lane * DPL, q[g]);
#pragma unroll
            for (int i = 0; i < DPL; ++i) q[g][i] *= scale;
        }
    }
    float m[G], l[G], o[G][DPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[g][i] = 0.f;
    }
    const int c0 = split * chunk, c1 = c0 + chunk < n_core ? c0 + chunk : n_core;
    const int32_t *ip = idx + (int64_t)prob * n_core;
    const float *wp = w + (int64_t)prob * n_core;
    const Tin *Kp = K + (int64_t)prob * n * D, *Vp = V + (int64_t)prob * n * D;
    // DEC_UNR entries per warp at a time: their row numbers, then all their K and V rows are requested
    // before the first one is used, so that several rows per warp are in flight (the kernel has
    // nothing to hide the memory latency with but its own loads)
    int32_t myrow = 0;
    float mylw = 0.f;
    auto fetch_entries = [&](int e0) {                                   // lane j < DEC_UNR: entry e0 + j
        myrow = 0;
        mylw = 0.f;
        if (lane < DEC_UNR && e0 + lane < c1) {
            myrow = (int32_t)checked_row(__ldg(ip + e0 + lane), n, status);
            mylw = log2f(__ldg(wp + e0 + lane));
        }
    };
    fetch_entries(c0 + warp * DEC_UNR);
    for (int e0 = c0 + warp * DEC_UNR; e0 < c1; e0 += DEC_WARPS * DEC_UNR) {
        float k[DEC_UNR][DPL], v[DEC_UNR][DPL], lw[DEC_UNR];
#pragma unroll
        for (int j = 0; j < DEC_UNR; ++j) {
            const int64_t row = __shfl_sync(0xffffffffu, myrow, j);
            lw[j] = __shfl_sync(0xffffffffu, mylw, j);
            load_dims<DPL>(Kp + row * D + lane * DPL, k[j]);            // (row 0 for entries past the end: unused)
            load_dims<DPL>(Vp + row * D + lane * DPL, v[j]);
        }
        fetch_entries(e0 + DEC_WARPS * DEC_UNR);                         // the next batch's row numbers, behind the rows
#pragma unroll
        for (int j = 0; j < DEC_UNR; ++j) {
            if (e0 + j >= c1) break;
            float s[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float a = 0.f;
#pragma unroll
                for (int i = 0; i < DPL; ++i) a = fmaf(q[g][i], k[j][i], a);
                s[g] = a;
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1)
#pragma unroll
                for (int g = 0; g < G; ++g) s[g] += __shfl_xor_sync(0xffffffffu, s[g], off);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float sg = s[g] + lw[j];                               // base-2 logit
                const float mn = fmaxf(m[g], sg);
                const float a = exp2f(m[g] - mn), pw = exp2f(sg - mn);       // exp2f(-inf) = 0 on the first entry
                l[g] = l[g] * a + pw;
#pragma unroll
                for (int i = 0; i < DPL; ++i) o[g][i] = o[g][i] * a + pw * v[j][i];
                m[g] = mn;
            }
        }
    }
    // combine the warps of the CTA
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) sm_o[warp][g][lane * DPL + i] = o[g][i];
        if (lane == 0) { sm_ml[warp][g][0] = m[g]; sm_ml[warp][g][1] = l[g]; }
    }
    __syncthreads();
    float *out = part + (((int64_t)prob * splits + split) * G) * (D + 2);
    for (int t = threadIdx.x; t < G * D; t += DEC_WARPS * 32) {
        const int g = t / D, d = t % D;
        float M = -INFINITY;
#pragma unroll
        for (int wv = 0; wv < DEC_WARPS; ++wv) M = fmaxf(M, sm_ml[wv][g][0]);
        float acc = 0.f, den = 0.f;
#pragma unroll
        for (int wv = 0; wv < DEC_WARPS; ++wv) {
            const float mw = sm_ml[wv][g][0];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
            acc += f * sm_o[wv][g][d];
            den += f * sm_ml[wv][g][1];
        }
        out[g * (D + 2) + d] = acc;
        if (d == 0) { out[g * (D + 2) + D] = M; out[g * (D + 2) + D + 1] = den; }
    }
}

// One CTA per (problem, query vector), one thread per dimension.  The splits' maxima and denominators are read
// by one thread each and combined through shared memory, and the accumulators with several loads in flight: the
// kernel is a chain of memory round trips and nothing else, so it is laid out to make that chain three long
// whatever the number of splits (a loop over the splits with one load per turn took 13 us for 37 splits).
constexpr int DEC_MAX_SPLITS = 256;
template <typename Tin, int D, int G>
__global__ void __launch_bounds__(D) decode_merge_kernel(const float *__restrict__ part, int splits, int q_heads, int kv_heads,
                                                         int n_q, Tin *__restrict__ O, int *__restrict__ status)
{
    __shared__ float sf[DEC_MAX_SPLITS];
    __shared__ float red[2][D / 32];
    const int prob = blockIdx.y, g = blockIdx.x, d = threadIdx.x;
    const int warp = d >> 5, lane = d & 31;
#ifndef ELM_BOUNDS_CHECK
    // this path has no bounded waits and (in this build) no row checks: its status word reads 0 - written here
    // rather than by a memset of its own, which would be a third of a decode step's launches
    if (prob == 0 && g == 0 && d == 0) *status = 0;
#endif
    const int b = prob / kv_heads, kvh = prob % kv_heads, rep = q_heads / kv_heads;
    const float *p = part + ((int64_t)prob * splits * G + g) * (D + 2);
    // launched with programmatic stream serialization: the CTAs of this kernel are resident while the partial
    // kernel still runs and wait here for its results, so the gap between the two launches is not on the path
    cudaGridDependencySynchronize();
    // thread s (and s + D, ...) fetches split s's maximum and denominator
    float M = -INFINITY;
    float ms[(DEC_MAX_SPLITS + D - 1) / D], ls[(DEC_MAX_SPLITS + D - 1) / D];
#pragma unroll
    for (int i = 0; i < (DEC_MAX_SPLITS + D - 1) / D; ++i) {
        const int sp = d + i * D;
        ms[i] = -INFINITY;
        ls[i] = 0.f;
        if (sp < splits) {
            ms[i] = __ldg(p + (int64_t)sp * G * (D + 2) + D);
            ls[i] = __ldg(p + (int64_t)sp * G * (D + 2) + D + 1);
        }
        M = fmaxf(M, ms[i]);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    if (lane == 0) red[0][warp] = M;
    __syncthreads();
    M = red[0][0];
#pragma unroll
    for (int i = 1; i < D / 32; ++i) M = fmaxf(M, red[0][i]);
    float den = 0.f;
#pragma unroll
    for (int i = 0; i < (DEC_MAX_SPLITS + D - 1) / D; ++i) {
        const int sp = d + i * D;
        if (sp < splits) {
            const float f = ms[i] == -INFINITY ? 0.f : exp2f(ms[i] - M);
            sf[sp] = f;
            den += f * ls[i];
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
    if (lane == 0) red[1][warp] = den;
    __syncthreads();
    den = 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) den += red[1][i];
    float acc = 0.f;
    int s0 = 0;
    for (; s0 + 8 <= splits; s0 += 8) {
        float x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = __ldg(p + (int64_t)(s0 + j) * G * (D + 2) + d);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc = fmaf(sf[s0 + j], x[j], acc);
    }
    for (; s0 < splits; ++s0) acc = fmaf(sf[s0], __ldg(p + (int64_t)s0 * G * (D + 2) + d), acc);
    const int h = kvh * rep + g / n_q, r = g % n_q;
    store_from(O, (((int64_t)b * q_heads + h) * n_q + r) * D + d, acc / den);
}

template <typename Tin, int D, int G>
int launch_decode(const Tin *Q, const Tin *K, const Tin *V, const int32_t *idx, const float *w, int n_core,
                  const elm_params *p, Tin *O, float *part, int *status, int splits, int groups, cudaStream_t st)
{
    const int problems = p->batch * p->kv_heads;
    const int chunk = (n_core + splits - 1) / splits;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)splits, (unsigned)problems);
        cfg.blockDim = dim3(DEC_WARPS * 32);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int64_t n_kv = p->n_kv;
        int q_heads = p->q_heads, kv_heads = p->kv_heads, n_q = p->n_q;
        ELM_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_partial_kernel<Tin, D, G>, Q, K, V, idx, w, n_kv, n_core, q_heads, kv_heads,
                                        n_q, groups, chunk, part, status));
    }
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)groups, (unsigned)problems);
        cfg.blockDim = dim3(D);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const float *part_c = part;
        int q_heads = p->q_heads, kv_heads = p->kv_heads, n_q = p->n_q;
        ELM_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_merge_kernel<Tin, D, G>, part_c, splits, q_heads, kv_heads, n_q, O, status));
    }
    count_launches(2);
    return cuda_status(cudaGetLastError());
}

template <typename Tin, int D>
int dispatch_decode(const Tin *Q, const Tin *K, const Tin *V, const int32_t *idx, const float *w, int n_core,
                    const elm_params *p, Tin *O, float *part, int *status, int splits, int groups, cudaStream_t st)
{
    if (groups <= 1) return launch_decode<Tin, D, 1>(Q, K, V, idx, w, n_core, p, O, part, status, splits, groups, st);
    if (groups <= 2) return launch_decode<Tin, D, 2>(Q, K, V, idx, w, n_core, p, O, part, status, splits, groups, st);
    if (groups <= 4) return launch_decode<Tin, D, 4>(Q, K, V, idx, w, n_core, p, O, part, status, splits, groups, st);
    return launch_decode<Tin, D, 8>(Q, K, V, idx, w, n_core, p, O, part, status, splits, groups, st);
}

}  // namespace

bool attend_decode_applies(const elm_params *p)
{
    if (p->precision != ELM_PREC_FP32) return false;
    const int64_t groups = (int64_t)(p->q_heads / p->kv_heads) * p->n_q;
    return groups <= DEC_GMAX;
}

int attend_decode(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w, int n_core,
                  const elm_params *p, void *O, unsigned char *ws, cudaStream_t st, bool timed)
{
    const AttendLayout L = attend_layout(p, n_core);
    const int problems = p->batch * p->kv_heads;
    const int groups = (p->q_heads / p->kv_heads) * p->n_q;
    const int G = groups <= 1 ? 1 : groups <= 2 ? 2 : groups <= 4 ? 4 : 8;
    // the partial results live where the other paths keep their gathered operands
    const size_t room = L.bias - L.Kc;
    const size_t per_split = (size_t)problems * G * (p->d + 2) * sizeof(float);
    // enough CTAs for about two per SM, but at least one batch of entries per warp
    const int sm_count = device_sm_count();
    int splits = (n_core + DEC_WARPS * DEC_UNR - 1) / (DEC_WARPS * DEC_UNR);
    // (3, 4, 6, 8 per SM were measured: 27 / 24 / 24 / 24 us at 2048 entries and 52 / 49 / 53 / 58 us at 12288 against 22 / 43)
    const int wanted = (2 * sm_count + problems - 1) / problems;
    if (splits > wanted) splits = wanted;
    const int most = (int)(room / per_split);
    if (splits > most) splits = most;
    if (splits > 256) splits = 256;
    if (splits < 1) return ELM_ERR_WORKSPACE;
    float *part = reinterpret_cast<float *>(ws + L.Kc);
    int *status = reinterpret_cast<int *>(ws + L.flags) + problems;
    StageTimer t(timed ? ELM_STAGE_ATTEND : -1, st, 2);
#ifdef ELM_BOUNDS_CHECK
    // the partial kernel reports bad row numbers through the status word
    ELM_CUDA_TRY(cudaMemsetAsync(ws + L.flags, 0, sizeof(int) * (size_t)(problems + 1), st));
#endif
    if (p->dtype == ELM_F32) {
        const float *q = (const float *)Q, *k = (const float *)K, *v = (const float *)V;
        return p->d == 64 ? dispatch_decode<float, 64>(q, k, v, idx, w, n_core, p, (float *)O, part, status, splits, groups, st)
                          : dispatch_decode<float, 128>(q, k, v, idx, w, n_core, p, (float *)O, part, status, splits, groups, st);
    }
    typedef __nv_bfloat16 bf;
    const bf *q = (const bf *)Q, *k = (const bf *)K, *v = (const bf *)V;
    return p->d == 64 ? dispatch_decode<bf, 64>(q, k, v, idx, w, n_core, p, (bf *)O, part, status, splits, groups, st)
                      : dispatch_decode<bf, 128>(q, k, v, idx, w, n_core, p, (bf *)O, part, status, splits, groups, st);
}

}  // namespace elm
