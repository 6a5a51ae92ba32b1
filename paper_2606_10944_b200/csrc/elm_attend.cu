// Weighted attention over a coreset, Eq. (def:att_approx):
//   O[j,:] = sum_c w_c exp(<q_j,k_c>/sqrt(d)) v_c / sum_c w_c exp(<q_j,k_c>/sqrt(d)).
// Stage gather copies the coreset rows of every attention problem into contiguous operands and
// turns the weights into a base-2 logit bias log2(w_c); stage attend is an online-softmax pass.
// This file holds the precision-generic SIMT kernel (fp64 mode and fp32 inputs); bf16 inputs in
// fp32 mode take the tensor-core kernel in elm_attend_tc.cu.
#include <math.h>

#include <cuda_fp8.h>

#include <mutex>
#include <type_traits>

#include "elm_attend.cuh"
#include "elm_common.cuh"

namespace elm {

// ---------------------------------------------------------------------------------------------
// Stage gather: Kc, Vc [problems][n_core][d] in the input dtype, bias [problems][n_core] in the arithmetic type
// (fp64 in the deterministic mode, so that the weights enter the logits at full precision there)
// ---------------------------------------------------------------------------------------------
// E4M3 bytes as the numbers they encode (every E4M3 value is a bf16 value)
__device__ __forceinline__ __nv_bfloat16 widen_e4m3(unsigned char b)
{
    const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)b, __NV_E4M3);
    return __float2bfloat16_rn(__half2float(__half(h)));
}
__device__ __forceinline__ float gather_elt(const float *p, int e) { return p[e]; }
__device__ __forceinline__ __nv_bfloat16 gather_elt(const __nv_bfloat16 *p, int e) { return p[e]; }
__device__ __forceinline__ __nv_bfloat16 gather_elt(const unsigned char *p, int e) { return widen_e4m3(p[e]); }

// [count] E4M3 bytes -> bf16, exactly
__global__ void __launch_bounds__(256) widen_e4m3_kernel(const unsigned char *__restrict__ src, __nv_bfloat16 *__restrict__ dst,
                                                        int64_t count)
{
    const int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 16;
    if (i + 16 <= count) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src + i));
        const unsigned char *b = reinterpret_cast<const unsigned char *>(&v);
        __align__(16) __nv_bfloat16 o[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) o[e] = widen_e4m3(b[e]);
        reinterpret_cast<uint4 *>(dst + i)[0] = reinterpret_cast<const uint4 *>(o)[0];
        reinterpret_cast<uint4 *>(dst + i)[1] = reinterpret_cast<const uint4 *>(o)[1];
    } else {
        for (int64_t e = i; e < count; ++e) dst[e] = widen_e4m3(src[e]);
    }
}
int widen_e4m3(const void *src, void *dst_bf16, int64_t count, cudaStream_t st)
{
    const int64_t blocks = (count + 4095) / 4096;
    widen_e4m3_kernel<<<(unsigned)blocks, 256, 0, st>>>((const unsigned char *)src, (__nv_bfloat16 *)dst_bf16, count);
    count_launches(1);
    return cuda_status(cudaGetLastError());
}

__device__ __forceinline__ float log2_as(float w, float) { return log2f(w); }
__device__ __forceinline__ double log2_as(float w, double) { return log2((double)w); }

template <typename Tin, typename Tsrc, typename Tb>
__global__ void __launch_bounds__(256) gather_kernel(const Tsrc *__restrict__ K,
                                                     const Tsrc *__restrict__ V,
                                                     const int32_t *__restrict__ idx,
                                                     const float *__restrict__ w, int64_t n, int d,
                                                     int n_core, Tin *__restrict__ Kc,
                                                     Tin *__restrict__ Vc, Tb *__restrict__ bias,
                                                     int *__restrict__ status)
{
    const int p = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = blockIdx.x * 8 + warp;
    if (c >= n_core) return;
    const int64_t row = checked_row(idx[(int64_t)p * n_core + c], n, status);
    const Tsrc *ks = K + ((int64_t)p * n + row) * d;
    const Tsrc *vs = V + ((int64_t)p * n + row) * d;
    Tin *kd = Kc + ((int64_t)p * n_core + c) * d;
    Tin *vd = Vc + ((int64_t)p * n_core + c) * d;
    for (int e = lane; e < d; e += 32) {
        kd[e] = gather_elt(ks, e);
        vd[e] = gather_elt(vs, e);
    }
    if (lane == 0) bias[(int64_t)p * n_core + c] = log2_as(w[(int64_t)p * n_core + c], Tb());
}

// ---------------------------------------------------------------------------------------------
// Stage attend (SIMT): one CTA = 64 queries of one head; coreset streamed in chunks of 32 points.
// Logits are kept in base 2: s = <q,k> * log2(e)/sqrt(d) + log2(w).
// ---------------------------------------------------------------------------------------------
template <typename Tin, typename T, int D>
__global__ void __launch_bounds__(128) attend_simt_kernel(const Tin *__restrict__ Q,
                                                          const Tin *__restrict__ Kc,
                                                          const Tin *__restrict__ Vc,
                                                          const T *__restrict__ bias,
                                                          Tin *__restrict__ O, int q_heads,
                                                          int kv_heads, int64_t n_q, int n_core,
                                                          int64_t q_row0, int64_t n_q_total, int tail_start,
                                                          const int32_t *__restrict__ birth,
                                                          const int32_t *__restrict__ death, int n_pad,
                                                          float *__restrict__ lse)
{
    constexpr int BM = 64, BN = 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *Qt = reinterpret_cast<T *>(smem_raw);        // [D][BM]   transposed query tile
    T *Kt = Qt + D * BM;                            // [D][BN]   transposed key chunk
    T *Vs = Kt + D * BN;                            // [BN][D]
    T *S = Vs + BN * D;                             // [BM][BN+1] logits, then probabilities
    T *rowscale = S + BM * (BN + 1);                // [BM] factor applied to the old accumulator
    T *rowsum = rowscale + BM;                      // [BM] running denominator
    T *rowmax = rowsum + BM;                        // [BM] running maximum
    T *sbias = rowmax + BM;                         // [BN]
    int32_t *sbirth = reinterpret_cast<int32_t *>(sbias + BN);   // [BN] lifetimes of the chunk's entries
    int32_t *sdeath = sbirth + BN;                               // [BN]

    const int tid = threadIdx.x;
    const int bh = blockIdx.y;                      // batch * q_heads + head
    const int b = bh / q_heads, h = bh % q_heads;
    const int64_t prob = (int64_t)b * kv_heads + ((int64_t)h * kv_heads) / q_heads;
    const int64_t q0 = (int64_t)blockIdx.x * BM;
    const Tin *Qp = Q + ((int64_t)bh * n_q_total + q_row0) * D;
    const Tin *Kp = Kc + prob * n_core * D;
    const Tin *Vp = Vc + prob * n_core * D;
    const T *bp = bias + prob * n_core;
    const T scale = (T)(1.4426950408889634 / sqrt((double)D));

    for (int e = tid; e < BM * D; e += 128) {
        int r = e / D, k = e % D;
        Qt[k * BM + r] = (q0 + r < n_q) ? load_as<T>(Qp, (q0 + r) * D + k) : (T)0;
    }
    if (tid < BM) { rowsum[tid] = 0; rowmax[tid] = -INFINITY; }

    const int ty = tid >> 3, tx = tid & 7;          // S tile: rows 4ty.., cols 4tx..
    constexpr int OC = D / 8;                       // output columns per thread
    T acc[4][OC];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < OC; ++c) acc[r][c] = 0;

    for (int c0 = 0; c0 < n_core; c0 += BN) {
        __syncthreads();
        for (int e = tid; e < BN * D; e += 128) {
            int c = e / D, k = e % D;
            bool ok = c0 + c < n_core;
            Kt[k * BN + c] = ok ? load_as<T>(Kp, (int64_t)(c0 + c) * D + k) : (T)0;
            Vs[c * D + k] = ok ? load_as<T>(Vp, (int64_t)(c0 + c) * D + k) : (T)0;
        }
        if (tid < BN) {
            sbias[tid] = (c0 + tid < n_core) ? (T)bp[c0 + tid] : (T)0;
            if (birth) {
                sbirth[tid] = (c0 + tid < n_core) ? birth[prob * n_pad + c0 + tid] : 0x7fffffff;
                sdeath[tid] = (c0 + tid < n_core) ? death[prob * n_pad + c0 + tid] : 0x7fffffff;
            }
        }
        __syncthreads();
        T s[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) s[r][c] = 0;
        for (int k = 0; k < D; ++k) {
            T qv[4], kv[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) { qv[r] = Qt[k * BM + 4 * ty + r]; kv[r] = Kt[k * BN + 4 * tx + r]; }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) s[r][c] += qv[r] * kv[c];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int col = 4 * tx + c;
                // a row sees the entries alive at its own position, or (tail rule) the list up to its own
                // entry of the causal tail
                const int64_t trow = q_row0 + q0 + 4 * ty + r;
                const bool seen = c0 + col < n_core &&
                                  (birth ? (sbirth[col] <= trow && trow < sdeath[col])
                                         : (int64_t)(c0 + col) <= (int64_t)tail_start + q0 + 4 * ty + r);
                S[(4 * ty + r) * (BN + 1) + col] = seen ? s[r][c] * scale + sbias[col] : (T)-INFINITY;
            }
        __syncthreads();
        if (tid < BM) {
            T *row = S + tid * (BN + 1);
            T mx = rowmax[tid];
            for (int c = 0; c < BN; ++c) mx = row[c] > mx ? row[c] : mx;
            T f = (rowmax[tid] == -INFINITY) ? (T)0 : (T)exp2((T)(rowmax[tid] - mx));
            T sum = 0;
            for (int c = 0; c < BN; ++c) {
                T pr = (row[c] == -INFINITY) ? (T)0 : (T)exp2((T)(row[c] - mx));
                row[c] = pr;
                sum += pr;
            }
            rowscale[tid] = f;
            rowsum[tid] = rowsum[tid] * f + sum;
            rowmax[tid] = mx;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            T f = rowscale[4 * ty + r];
#pragma unroll
            for (int c = 0; c < OC; ++c) acc[r][c] *= f;
        }
        for (int c = 0; c < BN; ++c) {
            T pr[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) pr[r] = S[(4 * ty + r) * (BN + 1) + c];
#pragma unroll
            for (int o = 0; o < OC; ++o) {
                T v = Vs[c * D + tx + 8 * o];
#pragma unroll
                for (int r = 0; r < 4; ++r) acc[r][o] += pr[r] * v;
            }
        }
    }
    Tin *Op = O + ((int64_t)bh * n_q_total + q_row0) * D;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        int64_t q = q0 + 4 * ty + r;
        if (q >= n_q) continue;
        T inv = (T)1 / rowsum[4 * ty + r];
#pragma unroll
        for (int o = 0; o < OC; ++o) store_from(Op, q * D + tx + 8 * o, acc[r][o] * inv);
        if (lse && tx == 0) lse[(int64_t)bh * n_q_total + q_row0 + q] = (float)(rowmax[4 * ty + r] + log2(rowsum[4 * ty + r]));
    }
}

AttendLayout attend_layout(const elm_params *p, int32_t n_core)
{
    AttendLayout L;
    const size_t problems = (size_t)p->batch * p->kv_heads;
    const size_t es = elt_bytes(p->dtype);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t n_pad = ((size_t)n_core + 127) / 128 * 128;      // the tensor-core path pads to its block size
    // E4M3 inputs: the gathered rows are kept as bf16 (exact), except the keys of the fp32-mode tensor-core path
    const size_t ges = p->dtype == ELM_E4M3 ? 2 : es;
    L.Kc = take(problems * n_pad * p->d * ges);
    L.Vc = take(problems * n_pad * p->d * ges);
    L.bias = take(problems * n_pad * 8);
    L.bx = take(problems * n_pad * 32);
    L.flags = take((problems + 1) * 4);
    L.qwide = take(p->dtype == ELM_E4M3 && p->precision == ELM_PREC_FP64_DET
                       ? (size_t)p->batch * p->q_heads * p->n_q * p->d * 2 : 0);
    L.total = off;
    return L;
}

template <typename Tin, typename T, int D>
static int launch_attend_simt(const Tin *Q, const Tin *Kc, const Tin *Vc, const T *bias, Tin *O,
                              const elm_params *p, int n_core, cudaStream_t st, const AttendWindow &win = AttendWindow())
{
    constexpr int BM = 64, BN = 32;
    const size_t smem = sizeof(T) * (size_t)(D * BM + D * BN + BN * D + BM * (BN + 1) + 3 * BM + BN) + 2 * BN * sizeof(int32_t);
    auto kern = attend_simt_kernel<Tin, T, D>;
    ELM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((unsigned)((p->n_q + BM - 1) / BM), (unsigned)(p->batch * p->q_heads));
    kern<<<grid, 128, smem, st>>>(Q, Kc, Vc, bias, O, p->q_heads, p->kv_heads, p->n_q, n_core, win.q_row0,
                                  win.n_q_total ? win.n_q_total : (int64_t)p->n_q, win.tail_start, win.birth, win.death,
                                  (n_core + 127) / 128 * 128, win.lse);
    count_launches(1);
    return cuda_status(cudaGetLastError());
}

// Tsrc: the type K and V are stored in (E4M3 bytes are widened by the gather; Q then is the widened copy)
template <typename Tin, typename T, typename Tsrc = Tin>
static int attend_impl(const Tin *Q, const Tsrc *K, const Tsrc *V, const int32_t *idx, const float *w,
                       int n_core, const elm_params *p, Tin *O, unsigned char *ws, cudaStream_t st, const AttendWindow &win)
{
    if constexpr (std::is_same<Tsrc, __nv_bfloat16>::value && std::is_same<T, float>::value)
        return attend_tc(Q, K, V, idx, w, n_core, p, O, ws, st, true, win);
    const AttendLayout L = attend_layout(p, n_core);
    Tin *Kc = reinterpret_cast<Tin *>(ws + L.Kc);
    Tin *Vc = reinterpret_cast<Tin *>(ws + L.Vc);
    T *bias = reinterpret_cast<T *>(ws + L.bias);
    const int problems = p->batch * p->kv_heads;
    {
        StageTimer t(ELM_STAGE_GATHER, st, 1);
        // this path has no bounded waits: its status word reads 0
        ELM_CUDA_TRY(cudaMemsetAsync(ws + L.flags, 0, sizeof(int) * (size_t)(problems + 1), st));
        gather_kernel<Tin, Tsrc, T><<<dim3((unsigned)((n_core + 7) / 8), (unsigned)problems), 256, 0, st>>>(
            K, V, idx, w, p->n_kv, p->d, n_core, Kc, Vc, bias, reinterpret_cast<int *>(ws + L.flags) + problems);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    StageTimer t(ELM_STAGE_ATTEND, st, 1);
    if (p->d == 64) return launch_attend_simt<Tin, T, 64>(Q, Kc, Vc, bias, O, p, n_core, st, win);
    return launch_attend_simt<Tin, T, 128>(Q, Kc, Vc, bias, O, p, n_core, st, win);
}


// ---------------------------------------------------------------------------------------------
// Built-in scratch for elm_attend_static.  The array lives in every GPU that loads this library
// until the process exits.  Its name is only a host-side handle: the device address is looked
// up once per device with cudaGetSymbolAddress and that address is what the kernels receive.
// ---------------------------------------------------------------------------------------------
}  // namespace elm

static __device__ __align__(256) unsigned char g_attend_static_scratch[ELM_ATTEND_STATIC_SCRATCH_BYTES];

namespace elm {

static std::mutex g_static_mutex;
static unsigned char *g_static_addr[64];    // device address of the array, per device ordinal

static int static_scratch_address(unsigned char **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return ELM_ERR_UNAVAILABLE;
    if (dev < 0 || dev >= 64) return ELM_ERR_UNAVAILABLE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void *addr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&addr, g_attend_static_scratch);
        if (e != cudaSuccess || addr == nullptr) return ELM_ERR_CUDA;
        g_static_addr[dev] = static_cast<unsigned char *>(addr);
    }
    *out = g_static_addr[dev];
    return ELM_OK;
}

// Same two launches as attend_impl, without the event-based stage timers (creating an event may
// allocate) and with the gathered operands placed in `scratch`.
template <typename Tin, typename T>
static int attend_enqueue_untimed(const Tin *Q, const Tin *K, const Tin *V, const int32_t *idx,
                                  const float *w, int n_core, const elm_params *p, Tin *O,
                                  unsigned char *scratch, cudaStream_t st)
{
    if constexpr (std::is_same<Tin, __nv_bfloat16>::value && std::is_same<T, float>::value)
        return attend_tc(Q, K, V, idx, w, n_core, p, O, scratch, st, false);
    const AttendLayout L = attend_layout(p, n_core);
    Tin *Kc = reinterpret_cast<Tin *>(scratch + L.Kc);
    Tin *Vc = reinterpret_cast<Tin *>(scratch + L.Vc);
    T *bias = reinterpret_cast<T *>(scratch + L.bias);
    const int problems = p->batch * p->kv_heads;
    // this path has no bounded waits: its status word reads 0
    ELM_CUDA_TRY(cudaMemsetAsync(scratch + L.flags, 0, sizeof(int) * (size_t)(problems + 1), st));
    gather_kernel<Tin, Tin, T><<<dim3((unsigned)((n_core + 7) / 8), (unsigned)problems), 256, 0, st>>>(
        K, V, idx, w, p->n_kv, p->d, n_core, Kc, Vc, bias, reinterpret_cast<int *>(scratch + L.flags) + problems);
    count_launches(1);
    ELM_CUDA_TRY(cudaGetLastError());
    if (p->d == 64) return launch_attend_simt<Tin, T, 64>(Q, Kc, Vc, bias, O, p, n_core, st);
    return launch_attend_simt<Tin, T, 128>(Q, Kc, Vc, bias, O, p, n_core, st);
}

}  // namespace elm

namespace elm {
// elm_attend after argument validation
int attend_enqueue(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w, int32_t n_core,
                   const elm_params *params, void *O, void *workspace, cudaStream_t st, const AttendWindow &win)
{
    unsigned char *ws = (unsigned char *)workspace;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    const bool whole = win.q_row0 == 0 && win.n_q_total == 0 && win.tail_start == 0x7fffffff && !win.birth && !win.lse;
    if (params->dtype == ELM_E4M3) {
        typedef __nv_bfloat16 bf;
        if (!whole) return ELM_ERR_DTYPE;                      // no windows or lifetimes on 8-bit inputs
        if (!det) return attend_tc_e4m3((const unsigned char *)Q, (const unsigned char *)K, (const unsigned char *)V, idx, w, n_core,
                                        params, (bf *)O, ws, st, true);
        // fp64 mode: the queries are widened into the workspace, the coreset rows by the gather
        bf *Qw = reinterpret_cast<bf *>(ws + attend_layout(params, n_core).qwide);
        const int rc = widen_e4m3(Q, Qw, (int64_t)params->batch * params->q_heads * params->n_q * params->d, st);
        if (rc != ELM_OK) return rc;
        return attend_impl<bf, double, unsigned char>(Qw, (const unsigned char *)K, (const unsigned char *)V, idx, w, n_core, params,
                                                      (bf *)O, ws, st, win);
    }
    if (whole && attend_decode_applies(params)) return attend_decode(Q, K, V, idx, w, n_core, params, O, ws, st, true);
    if (params->dtype == ELM_F32) {
        return det ? attend_impl<float, double>((const float *)Q, (const float *)K, (const float *)V, idx, w, n_core, params, (float *)O, ws, st, win)
                   : attend_impl<float, float>((const float *)Q, (const float *)K, (const float *)V, idx, w, n_core, params, (float *)O, ws, st, win);
    }
    typedef __nv_bfloat16 bf;
    return det ? attend_impl<bf, double>((const bf *)Q, (const bf *)K, (const bf *)V, idx, w, n_core, params, (bf *)O, ws, st, win)
               : attend_impl<bf, float>((const bf *)Q, (const bf *)K, (const bf *)V, idx, w, n_core, params, (bf *)O, ws, st, win);
}
}  // namespace elm

extern "C" int elm_attend_workspace_bytes(const elm_params *params, int32_t n_core, size_t *bytes)
{
    using namespace elm;
    if (!params || !bytes) return ELM_ERR_NULL;
    int rc = validate_attend_params(params, true);
    if (rc != ELM_OK) return rc;
    if (n_core < 1 || n_core > params->n_kv) return ELM_ERR_SHAPE;
    *bytes = attend_layout(params, n_core).total;
    return ELM_OK;
}

extern "C" int elm_attend(const void *Q, const void *K, const void *V, const int32_t *idx,
                          const float *w, int32_t n_core, const elm_params *params, void *O,
                          void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    int rc = validate_attend_params(params, true);
    if (rc != ELM_OK) return rc;
    if (!Q || !K || !V || !idx || !w || !O || !workspace) return ELM_ERR_NULL;
    if (n_core < 1 || n_core > params->n_kv) return ELM_ERR_SHAPE;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)idx | (uintptr_t)w | (uintptr_t)O) & 15)
        return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < attend_layout(params, n_core).total) return ELM_ERR_WORKSPACE;
    return attend_enqueue(Q, K, V, idx, w, n_core, params, O, workspace, (cudaStream_t)stream);
}

extern "C" int elm_attend_static(const void *Q, const void *K, const void *V, const int32_t *idx,
                                 const float *w, int32_t n_core, const elm_params *params, void *O,
                                 void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    int rc = validate_attend_params(params);
    if (rc != ELM_OK) return rc;
    if (!Q || !K || !V || !idx || !w || !O) return ELM_ERR_NULL;
    if (n_core < 1 || n_core > params->n_kv) return ELM_ERR_SHAPE;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)idx | (uintptr_t)w | (uintptr_t)O) & 15)
        return ELM_ERR_ALIGN;
    if (attend_layout(params, n_core).total > (size_t)ELM_ATTEND_STATIC_SCRATCH_BYTES) return ELM_ERR_STATIC_LIMIT;
    unsigned char *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != ELM_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    if (attend_decode_applies(params)) return attend_decode(Q, K, V, idx, w, n_core, params, O, scratch, st, false);
    if (params->dtype == ELM_F32) {
        return det ? attend_enqueue_untimed<float, double>((const float *)Q, (const float *)K, (const float *)V, idx, w, n_core, params, (float *)O, scratch, st)
                   : attend_enqueue_untimed<float, float>((const float *)Q, (const float *)K, (const float *)V, idx, w, n_core, params, (float *)O, scratch, st);
    }
    typedef __nv_bfloat16 bf;
    return det ? attend_enqueue_untimed<bf, double>((const bf *)Q, (const bf *)K, (const bf *)V, idx, w, n_core, params, (bf *)O, scratch, st)
               : attend_enqueue_untimed<bf, float>((const bf *)Q, (const bf *)K, (const bf *)V, idx, w, n_core, params, (bf *)O, scratch, st);
}

extern "C" int elm_attend_static_status(const elm_params *params, int32_t n_core, int32_t *status_host, void *stream)
{
    using namespace elm;
    if (!params || !status_host) return ELM_ERR_NULL;
    int rc = validate_attend_params(params);
    if (rc != ELM_OK) return rc;
    if (n_core < 1 || n_core > params->n_kv) return ELM_ERR_SHAPE;
    const AttendLayout L = attend_layout(params, n_core);
    if (L.total > (size_t)ELM_ATTEND_STATIC_SCRATCH_BYTES) return ELM_ERR_STATIC_LIMIT;
    unsigned char *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != ELM_OK) return rc;
    // the status word follows the per-problem "weights differ" flags, as in a caller's workspace
    const unsigned char *word = scratch + L.flags + 4 * (size_t)params->batch * params->kv_heads;
    ELM_CUDA_TRY(cudaMemcpyAsync(status_host, word, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    ELM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return ELM_OK;
}
