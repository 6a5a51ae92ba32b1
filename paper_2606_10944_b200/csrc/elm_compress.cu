// elm_compress: Offline-Compress2 (Algorithm 2 unrolled level by level) on the level machinery of elm_level.cuh.
#include "elm_level.cuh"

namespace elm {

// workspace layout of elm_compress
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
        ELM_CUDA_TRY(launch_after(prepass_kernel<Tin, T>, grid, dim3(256), 0, st, K, V, n, p->d, c.cnorm, c.vmax_bits, cur, (int64_t)0, (int64_t)-1));
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
        ELM_CUDA_TRY(launch_after(emit_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, w_out, idx_out, total, n_out, m == 0));
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
