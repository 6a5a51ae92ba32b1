// Compress2 on a sequence of any length, sink and window rows kept exactly (elm_compress_ragged).
#include "elm_level.cuh"

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
