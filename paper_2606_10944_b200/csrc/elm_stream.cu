// Streaming Thinformer Express: one token of every head per step (elm_stream_*).
#include "elm_level.cuh"

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
// build_list_kernel and, in the same launch, list[p][pos] = value for every problem p: the token's own entry into E
// or S_0 (Express.update), which lies behind the entries the pieces read.  A decode step is a handful of
// microsecond-sized launches, so each one saved shows.
__global__ void build_list_append_kernel(ListPieces pc, int64_t src_stride, int32_t *__restrict__ idx, float *__restrict__ w,
                                         int64_t cap, int32_t *__restrict__ list, int64_t pos, int32_t value)
{
    // (launched with programmatic stream serialization; nothing is read or written before this point)
    cudaGridDependencySynchronize();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t pr = blockIdx.y;
    if (i == 0) list[pr * src_stride + pos] = value;
    if (i >= pc.dst_off[pc.n]) return;
    int k = 0;
    while (i >= pc.dst_off[k + 1]) ++k;
    const int64_t o = i - pc.dst_off[k];
    idx[pr * cap + i] = pc.src[k] ? pc.src[k][pr * src_stride + pc.src_off[k] + o] : (int32_t)(pc.src_off[k] + o);
    w[pr * cap + i] = pc.w[k];
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
    bool appended = false;
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
        } else if (!sub) {
            // the token's entry into E (exact phase) or S_0 rides along (the bookkeeping follows below)
            int32_t *list = s->n + 1 <= n_out ? E : Slist(0);
            const int64_t pos = s->n + 1 <= n_out ? s->n_E : s->n_S[0];
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(blocks(total), (unsigned)BH);
            cfg.blockDim = dim3(256);
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            const int64_t cap = total;
            const int32_t value = (int32_t)t;
            ELM_CUDA_TRY(cudaLaunchKernelEx(&cfg, build_list_append_kernel, pc, n, ep_idx, ep_w, cap, list, pos, value));
            appended = true;
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
        if (appended) return (int)ELM_OK;                                  // done with the list's launch
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
