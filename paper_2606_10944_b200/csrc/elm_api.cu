// Host-side pieces of the C ABI that launch nothing themselves: argument validation, workspace
// sizing, the host-buffer convenience call, per-stage timing and status text.
#include <math.h>
#include <stdio.h>

#include <atomic>
#include <mutex>

#include <vector>

#include "elm_attend.cuh"
#include "elm_common.cuh"
#include "elm_compress.cuh"

namespace elm {

static std::atomic<int64_t> g_launches{0};
static int64_t g_stage_launches[ELM_N_STAGES];

Profiler &profiler()
{
    static Profiler p;
    return p;
}

void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

StageTimer::StageTimer(int stage, cudaStream_t stream, int launches) : stream_(stream)
{
    if (stage < 0) return;      // untimed caller
    Profiler &pr = profiler();
    g_stage_launches[stage] += launches;
    if (!pr.enabled || pr.n_records >= Profiler::kMaxRecords) return;
    if (pr.attend_only && stage != ELM_STAGE_ATTEND) return;
    rec_ = pr.n_records++;
    if (rec_ >= pr.events_created) {
        cudaEventCreate(&pr.ev_begin[rec_]);
        cudaEventCreate(&pr.ev_end[rec_]);
        pr.events_created = rec_ + 1;
    }
    pr.stage_of[rec_] = stage;
    pr.launches_of[rec_] = launches;
    cudaEventRecord(pr.ev_begin[rec_], stream_);
}

StageTimer::~StageTimer()
{
    if (rec_ >= 0) cudaEventRecord(profiler().ev_end[rec_], stream_);
}

int validate_params(const elm_params *p, bool allow_e4m3)
{
    if (p->batch < 1 || p->kv_heads < 1 || p->q_heads < 1 || p->n_q < 1) return ELM_ERR_SHAPE;
    if (p->q_heads % p->kv_heads != 0) return ELM_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return ELM_ERR_SHAPE;
    if (p->log2_nout < 0 || p->log2_nout > 24 || p->m < 0 || p->m > 12) return ELM_ERR_SHAPE;
    if (p->log2_nout + p->m > 30) return ELM_ERR_SHAPE;
    if ((int64_t)p->n_kv != ((int64_t)1 << (p->log2_nout + p->m))) return ELM_ERR_SHAPE;
    if (p->m >= 1 && p->log2_nout - p->m + 2 < 1) return ELM_ERR_SHAPE;      // level-0 groups >= 2 points
    if ((int64_t)p->batch * p->q_heads > 65535) return ELM_ERR_SHAPE;
    if (p->dtype != ELM_F32 && p->dtype != ELM_BF16 && !(allow_e4m3 && p->dtype == ELM_E4M3)) return ELM_ERR_DTYPE;
    if (p->dtype == ELM_E4M3 && p->d != 128) return ELM_ERR_SHAPE;
    if (p->precision != ELM_PREC_FP64_DET && p->precision != ELM_PREC_FP32) return ELM_ERR_DTYPE;
    if (!(p->delta > 0.0 && p->delta < 1.0)) return ELM_ERR_DELTA;
    if (p->delta_level)
        for (int i = 0; i < p->m; ++i)
            if (!(p->delta_level[i] > 0.0 && p->delta_level[i] < 1.0)) return ELM_ERR_DELTA;
    return ELM_OK;
}

// The attention calls read K and V through an index list: any n_kv, and log2_nout / m are not used.
int validate_attend_params(const elm_params *p, bool allow_e4m3)
{
    if (p->batch < 1 || p->kv_heads < 1 || p->q_heads < 1 || p->n_q < 1 || p->n_kv < 1) return ELM_ERR_SHAPE;
    if (p->q_heads % p->kv_heads != 0) return ELM_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return ELM_ERR_SHAPE;
    if ((int64_t)p->batch * p->q_heads > 65535) return ELM_ERR_SHAPE;
    if (p->dtype != ELM_F32 && p->dtype != ELM_BF16 && !(allow_e4m3 && p->dtype == ELM_E4M3)) return ELM_ERR_DTYPE;
    if (p->dtype == ELM_E4M3 && p->d != 128) return ELM_ERR_SHAPE;
    if (p->precision != ELM_PREC_FP64_DET && p->precision != ELM_PREC_FP32) return ELM_ERR_DTYPE;
    return ELM_OK;
}

}  // namespace elm

using namespace elm;

extern "C" int elm_workspace_bytes(const elm_params *params, size_t *compress_bytes, size_t *attend_bytes)
{
    if (!params) return ELM_ERR_NULL;
    int rc = validate_params(params, true);
    if (rc != ELM_OK) return rc;
    if (compress_bytes) *compress_bytes = compress_layout(params).total;
    if (attend_bytes) *attend_bytes = attend_layout(params, 1 << params->log2_nout).total;
    return ELM_OK;
}

extern "C" int elm_default_delta_levels(int32_t m, double delta, double *out_host)
{
    if (!out_host && m > 0) return ELM_ERR_NULL;
    if (m < 0 || m > 32) return ELM_ERR_SHAPE;
    if (!(delta > 0.0 && delta < 1.0)) return ELM_ERR_DELTA;
    // Corollary 2's delta_{m,i} = 4^(i+1-q) delta_m / (3q) with q = this call's depth and
    // delta_m = the caller's budget.
    for (int i = 0; i < m; ++i) out_host[i] = ldexp(delta, 2 * (i + 1 - m)) / (3.0 * (double)m);
    return ELM_OK;
}

namespace {
struct HostCallLayout {
    size_t Q, K, V, O, idx, w, ws_compress, ws_attend, total;
};
HostCallLayout host_layout(const elm_params *p)
{
    HostCallLayout L;
    const size_t es = elt_bytes(p->dtype);
    const size_t qo = (size_t)p->batch * p->q_heads * p->n_q * p->d * es;
    const size_t kv = (size_t)p->batch * p->kv_heads * p->n_kv * p->d * es;
    const size_t core = (size_t)p->batch * p->kv_heads * ((size_t)1 << p->log2_nout);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.Q = take(qo);
    L.K = take(kv);
    L.V = take(kv);
    L.O = take(qo);
    L.idx = take(core * 4);
    L.w = take(core * 4);
    L.ws_compress = take(compress_layout(p).total);
    L.ws_attend = take(attend_layout(p, 1 << p->log2_nout).total);
    L.total = off;
    return L;
}
}  // namespace

extern "C" int elm_host_call_scratch_bytes(const elm_params *params, size_t *bytes)
{
    if (!params || !bytes) return ELM_ERR_NULL;
    int rc = validate_params(params);
    if (rc != ELM_OK) return rc;
    *bytes = host_layout(params).total;
    return ELM_OK;
}

extern "C" int elm_compress_attend_host(const void *Q_host, const void *K_host, const void *V_host,
                                        void *O_host, int32_t *idx_host, float *w_host,
                                        const elm_params *params, uint64_t seed, void *device_scratch,
                                        size_t device_scratch_bytes, void *stream)
{
    if (!params) return ELM_ERR_NULL;
    int rc = validate_params(params);
    if (rc != ELM_OK) return rc;
    if (!Q_host || !K_host || !V_host || !O_host || !device_scratch) return ELM_ERR_NULL;
    if ((uintptr_t)device_scratch & 255) return ELM_ERR_ALIGN;
    const HostCallLayout L = host_layout(params);
    if (device_scratch_bytes < L.total) return ELM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *base = (unsigned char *)device_scratch;
    const size_t es = elt_bytes(params->dtype);
    const size_t kv = (size_t)params->batch * params->kv_heads * params->n_kv * params->d * es;
    const size_t core = (size_t)params->batch * params->kv_heads * ((size_t)1 << params->log2_nout);
    const int32_t n_core = 1 << params->log2_nout;
    // The link is the bottleneck of this call, so it is kept busy in both directions: K and V go
    // first and the compression runs behind them; the queries follow on a second stream in chunks
    // of one (batch entry, KV head) - the query heads that share a coreset are contiguous in Q - and
    // each chunk is attended as soon as it has landed, while its output leaves on a third stream
    // under the next chunk's upload.
    const int chunks = params->batch * params->kv_heads;
    const int rep = params->q_heads / params->kv_heads;
    const size_t q_chunk = (size_t)rep * params->n_q * params->d * es;       // bytes of Q (and of O) per chunk
    const size_t kv_chunk = (size_t)params->n_kv * params->d * es;
    cudaStream_t cin = nullptr, cout = nullptr;
    cudaEvent_t ev_kv = nullptr, ev_core = nullptr;
    std::vector<cudaEvent_t> ev_q(chunks, nullptr), ev_o(chunks, nullptr);
    auto cleanup = [&]() {
        if (cin) cudaStreamDestroy(cin);
        if (cout) cudaStreamDestroy(cout);
        if (ev_kv) cudaEventDestroy(ev_kv);
        if (ev_core) cudaEventDestroy(ev_core);
        for (int c = 0; c < chunks; ++c) {
            if (ev_q[c]) cudaEventDestroy(ev_q[c]);
            if (ev_o[c]) cudaEventDestroy(ev_o[c]);
        }
    };
#define ELM_HOST_TRY(expr)                                   \
    do {                                                     \
        if ((expr) != cudaSuccess) {                         \
            cudaStreamSynchronize(st);                       \
            if (cin) cudaStreamSynchronize(cin);             \
            if (cout) cudaStreamSynchronize(cout);           \
            cleanup();                                       \
            return ELM_ERR_CUDA;                             \
        }                                                    \
    } while (0)
    ELM_HOST_TRY(cudaStreamCreateWithFlags(&cin, cudaStreamNonBlocking));
    ELM_HOST_TRY(cudaStreamCreateWithFlags(&cout, cudaStreamNonBlocking));
    ELM_HOST_TRY(cudaEventCreateWithFlags(&ev_kv, cudaEventDisableTiming));
    ELM_HOST_TRY(cudaEventCreateWithFlags(&ev_core, cudaEventDisableTiming));
    for (int c = 0; c < chunks; ++c) {
        ELM_HOST_TRY(cudaEventCreateWithFlags(&ev_q[c], cudaEventDisableTiming));
        ELM_HOST_TRY(cudaEventCreateWithFlags(&ev_o[c], cudaEventDisableTiming));
    }
    ELM_HOST_TRY(cudaMemcpyAsync(base + L.K, K_host, kv, cudaMemcpyHostToDevice, st));
    ELM_HOST_TRY(cudaMemcpyAsync(base + L.V, V_host, kv, cudaMemcpyHostToDevice, st));
    ELM_HOST_TRY(cudaEventRecord(ev_kv, st));
    ELM_HOST_TRY(cudaStreamWaitEvent(cin, ev_kv, 0));                        // K and V have the link first
    for (int c = 0; c < chunks; ++c) {
        ELM_HOST_TRY(cudaMemcpyAsync(base + L.Q + (size_t)c * q_chunk, (const unsigned char *)Q_host + (size_t)c * q_chunk,
                                     q_chunk, cudaMemcpyHostToDevice, cin));
        ELM_HOST_TRY(cudaEventRecord(ev_q[c], cin));
    }
    rc = compress_enqueue(base + L.K, base + L.V, params, seed, (int32_t *)(base + L.idx), (float *)(base + L.w),
                          base + L.ws_compress, st, 0u);
    if (rc == ELM_OK) {
        ELM_HOST_TRY(cudaEventRecord(ev_core, st));
        ELM_HOST_TRY(cudaStreamWaitEvent(cout, ev_core, 0));
        if (idx_host) ELM_HOST_TRY(cudaMemcpyAsync(idx_host, base + L.idx, core * 4, cudaMemcpyDeviceToHost, cout));
        if (w_host) ELM_HOST_TRY(cudaMemcpyAsync(w_host, base + L.w, core * 4, cudaMemcpyDeviceToHost, cout));
    }
    elm_params one = *params;                                                // one attention problem per chunk
    one.batch = 1;
    one.kv_heads = 1;
    one.q_heads = rep;
    for (int c = 0; c < chunks && rc == ELM_OK; ++c) {
        ELM_HOST_TRY(cudaStreamWaitEvent(st, ev_q[c], 0));
        rc = attend_enqueue(base + L.Q + (size_t)c * q_chunk, base + L.K + (size_t)c * kv_chunk,
                            base + L.V + (size_t)c * kv_chunk, (const int32_t *)(base + L.idx) + (size_t)c * n_core,
                            (const float *)(base + L.w) + (size_t)c * n_core, n_core, &one,
                            base + L.O + (size_t)c * q_chunk, base + L.ws_attend, st);
        if (rc != ELM_OK) break;
        ELM_HOST_TRY(cudaEventRecord(ev_o[c], st));
        ELM_HOST_TRY(cudaStreamWaitEvent(cout, ev_o[c], 0));
        ELM_HOST_TRY(cudaMemcpyAsync((unsigned char *)O_host + (size_t)c * q_chunk, base + L.O + (size_t)c * q_chunk, q_chunk,
                                     cudaMemcpyDeviceToHost, cout));
    }
    const bool sync_ok = cudaStreamSynchronize(st) == cudaSuccess && cudaStreamSynchronize(cin) == cudaSuccess &&
                         cudaStreamSynchronize(cout) == cudaSuccess;
    cleanup();
#undef ELM_HOST_TRY
    if (rc != ELM_OK) return rc;
    return sync_ok ? ELM_OK : ELM_ERR_CUDA;
}

namespace elm {
int device_sm_count()
{
    static std::mutex mu;
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}
}  // namespace elm

extern "C" int elm_compress_status(const void *workspace, const elm_params *params, int32_t *status_host, void *stream)
{
    if (!workspace || !params || !status_host) return ELM_ERR_NULL;
    if (params->batch < 1 || params->kv_heads < 1) return ELM_ERR_SHAPE;
    // the status word follows the per-problem v_max words at the head of every compression workspace
    // (elm_compress, elm_compress_ragged, elm_express_*, elm_stream_*)
    const unsigned char *word = (const unsigned char *)workspace + 4 * (size_t)params->batch * params->kv_heads;
    ELM_CUDA_TRY(cudaMemcpyAsync(status_host, word, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    ELM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return ELM_OK;
}

extern "C" int elm_attend_status(const void *workspace, const elm_params *params, int32_t n_core,
                                 int32_t *status_host, void *stream)
{
    if (!workspace || !params || !status_host) return ELM_ERR_NULL;
    int rc = validate_attend_params(params, true);
    if (rc != ELM_OK) return rc;
    if (n_core < 1 || n_core > params->n_kv) return ELM_ERR_SHAPE;
    // the status word follows the per-problem "weights differ" flags
    const unsigned char *word = (const unsigned char *)workspace + attend_layout(params, n_core).flags +
                                4 * (size_t)params->batch * params->kv_heads;
    ELM_CUDA_TRY(cudaMemcpyAsync(status_host, word, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    ELM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return ELM_OK;
}

extern "C" int elm_debug_set(int32_t what, int64_t value) { return elm::debug_set_attend_tc(what, value); }

extern "C" int elm_profile_enable(int on)
{
    Profiler &pr = profiler();
    pr.enabled = on != 0;
    pr.attend_only = on == 2;
    pr.n_records = 0;
    for (int s = 0; s < ELM_N_STAGES; ++s) g_stage_launches[s] = 0;
    return ELM_OK;
}

extern "C" int elm_profile_read(float *ms_out, int64_t *launches_out, int32_t n_stages)
{
    Profiler &pr = profiler();
    if (!ms_out || n_stages < ELM_N_STAGES) return ELM_ERR_NULL;
    for (int s = 0; s < ELM_N_STAGES; ++s) ms_out[s] = 0.f;
    for (int r = 0; r < pr.n_records; ++r) {
        if (cudaEventSynchronize(pr.ev_end[r]) != cudaSuccess) return ELM_ERR_CUDA;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, pr.ev_begin[r], pr.ev_end[r]) != cudaSuccess) return ELM_ERR_CUDA;
        ms_out[pr.stage_of[r]] += ms;
    }
    if (launches_out)
        for (int s = 0; s < ELM_N_STAGES; ++s) launches_out[s] = g_stage_launches[s];
    pr.n_records = 0;
    for (int s = 0; s < ELM_N_STAGES; ++s) g_stage_launches[s] = 0;
    return ELM_OK;
}

extern "C" int64_t elm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" const char *elm_strerror(int status)
{
    switch (status) {
    case ELM_OK: return "ok";
    case ELM_ERR_NULL: return "a required pointer is NULL";
    case ELM_ERR_SHAPE: return "unsupported or inconsistent sizes";
    case ELM_ERR_DTYPE: return "unknown dtype or precision";
    case ELM_ERR_ALIGN: return "a pointer is not sufficiently aligned";
    case ELM_ERR_WORKSPACE: return "workspace too small";
    case ELM_ERR_DELTA: return "failure parameter outside (0, 1)";
    case ELM_ERR_CUDA: return "a CUDA call or kernel launch failed";
    case ELM_ERR_UNAVAILABLE: return "no usable CUDA device";
    case ELM_ERR_STATIC_LIMIT: return "coreset operands exceed the built-in static scratch (use elm_attend with a workspace)";
    default: return "unknown status";
    }
}

extern "C" int elm_version(void) { return 100; }
