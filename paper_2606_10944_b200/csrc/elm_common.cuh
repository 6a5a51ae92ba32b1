// Shared host/device helpers of the CUDA library (not used by, and sharing nothing with, the
// CPU oracle).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/elm.h"

namespace elm {

// ---------------------------------------------------------------------------------------------
// launch bookkeeping and per-stage timing
// ---------------------------------------------------------------------------------------------
struct Profiler {
    bool enabled = false;
    bool attend_only = false;     // events around the attention stage only (elm_profile_enable(2))
    static constexpr int kMaxRecords = 4096;
    int n_records = 0;
    cudaEvent_t ev_begin[kMaxRecords];
    cudaEvent_t ev_end[kMaxRecords];
    int stage_of[kMaxRecords];
    int launches_of[kMaxRecords];
    int events_created = 0;
};
Profiler &profiler();
void count_launches(int n);

// RAII: times everything enqueued on `stream` during its lifetime as one record of `stage`.
class StageTimer {
  public:
    StageTimer(int stage, cudaStream_t stream, int launches);
    ~StageTimer();

  private:
    int rec_ = -1;
    cudaStream_t stream_;
};

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? ELM_OK : ELM_ERR_CUDA; }

#define ELM_CUDA_TRY(expr)                                \
    do {                                                  \
        cudaError_t _e = (expr);                          \
        if (_e != cudaSuccess) return ELM_ERR_CUDA;       \
    } while (0)

// Launch with programmatic stream serialization: the grid may become resident before the kernel in front of it in
// the stream has finished, which takes the launch latency off a chain of short dependent kernels.  The kernel must
// call cudaGridDependencySynchronize() before it reads or writes global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Multiprocessors of the current device (looked up once per device ordinal; 148 if the query fails).
int device_sm_count();

// `allow_e4m3`: the entry point accepts 8-bit inputs (then d must be 128)
int validate_params(const elm_params *p, bool allow_e4m3 = false);
int validate_attend_params(const elm_params *p, bool allow_e4m3 = false);
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elt_bytes(int dtype) { return dtype == ELM_BF16 ? 2 : (dtype == ELM_E4M3 ? 1 : 4); }

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ T load_as(const float *p, int64_t i) { return (T)p[i]; }
template <typename T> __device__ __forceinline__ T load_as(const __nv_bfloat16 *p, int64_t i)
{
    return (T)__bfloat162float(p[i]);
}
__device__ __forceinline__ void store_from(float *p, int64_t i, double v) { p[i] = (float)v; }
__device__ __forceinline__ void store_from(float *p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void store_from(__nv_bfloat16 *p, int64_t i, double v)
{
    p[i] = __float2bfloat16_rn((float)v);
}
__device__ __forceinline__ void store_from(__nv_bfloat16 *p, int64_t i, float v)
{
    p[i] = __float2bfloat16_rn(v);
}

// Row numbers that come from the caller (idx of elm_attend) index K and V unchecked in a normal build.  A build
// with -DELM_BOUNDS_CHECK tests each against [0, n): a bad one is replaced by row 0 and reported through the
// call's status word (ELM_STATUS_BAD_ROW) - never by trapping.
constexpr int ELM_STATUS_BAD_ROW = 64;
__device__ __forceinline__ int64_t checked_row(int64_t row, int64_t n, int *status)
{
#ifdef ELM_BOUNDS_CHECK
    if (row < 0 || row >= n) {
        if (status) atomicExch(status, ELM_STATUS_BAD_ROW);
        return 0;
    }
#else
    (void)n;
    (void)status;
#endif
    return row;
}

// Philox4x32-10 (Salmon et al., SC'11), first output word only.
__host__ __device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2,
                                                                 uint32_t c3, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

// The uniform of pair `pair` of Halve call `group` at `level` of attention problem `problem`:
// top 24 bits of the first Philox word, so the value is exact in fp32 and fp64 alike.
// Second and third counter words of Halve call g of a level.  `lvl` packs three fields:
//   bits  0-15  the level's third counter word,
//   bits 16-39  the number of the level's first call (a streaming run makes the calls of a level one
//               launch at a time),
//   bits 40-63  non-zero when the level batches sibling segments of an Express round with that many
//               calls each: call g is then call g % calls of sibling g / calls, whose third word is
//               64 further on per sibling.
__host__ __device__ __forceinline__ int64_t pack_level(int code, int64_t first_call, int64_t calls_per_sibling)
{
    return (int64_t)code | (first_call << 16) | (calls_per_sibling << 40);
}
__device__ __forceinline__ void call_counter(int g, int64_t lvl, uint32_t &group, uint32_t &code)
{
    const uint32_t per = (uint32_t)(lvl >> 40);
    code = (uint32_t)lvl & 0xffffu;
    group = (uint32_t)(lvl >> 16) & 0xffffffu;
    if (per) {
        group += (uint32_t)g % per;
        code += 64u * ((uint32_t)g / per);
    } else {
        group += (uint32_t)g;
    }
}

template <typename T>
__host__ __device__ __forceinline__ T halving_uniform(uint64_t seed, uint32_t pair, uint32_t group,
                                                      uint32_t level, uint32_t problem)
{
    uint32_t w = philox4x32_10_word0(pair, group, level, problem, (uint32_t)seed, (uint32_t)(seed >> 32));
    return (T)(w >> 8) * (T)(1.0 / 16777216.0);
}

// exp with the underflow floor used throughout the halving path: a shifted exponent below the
// floor gives exactly 0, so no subnormal ever enters a difference of kernel values.
__device__ __forceinline__ double floored_exp(double x) { return x < -700.0 ? 0.0 : exp(x); }
__device__ __forceinline__ float floored_exp(float x) { return x < -80.0f ? 0.0f : __expf(x); }

}  // namespace elm
