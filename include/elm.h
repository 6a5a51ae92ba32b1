/*
 * elm.h -- C ABI of the B200 (sm_100a) kernel-halving compression + weighted attention library.
 *
 * The two main calls follow the problem statement of "Express Language Modeling"
 * (arXiv 2606.10944):
 *
 *   elm_compress   a thinning algorithm in the sense of Definition 1: every attention problem
 *                  (one batch entry, one KV head) with n key-value pairs is reduced to a coreset
 *                  of n_out = 2^log2_nout of its own points with positive weights summing to 1.
 *                  The thinning is Offline-Compress2 (the recursive form of Algorithm 2) with
 *                  Halve = KH(delta) (Algorithm A.1) under the key-value attention kernel of
 *                  Eq. (katt).
 *   elm_attend     Eq. (def:att_approx) / the return line of Algorithm 5: every query attends
 *                  over one weighted coreset with softmax weights w * exp(<q,k>/sqrt(d)).
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers unless the name ends in _host.  The caller owns
 *     every buffer; the library allocates no device memory and keeps no pointer after return.
 *   - Tensors are dense and row-major: Q, O [batch][q_heads][n_q][d]; K, V [batch][kv_heads][n_kv][d];
 *     idx, w [batch][kv_heads][n_core].  Element type of Q, K, V, O is params->dtype.
 *     Base pointers must be 16-byte aligned.
 *   - Query head h of a batch entry reads KV head floor(h * kv_heads / q_heads) (grouped queries).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Device calls
 *     only enqueue work; they do not synchronise.
 *   - The return value is ELM_OK (0) or a negative elm_status.  Argument errors are detected on
 *     the host before anything is launched.  Nothing throws across this boundary.
 */
#ifndef ELM_H
#define ELM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ELM_E4M3: 8-bit floats (OCP E4M3, the finite-only variant: 4 exponent bits, 3 mantissa bits, no infinities) for
 * Q, K and V, taken as the numbers they encode - no scale factors.  The paper's Conclusion names FP8 as future
 * work; this library accepts it in elm_workspace_bytes, elm_compress, elm_attend (and their helper calls) with
 * d = 128.  O is then bf16.  Every E4M3 value is also a bf16 value, so the compression and the fp64-mode
 * attention run on an exact widened copy (in the workspace) and give what they would give on bf16 inputs holding
 * the same numbers; the fp32-mode attention computes S = Q K^T with 8-bit tensor-core operands and fp32
 * accumulation (products of E4M3 numbers are exact in fp32), the probabilities and P V in bf16 as for bf16 inputs. */
typedef enum { ELM_F32 = 0, ELM_BF16 = 1, ELM_E4M3 = 2 } elm_dtype;

typedef enum {
    ELM_PREC_FP64_DET = 0, /* all kernel-halving arithmetic in fp64: decisions reproduce an fp64
                              CPU statement of Algorithm A.1 unless a uniform falls within
                              rounding distance of its swap probability */
    ELM_PREC_FP32 = 1      /* fp32 accumulation; bf16 inputs use the tensor cores */
} elm_precision;

typedef enum {
    ELM_OK = 0,
    ELM_ERR_NULL = -1,        /* a required pointer is NULL */
    ELM_ERR_SHAPE = -2,       /* unsupported or inconsistent sizes */
    ELM_ERR_DTYPE = -3,       /* unknown dtype / precision */
    ELM_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned */
    ELM_ERR_WORKSPACE = -5,   /* workspace too small */
    ELM_ERR_DELTA = -6,       /* a failure parameter outside (0, 1) */
    ELM_ERR_CUDA = -7,        /* a CUDA runtime call or launch failed */
    ELM_ERR_UNAVAILABLE = -8, /* no usable CUDA device */
    ELM_ERR_STATIC_LIMIT = -9 /* elm_attend_static: the coreset does not fit the built-in scratch */
} elm_status;

typedef struct elm_params {
    int32_t batch;       /* B >= 1 */
    int32_t q_heads;     /* H_q, a multiple of kv_heads */
    int32_t kv_heads;    /* H_kv */
    int32_t n_kv;        /* n: key-value pairs per attention problem; must equal 2^m * 2^log2_nout */
    int32_t n_q;         /* queries per head (any value >= 1) */
    int32_t d;           /* head dimension: 64 or 128 */
    int32_t log2_nout;   /* coreset size n_out = 2^log2_nout (Algorithm 4's h) */
    int32_t m;           /* Compress2 depth (Algorithm 2); 0 returns every point; the level-0
                            groups hold n_kv / 4^(m-1) points and must hold at least 2 */
    int32_t dtype;       /* elm_dtype of Q, K, V and O (ELM_E4M3: of Q, K, V; O is bf16) */
    int32_t precision;   /* elm_precision */
    double delta;        /* failure budget delta in (0,1); the paper's experiments use 1/2 */
    const double *delta_level; /* optional HOST array[m]: KH failure parameter of level i.  NULL
                                  selects delta_i = 4^(i+1-m) * delta / (3m), the schedule of
                                  Corollary 2 with this call's own depth */
} elm_params;

/* Bytes of device workspace elm_compress and elm_attend need for `params` (n_core taken as
 * n_out).  Either output pointer may be NULL. */
int elm_workspace_bytes(const elm_params *params, size_t *compress_bytes, size_t *attend_bytes);

/* The default per-level failure parameters described at elm_params.delta_level; out[m] on the host. */
int elm_default_delta_levels(int32_t m, double delta, double *out_host);

/*
 * Definition 1 + Offline-Compress2 + Algorithm A.1 under Eq. (katt).
 *   K, V       [batch][kv_heads][n_kv][d], read only.
 *   seed       selects the uniforms: pair i of Halve call g at level l of problem p uses the first
 *              word of Philox4x32-10(counter = (i, g, l, p), key = (seed low, seed high)), top 24 bits.
 *   idx_out    [batch][kv_heads][n_out] row numbers in [0, n_kv), in the order Algorithm A.1 appends
 *              them (not sorted); all distinct.
 *   w_out      [batch][kv_heads][n_out], every entry 1/n_out.
 *   workspace  at least compress_bytes of elm_workspace_bytes, 256-byte aligned; contents are
 *              scratch.  Two calls that overlap in time need separate workspaces.
 * v_max of Eq. (katt) is taken per attention problem.  exp(<k,k'>/sqrt(d)) is evaluated with a
 * running shift (the largest ||k||^2/sqrt(d) seen so far in the Halve call), which leaves every
 * swap probability unchanged and keeps the arithmetic finite for any input.
 */
int elm_compress(const void *K, const void *V, const elm_params *params, uint64_t seed,
                 int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes,
                 void *stream);

/*
 * Algorithm 2 (Compress2 in its streaming form) on a sequence of any length, the first n_sink and the
 * last n_window rows kept exactly (the paper's experiments keep 32 and 32 and compress the rows in
 * between).  The n_mid = n_kv - n_sink - n_window middle rows are what Compress2(m, n_in = 2^m n_out)
 * holds after n_mid updates in row order: level i has made floor(a_i / t_i) Halve calls on consecutive
 * stretches of t_i = n_in 2^i / 4^(m-1) points (a_0 = n_mid, a_(i+1) = half of what level i consumed);
 * the a_i mod t_i points left over stay in S_i.  wtd_cache() gives a point of S_i the weight 2^(i-m);
 * sink and window rows carry the weight of a raw point, 2^-m; all weights are then divided by their
 * sum n_kv 2^-m (Definition 1: positive, summing to 1), i.e. 2^i / n_kv and 1 / n_kv.
 *   params     n_kv: any length >= 1 with 0 <= n_mid <= 2^m n_out; m >= 1 needs log2_nout - m + 2 >= 1
 *              as in elm_compress; q_heads and n_q are not used.
 *   K, V       [batch][kv_heads][n_kv][d]; v_max and the uniforms as in elm_compress (call g of level l
 *              is the g-th stretch of that level), so with n_kv = 2^m n_out and no sink or window rows
 *              the result is that of elm_compress.
 *   idx_out, w_out   [batch][kv_heads][count], count from elm_compress_ragged_count (it depends on the
 *              sizes only): sink rows, S_0, S_1, ..., S_m (each in append order), window rows.
 *   workspace  at least the bytes elm_compress_ragged_count reports, 256-byte aligned.
 * The result feeds elm_attend (n_core = count) unchanged.
 */
int elm_compress_ragged_count(const elm_params *params, int32_t n_sink, int32_t n_window, int32_t *count,
                              size_t *workspace_bytes);
int elm_compress_ragged(const void *K, const void *V, const elm_params *params, int32_t n_sink, int32_t n_window,
                        uint64_t seed, int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes,
                        void *stream);

/*
 * Eq. (def:att_approx) with one coreset per attention problem (Algorithm 5's return line).
 *   Q          [batch][q_heads][n_q][d]
 *   K, V       the ORIGINAL [batch][kv_heads][n_kv][d] tensors; rows are gathered through idx.
 *   idx, w     [batch][kv_heads][n_core]; any positive finite weights (they need not sum to 1),
 *              1 <= n_core <= n_kv.  Every entry of idx must lie in [0, n_kv): the rows are read
 *              through it unchecked (the caller's obligation; a build with -DELM_BOUNDS_CHECK
 *              skips such an entry and reports it through the status word instead).
 *   params     n_kv may be any length >= 1 here; log2_nout, m, delta are not used.
 *   O          [batch][q_heads][n_q][d], same dtype as Q.
 *   workspace  at least elm_attend_workspace_bytes(params, n_core), 256-byte aligned.
 * precision FP64_DET accumulates in fp64, FP32 in fp32 (bf16 inputs: tensor cores).
 */
int elm_attend(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w,
               int32_t n_core, const elm_params *params, void *O, void *workspace,
               size_t workspace_bytes, void *stream);

/* Workspace of elm_attend for an explicit coreset size. */
int elm_attend_workspace_bytes(const elm_params *params, int32_t n_core, size_t *bytes);

/*
 * elm_attend for callers that cannot hand over a workspace.  (The paper has no counterpart: this
 * is a packaging variant of elm_attend, same arithmetic, same kernels.)
 *
 * Who needs it: code that runs after a serving process has given all device memory to its own
 * pool, plug-ins that are forbidden to call the CUDA allocator on the request path (an allocation
 * there can stall every stream of the process or fail outright when the pool owns the card), and
 * embedders that only hold raw pointers to Q/K/V/O and have nowhere to carve a workspace from.
 * This entry point calls no cudaMalloc, cudaFree or any other allocating routine, and takes no
 * workspace argument.  The gathered coreset operands are staged in an array of
 * ELM_ATTEND_STATIC_SCRATCH_BYTES that is compiled into the library as device global memory;
 * every GPU that loads the library holds that array until the process exits.
 *
 * Arguments, layouts, dtype / precision handling and results are those of elm_attend.
 * Limits and rules:
 *   - elm_attend_workspace_bytes(params, n_core) must not exceed ELM_ATTEND_STATIC_SCRATCH_BYTES
 *     (e.g. 8 KV problems x 2048 coreset points x d = 128 in bf16 needs about 8.1 MiB); larger
 *     requests return ELM_ERR_STATIC_LIMIT before anything is launched.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  Each
 *     call rewrites every byte it later reads, so nothing needs clearing, but two calls whose
 *     kernels can overlap on the GPU (different streams, no ordering between them) race on it:
 *     order them, or use elm_attend with separate workspaces.
 *   - Per-stage timing (elm_profile_enable) does not cover this entry point.
 *   - The bounded waits of the tensor-core kernels report through a status word that lives in the
 *     same array; elm_attend_static_status copies it to *status_host (0 = every wait completed) after
 *     synchronising `stream`, for the (params, n_core) of the last call on this device.  It allocates
 *     nothing either.  A non-zero word means O of that call is undefined.
 */
#define ELM_ATTEND_STATIC_SCRATCH_BYTES (16u << 20)
int elm_attend_static(const void *Q, const void *K, const void *V, const int32_t *idx, const float *w,
                      int32_t n_core, const elm_params *params, void *O, void *stream);
int elm_attend_static_status(const elm_params *params, int32_t n_core, int32_t *status_host, void *stream);

/*
 * Offline-Express (the recursive form of Algorithm 1, "Express", with Subsample - Algorithm 3 - and
 * Compress2 - Algorithm 2 - inside and Halve = KH(delta) with the failure parameters of Corollary 2,
 * i.e. KH-Express): the n_out points a streaming Express cache holds after n_kv = n_out 4^R key-value
 * pairs, R >= 0, for every attention problem.  E starts as the first n_out points; round r = 0 .. R-1
 * (thinning factor m = 2r) thins the next three segments of n_out 2^m points each - one stratified
 * uniform draw per 2^(m - mbar) points when m > mbar, then Compress2 of depth min(m, mbar) - appends
 * the three results to E and halves the 4 n_out points of E twice with KH(delta_m / 2), where
 * delta_m = (delta/2)(1/log2(m/2 + 2) - 1/log2(m/2 + 3)); level i of a depth-q Compress2 uses
 * KH(4^(i+1-q) delta_m / (3q)).
 *   params     batch, kv_heads, n_kv, d, log2_nout (>= 1), dtype, precision and delta are used;
 *              n_kv must equal 2^log2_nout * 4^R.  q_heads, n_q, m and delta_level are ignored.
 *   mbar       inflation factor of Algorithm 1 (0 .. 30); the paper's experiments use log2_nout - 2
 *              for prefill.
 *   seed       uniforms as in elm_compress, with the counter's third word numbering the call's place
 *              in the recursion: i + 64 (4r + j) for Halve_i of segment j in {1,2,3} of round r,
 *              62 / 63 + 64 (4r) for the two halvings of E, 61 + 64 (4r + j) for the draws of
 *              segment j (first word = stratum number, point = stratum start + floor(U 2^(m-mbar))).
 *   idx_out    [batch][kv_heads][n_out] row numbers in [0, n_kv) in the order the last halving
 *              appends them; w_out the same shape, every entry 1/n_out.
 *   workspace  at least elm_express_workspace_bytes(params, mbar) bytes, 256-byte aligned.
 * v_max of Eq. (katt) is taken over the whole sequence of the problem.  In fp64 mode a call of more
 * than 2048 pairs (n_out > 1024 here) is not supported and returns ELM_ERR_SHAPE.
 * This is the compression half of causal prefill with Thinformer Express (Algorithm 5); see
 * elm_express_prefill for the attention of every query over the cache as of its own position.
 */
int elm_express_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes);

/*
 * Thinformer Express (Algorithm 5) in prefill: O[t] = WtdAttention(q_t, cache as of token t plus token
 * t itself) for every token t of every head, where the cache is that of the Express run described at
 * elm_express_compress (computed by the same recursion, with the same uniforms), and that cache after
 * the last token in idx_out / w_out.  Token t's cache is: E with the segments finished so far (weight
 * 1), for every Compress2 level i the outputs of Halve calls that the next level has not consumed yet
 * (weight 2^(i-q), q = the current Compress2 depth), and the tokens since the last level-0 Halve call
 * up to t (weight 2^-q).  The first 4 n_out tokens attend exactly (causally).
 *   Q, O       [batch][q_heads][n_kv][d] (params->n_q must equal n_kv); K, V as for elm_compress.
 *   Limits     level-0 Halve calls need >= 2 points: min(2 (R-1), mbar) <= log2_nout + 1, else ELM_ERR_SHAPE.
 *   workspace  at least elm_express_prefill_workspace_bytes(params, mbar) bytes, 256-byte aligned.
 * In a round whose thinning factor exceeds mbar (Subsample active) the kept points differ from problem to
 * problem; a token that is not kept still attends to itself with the weight of a point of S_0.
 * Every cache entry carries the span of tokens that see it.  bf16 inputs in fp32 mode, in rounds whose segments
 * are multiples of 256 tokens: the entries of a whole round are gathered once and one attention launch serves the
 * round, each pair of 128-query tiles streaming the blocks of 128 entries that hold something its tokens see.
 * Otherwise: one attention launch per window of about 512 tokens over every entry some token of the window sees.
 * The call copies a table of a few hundred KB from pageable host memory to the device per round (which pairs of
 * query tiles each persistent CTA takes) - it enqueues, but is not capturable into a CUDA graph.
 */
int elm_express_prefill_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes);
int elm_express_prefill(const void *Q, const void *K, const void *V, const elm_params *params, int32_t mbar,
                        uint64_t seed, void *O, int32_t *idx_out, float *w_out, void *workspace,
                        size_t workspace_bytes, void *stream);
int elm_express_compress(const void *K, const void *V, const elm_params *params, int32_t mbar, uint64_t seed,
                         int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Streaming Thinformer Express (Algorithms 1, 2 and 5 with Halve = KH(delta) at the failure parameters
 * of Corollary 2), one token per call: elm_stream_step first attends the new token's queries over the
 * weighted cache plus the token itself, then feeds the token's key-value pair to the cache
 * (Express.update: exact phase, Compress2 levels S_0..S_q with a Halve call whenever a level is full,
 * hand-over to E at the end of a thin phase, two halvings of E at the end of a round).  The cache never
 * exceeds 6 n_out points.  After n_out 4^R tokens it equals the result of elm_express_compress, and
 * every output equals elm_express_prefill's.
 *   elm_stream     plain HOST struct owned by the caller; elm_stream_init fills it, the library keeps no
 *                  other state.  All arrays live in the caller's device workspace.
 *   params         batch, q_heads, kv_heads, d, log2_nout, dtype, precision, delta as elsewhere; n_kv is
 *                  the CAPACITY (rows of K and V per problem); n_q must be 1.
 *   K, V           [batch][kv_heads][n_kv][d]; row t must be valid when step t is enqueued.
 *   n_known        rows of K and V already valid at init: v_max of Eq. (katt) starts as the largest
 *                  |v| over them and grows with the tokens seen later (with n_known = the whole
 *                  sequence this is the v_max of elm_express_compress).
 *   Q_t, O_t       [batch][q_heads][1][d]
 *   Limits         mbar <= 12; level-0 Halve calls need >= 2 points.
 * Thinning factors above mbar (Subsample, Algorithm 3): problem p keeps one token of every stratum of
 * 2^(m - mbar), chosen by the uniform of counter (stratum, 0, 61 + 64 (4 r + j), p), so inside a stratum
 * the problems take their Compress2.update - and the Halve calls it triggers, one problem at a time - at
 * different tokens; the counters in elm_stream describe the state at the stratum's start and move on at
 * its end.  Where the problems' lists then differ in length, a shorter one repeats its last entry with
 * that entry's weight split over the copies (every weighted sum over the list is unchanged).
 * Calls only enqueue work on `stream`; the host struct is updated immediately (the schedule of Halve
 * calls depends on the token count and the draws alone).
 */
typedef struct elm_stream {
    int64_t n, ell, n_E;          /* tokens seen, tokens of the current thin phase, points in E */
    int32_t m, b, q, mbar;        /* thinning factor, finished segments of the round, Compress2 depth */
    int64_t n_S[16], calls[16];   /* points in S_i; Halve calls made at level i of the current Compress2 */
    int64_t n_known;
    uint64_t seed;
} elm_stream;
int elm_stream_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes);
int elm_stream_init(elm_stream *s, const void *K, const void *V, int64_t n_known, const elm_params *params,
                    int32_t mbar, uint64_t seed, void *workspace, size_t workspace_bytes, void *stream);
int elm_stream_step(elm_stream *s, const void *Q_t, const void *K, const void *V, const elm_params *params,
                    void *O_t, void *workspace, size_t workspace_bytes, void *stream);
/* n_tokens calls of elm_stream_step enqueued by one call (Algorithm 4's attend, token after token): Q_T and O_T hold
 * the tokens' queries and outputs one after the other, [n_tokens][batch][q_heads][1][d]; token i is row s->n + i of K
 * and V when the call starts.  Stops at the first step that fails and returns its status (the steps before it stay
 * enqueued and counted in *s). */
int elm_stream_steps(elm_stream *s, int32_t n_tokens, const void *Q_T, const void *K, const void *V,
                     const elm_params *params, void *O_T, void *workspace, size_t workspace_bytes, void *stream);
/* The current cache, wtd_cache() of Algorithm 1: at most 6 n_out entries per problem, [batch][kv_heads][count]
 * row numbers and (unnormalised) weights 2^(i-q) / 1; *count_host receives the number of entries (inside a
 * stratum of a subsampled phase: of the longest list; see above for the padding of the others). */
int elm_stream_cache(const elm_stream *s, const elm_params *params, int32_t *idx_out, float *w_out,
                     int32_t *count_host, void *workspace, size_t workspace_bytes, void *stream);

/*
 * End-to-end convenience call on HOST buffers: copies Q, K, V to the device, runs elm_compress and
 * elm_attend, copies O (and, when non-NULL, idx and w) back, and returns when everything has
 * arrived.  The host link bounds this call, so uploads, kernels and downloads overlap: K and V go
 * first on `stream` with the compression behind them; Q follows on a second, internal stream in
 * chunks of one attention problem's query heads; each chunk is attended on `stream` as soon as it
 * has landed and its part of O leaves on a third stream.  The internal streams and events are
 * created and destroyed inside the call (no device memory is allocated).  Host buffers may be
 * pageable or pinned; only pinned buffers overlap.  `device_scratch` is a DEVICE buffer of at
 * least elm_host_call_scratch_bytes(params) bytes, 256-byte aligned, owned by the caller.
 */
int elm_host_call_scratch_bytes(const elm_params *params, size_t *bytes);
int elm_compress_attend_host(const void *Q_host, const void *K_host, const void *V_host,
                             void *O_host, int32_t *idx_host, float *w_host,
                             const elm_params *params, uint64_t seed, void *device_scratch,
                             size_t device_scratch_bytes, void *stream);

/*
 * Per-stage device timing (off by default).  When enabled, every elm_compress / elm_attend call
 * records CUDA events around each of its stages on the caller's stream; elm_profile_read
 * synchronises those events and returns, for stage s < ELM_N_STAGES, the accumulated milliseconds
 * and kernel launches since the last read, then resets them.  Not thread safe.
 * elm_profile_enable(1) times every stage; elm_profile_enable(2) only ELM_STAGE_ATTEND (launches are still
 * counted for all).  The events between the stages cost time of their own - on cfg5 the compression's twenty
 * short launches take 1.09 ms with them and 0.94 ms without, because a kernel behind an event cannot become
 * resident while its predecessor drains (the kernels are launched with programmatic stream serialization) - so a
 * caller that times whole steps leaves the mode at 0 or 2.
 */
enum {
    ELM_STAGE_PREPASS = 0,  /* v_max, key norms, identity index list */
    ELM_STAGE_LEVEL_PREP,   /* per-level running shifts */
    ELM_STAGE_GRAM,         /* kernel evaluation -> pair Gram */
    ELM_STAGE_WALK,         /* halving walk */
    ELM_STAGE_EMIT,         /* weights */
    ELM_STAGE_GATHER,       /* coreset rows -> contiguous operands */
    ELM_STAGE_ATTEND,       /* weighted attention */
    ELM_N_STAGES
};
int elm_profile_enable(int on);
int elm_profile_read(float *ms_out, int64_t *launches_out, int32_t n_stages);

/*
 * Device-side health of the last elm_compress / elm_attend call that used `workspace`.  Every wait
 * inside the tensor-core kernels (on an mbarrier) is bounded; a wait that expires (about 2 s)
 * records a non-zero code in a status word inside the workspace and the launch winds down instead
 * of hanging, leaving its outputs undefined.  These calls copy that word to *status_host (0 = every
 * wait completed) after synchronising `stream`.  `params` / `n_core` must be those of the call.
 * elm_compress_status reads batch and kv_heads only and serves the workspace of every compression
 * call (elm_compress, elm_compress_ragged, elm_express_compress / _prefill, elm_stream_*).
 */
int elm_compress_status(const void *workspace, const elm_params *params, int32_t *status_host, void *stream);
int elm_attend_status(const void *workspace, const elm_params *params, int32_t n_core, int32_t *status_host,
                      void *stream);

/*
 * Test hooks (no counterpart in the paper).  They exist so that the failure path of the bounded waits can be
 * exercised without hanging or faulting anything:
 *   ELM_DEBUG_WAIT_LIMIT_NS            the time limit of the bounded waits of the tensor-core attention kernel
 *                                      (default 2 000 000 000; at least 1 000 000), for launches from now on;
 *   ELM_DEBUG_ATTEND_MISSING_ARRIVALS  the NEXT tensor-core elm_attend launch expects `value` arrivals on its
 *                                      "probabilities ready" barriers that nobody makes: the waits on them run
 *                                      out, the launch winds down, elm_attend_status reads non-zero and O is
 *                                      undefined.  One launch only; later calls are normal again.
 * Environment variables read by the library (tuning aids, off the documented path): ELM_WALK_CHAIN_MIN_PAIRS
 * (default 1024: Halve calls with at least this many pairs take the cluster walk kernel; 32 .. 4096) and
 * ELM_PREFILL_WINDOW (default 512: tokens per attention launch of elm_express_prefill in the rounds that are
 * taken in windows; a power of two >= 64) and ELM_PREFILL_ROUNDS (default on; 0: every thinned round of the prefill
 * is taken in windows - otherwise bf16 inputs in fp32 mode take one attention launch per round whenever a round's
 * segments are multiples of 256 tokens).
 * A build with -DELM_BOUNDS_CHECK (ELM_NVCC_EXTRA of the build script) checks every caller-supplied row number
 * of elm_attend against [0, n_kv): a bad one reads row 0 instead and sets the status word to 64.
 */
enum { ELM_DEBUG_WAIT_LIMIT_NS = 0, ELM_DEBUG_ATTEND_MISSING_ARRIVALS = 1 };
int elm_debug_set(int32_t what, int64_t value);
/*
 * Host-only consistency check of elm_express_prefill's one-launch-per-round form (no CUDA call; for tests): for
 * round r >= 1 of the run described by (params, mbar) it rebuilds, on the host, the lifetime of every entry of the
 * round's list and the blocks of 128 entries each pair of 128-query tiles streams, with the kept points of
 * subsampled rounds drawn from `seed`, and counts in *missing the (pair, entry) combinations where a token of the
 * pair sees the entry but the entry's block is not in the pair's list, plus the entries of blocks listed as "seen
 * whole by the pair" that some token of the pair does not see, plus the places where a birth or a death decreases
 * within a block (must be 0).  *listed_blocks / *needed_blocks:
 * blocks streamed over all pairs, and how many of them hold an entry the pair sees; *partly_blocks: how many are
 * listed as possibly partly visible (the attention kernel looks at lifetimes only there).  ELM_ERR_SHAPE when the
 * round does not take that form (other storage or precision, segments that are not multiples of 256 tokens).
 */
int elm_debug_round_check(const elm_params *params, int32_t mbar, int32_t r, uint64_t seed, int64_t *missing,
                          int64_t *listed_blocks, int64_t *needed_blocks, int64_t *partly_blocks);

/* Kernels launched by this library since it was loaded (all calls, all stages). */
int64_t elm_launch_count(void);

const char *elm_strerror(int status);
int elm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ELM_H */
