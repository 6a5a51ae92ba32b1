/*
 * elm_oracle.c -- CPU oracle for kernel-halving compression and weighted attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what the
 * CUDA library computes.  Only the test-suite, the smoke check and the benchmark's CPU
 * baseline may call it; the product never does, and the two share no code.
 *
 * Every routine follows one passage of "Express Language Modeling" (arXiv 2606.10944):
 *
 *   oracle_katt               Eq. (katt): key-value attention kernel
 *   oracle_kh                 Algorithm A.1: KH(delta) kernel halving
 *   oracle_compress2          Algorithm "Offline-Compress2" (recursive form of Algorithm 2)
 *   oracle_compress2_stream   Algorithm 2 itself, one update per point, any length, sink / window rows kept
 *   oracle_wtd_attention      Algorithm 5 / Eq. (def:att_approx): weighted attention
 *   oracle_exact_attention    Eq. (unmaskedatt): exact unmasked attention
 *   oracle_mmd2               squared kernel MMD between a point set and a weighted subset
 *   oracle_thinformer_express Algorithms 1-5 + Corollary 2: streaming Express cache with KH, per-token attention
 *   oracle_exact_causal_attention  Eq. (def:att)
 *   oracle_philox4x32_10      the counter-based generator the uniforms come from
 *
 * Inputs are float arrays (bf16 and fp32 tensors are both exactly representable there);
 * every arithmetic step is carried out in double, one term at a time, in index order.
 * There is no blocking, caching, fusion or reordering.
 *
 * Readings taken where the paper leaves a choice (each is restated where it is used):
 *   R-shift   exp(<k,k'>/sqrt(d)) is evaluated as exp(<k,k'>/sqrt(d) - M_i) with M_i the
 *             largest ||k||^2/sqrt(d) among the first 2i points of the call; the carried
 *             b_max is rescaled when M_i grows.  Every decision depends on alpha_i/a_i
 *             only, which does not change when the kernel is multiplied by a constant.
 *   R-floor   a shifted exponent below -700 gives a kernel value of exactly 0.
 *   R-tie     a_i == 0 (or not finite)  =>  swap probability 1/2.
 *   R-unif    swap iff U < p, U = (first Philox word >> 8) * 2^-24.
 *   R-order   S^(1) is kept in append order; groups are concatenated in group order.
 *   R-vmax    v_max is taken per attention problem (one batch entry, one KV head).
 *   R-delta   level i of a depth-m Compress2 uses delta_i = 4^(i+1-m) * delta / (3m).
 *
 * Pins: tests/test_oracle_*.py check this file against Philox known-answer vectors,
 * NumPy statements of the definitions, brute force on tiny inputs and the structural
 * facts the paper fixes.  The numeric coreset for a given seed depends on the readings
 * above and is therefore parity-unpinned by the paper itself (no worked example exists).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_EXP_FLOOR (-700.0)

/* ------------------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3").         */
/* ------------------------------------------------------------------------------------ */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* R-unif: the uniform of pair `pair` of Halve call `group` at level `level` of problem
 * `head` (= batch index * kv_heads + kv head).  24 bits, so the value is exact in fp32. */
double oracle_uniform(uint64_t seed, uint32_t pair, uint32_t group, uint32_t level,
                      uint32_t head)
{
    uint32_t ctr[4] = { pair, group, level, head };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return (double)(out[0] >> 8) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------------------------------ */
/* Eq. (katt)                                                                            */
/* ------------------------------------------------------------------------------------ */
static double dot_rows(const float *X, int d, int64_t a, int64_t b)
{
    const float *xa = X + a * (int64_t)d;
    const float *xb = X + b * (int64_t)d;
    double s = 0.0;
    for (int t = 0; t < d; ++t) s += (double)xa[t] * (double)xb[t];
    return s;
}

/* v_max = max_i ||v_i||_inf over the n value vectors of one attention problem (R-vmax). */
double oracle_vmax(const float *V, int64_t n, int d)
{
    double m = 0.0;
    for (int64_t i = 0; i < n * (int64_t)d; ++i) {
        double a = fabs((double)V[i]);
        if (a > m) m = a;
    }
    return m;
}

/* kappa_att((k_a,v_a),(k_b,v_b)) * exp(-shift).  shift = 0 and use_floor = 0 is the
 * paper's formula as printed; R-floor applies when use_floor != 0. */
double oracle_katt(const float *K, const float *V, int d, double vmax, int64_t a, int64_t b,
                   double shift, int use_floor)
{
    double e = dot_rows(K, d, a, b) / sqrt((double)d) - shift;
    double ex = (use_floor && e < ORACLE_EXP_FLOOR) ? 0.0 : exp(e);
    return ex * (dot_rows(V, d, a, b) + vmax * vmax);
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm A.1: KH(delta)                                                              */
/* ------------------------------------------------------------------------------------ */
/*
 * x[0..s)     the call's point sequence (row numbers into K and V), s even
 * U[0..s/2)   the uniform used by pair i (0-based)
 * shift_mode  0: the printed formula, no shift (overflows for large keys; tests only)
 *             1: R-shift + R-floor
 * S1, S2      outputs, s/2 row numbers each (S2 may be NULL)
 * diag        optional [s/2][4]: alpha_i, a_i, p_i, swapped (1.0/0.0)
 * returns 0, or -1 on a bad argument.
 */
int oracle_kh(const float *K, const float *V, int d, double vmax, const int32_t *x, int s,
              double delta, int shift_mode, const double *U, int32_t *S1, int32_t *S2,
              double *diag)
{
    if (s < 0 || (s & 1) || !(delta > 0.0)) return -1;
    const int np = s / 2;
    const double rd = sqrt((double)d);
    double bmax = 0.0;   /* b_{max,0} = 0 */
    double Mprev = 0.0;
    for (int i = 1; i <= np; ++i) {
        const int64_t xa = x[2 * i - 2];   /* x  = x_{2i-1} */
        const int64_t xb = x[2 * i - 1];   /* x' = x_{2i}   */
        double M = 0.0;
        if (shift_mode) {
            /* R-shift: M_i = max over the first 2i points of ||k||^2 / sqrt(d) */
            double ca = dot_rows(K, d, xa, xa) / rd;
            double cb = dot_rows(K, d, xb, xb) / rd;
            M = ca > cb ? ca : cb;
            if (i > 1 && Mprev > M) M = Mprev;
            /* b_max was measured with shift M_{i-1}; b scales as exp(-M/2) */
            if (i > 1) bmax = bmax * exp(-(M - Mprev) / 2.0);
        }
        /* b_i^2 = ||f_i||^2 = k(x,x) + k(x',x') - 2 k(x,x') */
        double b2 = oracle_katt(K, V, d, vmax, xa, xa, M, shift_mode)
                  + oracle_katt(K, V, d, vmax, xb, xb, M, shift_mode)
                  - 2.0 * oracle_katt(K, V, d, vmax, xa, xb, M, shift_mode);
        if (b2 < 0.0) b2 = 0.0;
        double b = sqrt(b2);
        if (b > bmax) bmax = b;                          /* b_{max,i} */
        double a = b * bmax * (0.5 + log(2.0 * (double)s / delta));   /* a_i */
        /* alpha_i = sum_{j<=2i-2} (k(x_j,x) - k(x_j,x')) - 2 sum_{z in S1} (k(z,x) - k(z,x')) */
        double sum_all = 0.0;
        for (int j = 1; j <= 2 * i - 2; ++j) {
            int64_t xj = x[j - 1];
            sum_all += oracle_katt(K, V, d, vmax, xj, xa, M, shift_mode)
                     - oracle_katt(K, V, d, vmax, xj, xb, M, shift_mode);
        }
        double sum_s1 = 0.0;
        for (int j = 0; j < i - 1; ++j) {
            int64_t z = S1[j];
            sum_s1 += oracle_katt(K, V, d, vmax, z, xa, M, shift_mode)
                    - oracle_katt(K, V, d, vmax, z, xb, M, shift_mode);
        }
        double alpha = sum_all - 2.0 * sum_s1;
        /* swap probability min(1, (1/2)(1 - alpha/a)_+), R-tie when a_i is unusable */
        double p;
        if (a > 0.0 && isfinite(a)) {
            double t = 1.0 - alpha / a;
            if (t < 0.0) t = 0.0;
            p = 0.5 * t;
            if (p > 1.0) p = 1.0;
        } else {
            p = 0.5;
        }
        int swapped = U[i - 1] < p;
        int64_t keep = swapped ? xb : xa;
        int64_t drop = swapped ? xa : xb;
        S1[i - 1] = (int32_t)keep;
        if (S2) S2[i - 1] = (int32_t)drop;
        if (diag) {
            diag[4 * (i - 1) + 0] = alpha;
            diag[4 * (i - 1) + 1] = a;
            diag[4 * (i - 1) + 2] = p;
            diag[4 * (i - 1) + 3] = swapped ? 1.0 : 0.0;
        }
        Mprev = M;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------ */
/* Offline-Compress2                                                                     */
/* ------------------------------------------------------------------------------------ */
/* R-delta */
void oracle_default_delta_levels(int m, double delta, double *out)
{
    for (int i = 0; i < m; ++i) out[i] = pow(4.0, (double)(i + 1 - m)) * delta / (3.0 * (double)m);
}

typedef struct {
    const float *K, *V;
    int d;
    double vmax;
    const double *delta_level;
    uint64_t seed;
    uint32_t head;
    double min_margin;     /* min_i |U_i - p_i| over all calls */
    double *call_log;      /* optional [cap][4]: level, call number, points in, delta used */
    int64_t call_log_cap, call_log_n;
} compress2_ctx;

/* One recursion of Offline-Compress2: `x` holds n_in = 2^m * n_out points; `level` counts
 * how many recursions came before (it selects Halve_level and the uniforms' counter). */
static int compress2_rec(compress2_ctx *c, int m, int level, int32_t *x, int64_t n_in)
{
    if (m == 0) return 0;                                   /* base case: unchanged */
    int64_t groups = (int64_t)1 << (2 * (m - 1));           /* 4^(m-1) */
    int64_t gs = n_in / groups;                             /* group size */
    if (gs * groups != n_in || gs < 2 || (gs & 1)) return -1;
    int32_t *next = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_in / 2));
    double *U = (double *)malloc(sizeof(double) * (size_t)(gs / 2));
    double *diag = (double *)malloc(sizeof(double) * 4 * (size_t)(gs / 2));
    if (!next || !U || !diag) { free(next); free(U); free(diag); return -2; }
    int rc = 0;
    for (int64_t g = 0; g < groups && rc == 0; ++g) {
        for (int64_t i = 0; i < gs / 2; ++i)
            U[i] = oracle_uniform(c->seed, (uint32_t)i, (uint32_t)g, (uint32_t)level, c->head);
        rc = oracle_kh(c->K, c->V, c->d, c->vmax, x + g * gs, (int)gs, c->delta_level[level],
                       1, U, next + g * (gs / 2), NULL, diag);
        if (c->call_log && c->call_log_n < c->call_log_cap) {
            double *r = c->call_log + 4 * c->call_log_n;
            r[0] = (double)level; r[1] = (double)g; r[2] = (double)gs; r[3] = c->delta_level[level];
        }
        c->call_log_n += 1;
        for (int64_t i = 0; i < gs / 2; ++i) {
            double mg = fabs(U[i] - diag[4 * i + 2]);
            if (mg < c->min_margin) c->min_margin = mg;
        }
    }
    if (rc == 0) {
        memcpy(x, next, sizeof(int32_t) * (size_t)(n_in / 2));   /* concatenation, group order */
        rc = compress2_rec(c, m - 1, level + 1, x, n_in / 2);
    }
    free(next); free(U); free(diag);
    return rc;
}

/*
 * Offline-Compress2(m, all n rows of one attention problem, KH) with n = 2^m * n_out.
 * idx_out[n_out] receives the coreset rows (R-order), w_out[n_out] the weights 1/n_out
 * (positive, summing to 1).  delta_level[m] may be NULL (R-delta with `delta`).
 * min_margin (optional) receives min |U - p| over every decision taken.
 * call_log (optional, [call_log_cap][4]) receives one row per Halve call in the order the calls are
 * made: level, number of the call at its level, points in, delta used; call_log_count the number
 * of calls made (rows beyond the capacity are counted, not written).
 */
int oracle_compress2_calls(const float *K, const float *V, int64_t n, int d, int log2_nout, int m,
                           double delta, const double *delta_level, uint64_t seed, uint32_t head,
                           int32_t *idx_out, double *w_out, double *min_margin,
                           double *call_log, int64_t call_log_cap, int64_t *call_log_count)
{
    int64_t n_out = (int64_t)1 << log2_nout;
    if (m < 0 || n != (n_out << m)) return -1;
    double *dl = (double *)malloc(sizeof(double) * (size_t)(m > 0 ? m : 1));
    int32_t *x = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    if (!dl || !x) { free(dl); free(x); return -2; }
    if (delta_level) memcpy(dl, delta_level, sizeof(double) * (size_t)m);
    else oracle_default_delta_levels(m, delta, dl);
    for (int64_t i = 0; i < n; ++i) x[i] = (int32_t)i;
    compress2_ctx c = { K, V, d, oracle_vmax(V, n, d), dl, seed, head, 2.0, call_log, call_log_cap, 0 };
    int rc = compress2_rec(&c, m, 0, x, n);
    if (rc == 0) {
        for (int64_t i = 0; i < n_out; ++i) { idx_out[i] = x[i]; w_out[i] = 1.0 / (double)n_out; }
        if (min_margin) *min_margin = c.min_margin;
        if (call_log_count) *call_log_count = c.call_log_n;
    }
    free(dl); free(x);
    return rc;
}

int oracle_compress2(const float *K, const float *V, int64_t n, int d, int log2_nout, int m,
                     double delta, const double *delta_level, uint64_t seed, uint32_t head,
                     int32_t *idx_out, double *w_out, double *min_margin)
{
    return oracle_compress2_calls(K, V, n, d, log2_nout, m, delta, delta_level, seed, head, idx_out, w_out,
                                  min_margin, NULL, 0, NULL);
}

/* The same for `problems` independent attention problems laid out back to back
 * ([problems][n][d]); problem p draws its uniforms with head counter p. */
int oracle_compress2_batched(const float *K, const float *V, int problems, int64_t n, int d,
                             int log2_nout, int m, double delta, const double *delta_level,
                             uint64_t seed, int32_t *idx_out, double *w_out, double *min_margin)
{
    int64_t n_out = (int64_t)1 << log2_nout;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int p = 0; p < problems; ++p) {
        double mg = 2.0;
        int rc = oracle_compress2(K + (int64_t)p * n * d, V + (int64_t)p * n * d, n, d, log2_nout, m,
                                  delta, delta_level, seed, (uint32_t)p, idx_out + p * n_out,
                                  w_out + p * n_out, &mg);
        if (min_margin) min_margin[p] = mg;
        if (rc != 0) {
#pragma omp atomic write
            bad = rc;
        }
    }
    return bad;
}

/* ------------------------------------------------------------------------------------ */
/* Compress2 in its streaming form (Algorithm 2), for sequences of any length, with the  */
/* first n_sink and last n_window rows kept exactly.                                     */
/*                                                                                        */
/*   Compress2(m, n_in = 2^m n_out, Halve): S_0 <- S_0 + {x}; for i = 0..m-1: when S_i    */
/*   holds n_in 2^i / 4^(m-1) points, S_{i+1} <- S_{i+1} + Halve_i(S_i), S_i <- {}.        */
/*   wtd_cache() = [(S_i, 2^(i-m))]_{i=0..m}.                                              */
/*                                                                                        */
/* The middle rows n_sink .. n - n_window - 1 are fed one by one (at most n_in of them);  */
/* whatever has not been halved yet stays in its level with that level's weight.  The    */
/* sink and window rows carry the weight of a raw point, 2^-m.  Readings:                */
/*   R-norm    all weights are divided by their sum n 2^-m, so that they are positive and */
/*             sum to 1 (Definition 1): a point of S_i gets 2^i / n, a sink 1 / n.        */
/*   R-out     output order: sinks, S_0, S_1, ..., S_m (each in append order), window.    */
/*   R-vmax    v_max over all n rows of the problem.                                      */
/*   uniforms  as in oracle_compress2: counter (pair, number of the call at its level,    */
/*             level, head); with n = n_in and no sinks the result equals Offline-Compress2. */
/* ------------------------------------------------------------------------------------ */
int oracle_compress2_stream(const float *K, const float *V, int64_t n, int d, int log2_nout, int m,
                            double delta, const double *delta_level, uint64_t seed, uint32_t head,
                            int32_t n_sink, int32_t n_window, int32_t *idx_out, double *w_out,
                            int32_t capacity, int32_t *count)
{
    const int64_t n_out = (int64_t)1 << log2_nout;
    const int64_t n_in = n_out << m;
    const int64_t n_mid = n - n_sink - n_window;
    if (m < 0 || m > 30 || n_sink < 0 || n_window < 0 || n_mid < 0 || n_mid > n_in) return -1;
    if (m >= 1 && ((n_in >> (2 * (m - 1))) < 2)) return -1;            /* level-0 calls of at least one pair */
    double dl[32];
    if (delta_level) memcpy(dl, delta_level, sizeof(double) * (size_t)m);
    else oracle_default_delta_levels(m, delta, dl);
    const double vmax = oracle_vmax(V, n, d);
    int32_t *S[32];
    int64_t nS[32], calls[32], thresh[32];
    int rc = 0;
    for (int i = 0; i <= m; ++i) { S[i] = NULL; nS[i] = 0; calls[i] = 0; }
    for (int i = 0; i <= m; ++i) {
        thresh[i] = m >= 1 ? ((n_in << i) >> (2 * (m - 1))) : n_in + 1;
        /* S_i never holds more than its threshold (S_m: n_out points, or everything when m = 0) */
        const int64_t room = i < m ? thresh[i] : (m == 0 ? n_in : n_out);
        S[i] = (int32_t *)malloc(sizeof(int32_t) * (size_t)(room > 0 ? room : 1));
        if (!S[i]) rc = -2;
    }
    for (int64_t t = 0; t < n_mid && rc == 0; ++t) {
        S[0][nS[0]++] = (int32_t)(n_sink + t);                          /* update(x) */
        for (int i = 0; i < m && rc == 0; ++i) {
            if (nS[i] != thresh[i]) continue;
            const int64_t s = thresh[i];
            double *U = (double *)malloc(sizeof(double) * (size_t)(s / 2));
            if (!U) { rc = -2; break; }
            for (int64_t a = 0; a < s / 2; ++a)
                U[a] = oracle_uniform(seed, (uint32_t)a, (uint32_t)calls[i], (uint32_t)i, head);
            rc = oracle_kh(K, V, d, vmax, S[i], (int)s, dl[i], 1, U, S[i + 1] + nS[i + 1], NULL, NULL);
            free(U);
            calls[i] += 1;
            nS[i + 1] += s / 2;
            nS[i] = 0;
        }
    }
    if (rc == 0) {
        int64_t c = 0, total = n_sink + n_window;
        for (int i = 0; i <= m; ++i) total += nS[i];
        if (count) *count = (int32_t)total;
        if (total > capacity) rc = -3;
        if (rc == 0) {
            for (int32_t a = 0; a < n_sink; ++a) { idx_out[c] = a; w_out[c] = 1.0 / (double)n; ++c; }
            for (int i = 0; i <= m; ++i)
                for (int64_t a = 0; a < nS[i]; ++a) { idx_out[c] = S[i][a]; w_out[c] = ldexp(1.0, i) / (double)n; ++c; }
            for (int32_t a = 0; a < n_window; ++a) { idx_out[c] = (int32_t)(n - n_window + a); w_out[c] = 1.0 / (double)n; ++c; }
        }
    }
    for (int i = 0; i <= m; ++i) free(S[i]);
    return rc;
}

/* ------------------------------------------------------------------------------------ */
/* Weighted attention and exact attention                                                */
/* ------------------------------------------------------------------------------------ */
/*
 * O[j,:] = sum_c w_c exp(<q_j,k_c>/sqrt(d)) v_c / sum_c w_c exp(<q_j,k_c>/sqrt(d)),
 * c ranging over idx[0..n_core).  The row maximum of the exponent is subtracted in both
 * sums, which leaves the ratio unchanged.  Q is [nq][d]; K, V are the problem's full
 * [n][d] arrays; O is [nq][d] in double.
 */
int oracle_wtd_attention(const float *Q, const float *K, const float *V, const int32_t *idx,
                         const double *w, int n_core, int64_t nq, int d, double *O)
{
    if (n_core <= 0) return -1;
    const double rd = sqrt((double)d);
    double *e = (double *)malloc(sizeof(double) * (size_t)n_core);
    if (!e) return -2;
    for (int64_t j = 0; j < nq; ++j) {
        const float *q = Q + j * d;
        double mx = -INFINITY;
        for (int c = 0; c < n_core; ++c) {
            const float *k = K + (int64_t)idx[c] * d;
            double s = 0.0;
            for (int t = 0; t < d; ++t) s += (double)q[t] * (double)k[t];
            e[c] = s / rd;
            if (e[c] > mx) mx = e[c];
        }
        double den = 0.0;
        for (int t = 0; t < d; ++t) O[j * d + t] = 0.0;
        for (int c = 0; c < n_core; ++c) {
            double p = w[c] * exp(e[c] - mx);
            const float *v = V + (int64_t)idx[c] * d;
            den += p;
            for (int t = 0; t < d; ++t) O[j * d + t] += p * (double)v[t];
        }
        for (int t = 0; t < d; ++t) O[j * d + t] /= den;
    }
    free(e);
    return 0;
}

/* Exact unmasked attention of nq queries over all n key-value pairs (equal weights 1/n). */
int oracle_exact_attention(const float *Q, const float *K, const float *V, int64_t n, int64_t nq,
                           int d, double *O)
{
    const double rd = sqrt((double)d);
    double *e = (double *)malloc(sizeof(double) * (size_t)n);
    if (!e) return -2;
    for (int64_t j = 0; j < nq; ++j) {
        const float *q = Q + j * d;
        double mx = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            const float *k = K + i * d;
            double s = 0.0;
            for (int t = 0; t < d; ++t) s += (double)q[t] * (double)k[t];
            e[i] = s / rd;
            if (e[i] > mx) mx = e[i];
        }
        double den = 0.0;
        for (int t = 0; t < d; ++t) O[j * d + t] = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double p = exp(e[i] - mx) / (double)n;
            const float *v = V + i * d;
            den += p;
            for (int t = 0; t < d; ++t) O[j * d + t] += p * (double)v[t];
        }
        for (int t = 0; t < d; ++t) O[j * d + t] /= den;
    }
    free(e);
    return 0;
}

/*
 * Batched drivers over [problems_q] query heads; query head h reads KV problem
 * floor(h * problems_kv / problems_q) of its batch entry (grouped queries).
 * Layouts: Q,O [batch][q_heads][nq][d]; K,V [batch][kv_heads][n][d];
 * idx,w [batch][kv_heads][n_core].
 */
int oracle_wtd_attention_batched(const float *Q, const float *K, const float *V,
                                 const int32_t *idx, const double *w, int batch, int q_heads,
                                 int kv_heads, int64_t n, int64_t nq, int d, int n_core, double *O)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < batch * q_heads; ++bh) {
        int b = bh / q_heads, h = bh % q_heads;
        int kvh = (int)(((int64_t)h * kv_heads) / q_heads);
        int64_t kv = (int64_t)b * kv_heads + kvh;
        int rc = oracle_wtd_attention(Q + (int64_t)bh * nq * d, K + kv * n * d, V + kv * n * d,
                                      idx + kv * n_core, w + kv * n_core, n_core, nq, d,
                                      O + (int64_t)bh * nq * d);
        if (rc != 0) {
#pragma omp atomic write
            bad = rc;
        }
    }
    return bad;
}

int oracle_exact_attention_batched(const float *Q, const float *K, const float *V, int batch,
                                   int q_heads, int kv_heads, int64_t n, int64_t nq, int d, double *O)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < batch * q_heads; ++bh) {
        int b = bh / q_heads, h = bh % q_heads;
        int kvh = (int)(((int64_t)h * kv_heads) / q_heads);
        int64_t kv = (int64_t)b * kv_heads + kvh;
        int rc = oracle_exact_attention(Q + (int64_t)bh * nq * d, K + kv * n * d, V + kv * n * d, n,
                                        nq, d, O + (int64_t)bh * nq * d);
        if (rc != 0) {
#pragma omp atomic write
            bad = rc;
        }
    }
    return bad;
}

/* ------------------------------------------------------------------------------------ */
/* MMD^2 between the equal-weight set `in` and the weighted set (`out`, w):              */
/*   mean_{a,b in in} k(a,b) - 2 sum_{a in in} sum_{c in out} w_c k(a,c) / n_in          */
/*   + sum_{c,c' in out} w_c w_c' k(c,c'),  every k multiplied by exp(-shift).           */
/* ------------------------------------------------------------------------------------ */
double oracle_mmd2(const float *K, const float *V, int d, double vmax, const int32_t *in, int n_in,
                   const int32_t *out, const double *w, int n_out, double shift)
{
    double t_in = 0.0, t_x = 0.0, t_out = 0.0;
    for (int a = 0; a < n_in; ++a)
        for (int b = 0; b < n_in; ++b)
            t_in += oracle_katt(K, V, d, vmax, in[a], in[b], shift, 0);
    for (int a = 0; a < n_in; ++a)
        for (int c = 0; c < n_out; ++c)
            t_x += w[c] * oracle_katt(K, V, d, vmax, in[a], out[c], shift, 0);
    for (int c = 0; c < n_out; ++c)
        for (int e = 0; e < n_out; ++e)
            t_out += w[c] * w[e] * oracle_katt(K, V, d, vmax, out[c], out[e], shift, 0);
    return t_in / ((double)n_in * (double)n_in) - 2.0 * t_x / (double)n_in + t_out;
}

/* ------------------------------------------------------------------------------------ */
/* Express / KH-Express / Thinformer Express: Algorithms 1-5 and Corollary 2, streaming.   */
/* One update per point, exactly in the order the algorithms state.                        */
/*                                                                                          */
/* Readings (beyond those at the top of this file):                                        */
/*   R-vmax-causal  v_max of Eq. (katt) is taken over the whole observed sequence (the      */
/*                  prefill setting: every token is known in advance).                     */
/*   R-ctr          uniforms: Philox counter (pair, call number at that level of the       */
/*                  current Compress2 instance, code, problem) with                        */
/*                    code = level i + 64 (4 r + j)   Halve_i of sibling j in {1,2,3} of     */
/*                                                    round r = m/2,                        */
/*                    code = 62 + h + 64 (4 r)        h-th of the two E halvings of round r, */
/*                    code = 61 + 64 (4 r + j)        Subsample of sibling j, counter word 0 */
/*                                                    = stratum number.                    */
/*   R-unif-int     Unif([n, n + 2^(m-mbar))) = n + floor(U 2^(m-mbar)), U the 24-bit uniform. */
/* ------------------------------------------------------------------------------------ */
typedef struct {
    /* problem */
    const float *K, *V;
    int d;
    double vmax, delta;
    uint64_t seed;
    uint32_t head;
    int64_t n_out;
    int mbar;
    /* Express state (Algorithm 1) */
    int m;              /* thinning factor */
    int64_t n, ell;
    int32_t *E;
    int64_t nE;
    int b;              /* completed thin phases since the last halve phase */
    /* Subsample(m, mbar) state (Algorithm 3) */
    int64_t s_n, s_i;
    /* Compress2(q, 2^q n_out, Halve_m) state (Algorithm 2) */
    int q;
    int32_t *S[40];
    int64_t nS[40];
    int64_t calls[40];
    int64_t halve_calls;   /* total KH calls made (cost accounting) */
    double *halve_log;     /* optional [cap][5]: thinning factor m, level i (-1, -2: first, second halving
                              of E), points in, delta used, sibling j (0 for E) */
    int64_t halve_log_cap;
} express_state;

static double kh_express_delta_m(double delta, int m)
{
    return 0.5 * delta * (1.0 / log2(0.5 * m + 2.0) - 1.0 / log2(0.5 * m + 3.0));
}

static void express_reset_thin(express_state *st)
{
    st->s_n = 0;
    st->s_i = 0;
    st->q = st->m < st->mbar ? st->m : st->mbar;
    for (int i = 0; i <= st->q; ++i) { st->nS[i] = 0; st->calls[i] = 0; }
}

static int express_halve(express_state *st, int32_t *x, int64_t s, double dlt, uint32_t code, uint32_t call,
                         int32_t *out, int level)
{
    if (st->halve_log && st->halve_calls < st->halve_log_cap) {
        double *r = st->halve_log + 5 * st->halve_calls;
        r[0] = (double)st->m; r[1] = (double)level; r[2] = (double)s; r[3] = dlt;
        r[4] = level >= 0 ? (double)(st->b + 1) : 0.0;
    }
    double *U = (double *)malloc(sizeof(double) * (size_t)(s / 2));
    if (!U) return -2;
    for (int64_t i = 0; i < s / 2; ++i) U[i] = oracle_uniform(st->seed, (uint32_t)i, call, code, st->head);
    int rc = oracle_kh(st->K, st->V, st->d, st->vmax, x, (int)s, dlt, 1, U, out, NULL, NULL);
    free(U);
    st->halve_calls += 1;
    return rc;
}

/* Compress2.update(x) with Halve_i = KH(delta_{m,i}) */
static int express_compress2_update(express_state *st, int32_t x)
{
    const int q = st->q;
    const int64_t n_in = st->n_out << q;
    st->S[0][st->nS[0]++] = x;
    for (int i = 0; i < q; ++i) {
        const int64_t thresh = (n_in << i) >> (2 * (q - 1));            /* n_in 2^i / 4^(q-1) */
        if (st->nS[i] == thresh) {
            const double dm = kh_express_delta_m(st->delta, st->m);
            const double dlt = pow(4.0, (double)(i + 1 - q)) * dm / (3.0 * (double)q);
            const uint32_t code = (uint32_t)i + 64u * (uint32_t)(4 * (st->m / 2) + st->b + 1);
            int rc = express_halve(st, st->S[i], thresh, dlt, code, (uint32_t)st->calls[i], st->S[i + 1] + st->nS[i + 1], i);
            if (rc != 0) return rc;
            st->calls[i] += 1;
            st->nS[i + 1] += thresh / 2;
            st->nS[i] = 0;
        }
    }
    return 0;
}

/* Subsample.keep(x) */
static int express_subsample_keep(express_state *st)
{
    st->s_n += 1;
    if (st->m <= st->mbar) return 1;
    const int64_t w = (int64_t)1 << (st->m - st->mbar);
    if ((st->s_n - 1) % w == 0) {
        const uint32_t code = 61u + 64u * (uint32_t)(4 * (st->m / 2) + st->b + 1);
        const double U = oracle_uniform(st->seed, (uint32_t)((st->s_n - 1) / w), 0u, code, st->head);
        st->s_i = st->s_n + (int64_t)floor(U * (double)w);
    }
    return st->s_n == st->s_i;
}

/* Express.update(x) */
static int express_update(express_state *st, int32_t x)
{
    st->n += 1;
    if (st->n <= st->n_out) { st->E[st->nE++] = x; return 0; }          /* exact phase */
    st->ell += 1;                                                        /* thin phase */
    if (express_subsample_keep(st)) {
        int rc = express_compress2_update(st, x);
        if (rc != 0) return rc;
    }
    if (st->ell == (st->n_out << st->m)) {
        for (int64_t i = 0; i < st->nS[st->q]; ++i) st->E[st->nE++] = st->S[st->q][i];
        st->nS[st->q] = 0;
        st->ell = 0;
        st->b += 1;
    }
    if (st->n == 4 * (st->n_out << st->m)) {                             /* halve phase */
        const double dm = kh_express_delta_m(st->delta, st->m);
        int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)(2 * st->n_out));
        if (!tmp) return -2;
        int rc = express_halve(st, st->E, 4 * st->n_out, 0.5 * dm, 62u + 64u * (uint32_t)(4 * (st->m / 2)), 0u, tmp, -1);
        if (rc == 0) rc = express_halve(st, tmp, 2 * st->n_out, 0.5 * dm, 63u + 64u * (uint32_t)(4 * (st->m / 2)), 0u, st->E, -2);
        free(tmp);
        if (rc != 0) return rc;
        st->nE = st->n_out;
        st->m += 2;
        st->b = 0;
    }
    if (st->ell == 0) express_reset_thin(st);
    return 0;
}

/*
 * Thinformer Express over one attention problem: for t = 1..n
 *     o_t = WtdAttention((q_t, k_t, v_t), C)   then   C.update((k_t, v_t)).
 * Outputs (each may be NULL):
 *   O[n][d]          the attention outputs
 *   cache_size[n]    points in wtd_cache() when token t arrives (the input token not counted)
 *   final_idx/final_w/final_count  wtd_cache() after the last update (capacity 6 n_out)
 *   halve_calls      number of KH calls made
 *   halve_log        [halve_log_cap][5], one row per KH call in the order made: thinning factor m of
 *                    the round, level i of the Compress2 call (-1 / -2 for the first / second halving
 *                    of the Express coreset), points in, delta used, sibling (1..3; 0 for E)
 */
int oracle_thinformer_express_log(const float *Q, const float *K, const float *V, int64_t n, int d, int log2_nout,
                                  int mbar, double delta, uint64_t seed, uint32_t head, double *O,
                                  int32_t *cache_size, int32_t *final_idx, double *final_w, int32_t *final_count,
                                  int64_t *halve_calls, double *halve_log, int64_t halve_log_cap)
{
    if (log2_nout < 0 || mbar < 0 || !(delta > 0.0 && delta < 1.0)) return -1;
    express_state st;
    memset(&st, 0, sizeof(st));
    st.K = K; st.V = V; st.d = d; st.delta = delta; st.seed = seed; st.head = head;
    st.n_out = (int64_t)1 << log2_nout;
    st.mbar = mbar;
    st.halve_log = halve_log; st.halve_log_cap = halve_log_cap;
    st.vmax = oracle_vmax(V, n, d);                                       /* R-vmax-causal */
    st.E = (int32_t *)malloc(sizeof(int32_t) * (size_t)(4 * st.n_out));
    int rc = st.E ? 0 : -2;
    for (int i = 0; i <= mbar && rc == 0; ++i) {
        /* level i of any Compress2(q <= mbar) holds at most max(n_out 2^(2-q+i), n_out) points */
        st.S[i] = (int32_t *)malloc(sizeof(int32_t) * (size_t)(4 * st.n_out));
        if (!st.S[i]) rc = -2;
    }
    const int64_t cap = 6 * st.n_out + 1;
    int32_t *cidx = (int32_t *)malloc(sizeof(int32_t) * (size_t)cap);
    double *cw = (double *)malloc(sizeof(double) * (size_t)cap);
    float *qrow = NULL;
    if (!cidx || !cw) rc = -2;
    if (rc == 0) express_reset_thin(&st);
    for (int64_t t = 0; t < n && rc == 0; ++t) {
        /* wtd_cache(): [(S_i, 2^(i-q))]_{i=0..q} then (E, 1) */
        int64_t c = 0;
        for (int i = 0; i <= st.q; ++i)
            for (int64_t a = 0; a < st.nS[i]; ++a) { cidx[c] = st.S[i][a]; cw[c] = ldexp(1.0, i - st.q); ++c; }
        for (int64_t a = 0; a < st.nE; ++a) { cidx[c] = st.E[a]; cw[c] = 1.0; ++c; }
        if (cache_size) cache_size[t] = (int32_t)c;
        if (O) {
            /* incorporate the input token into S_0 (weight 2^(-q)) and attend */
            cidx[c] = (int32_t)t; cw[c] = ldexp(1.0, -st.q); ++c;
            rc = oracle_wtd_attention(Q + t * d, K, V, cidx, cw, (int)c, 1, d, O + t * d);
            if (rc != 0) break;
        }
        rc = express_update(&st, (int32_t)t);
    }
    if (rc == 0) {
        int64_t c = 0;
        for (int i = 0; i <= st.q; ++i)
            for (int64_t a = 0; a < st.nS[i]; ++a) {
                if (final_idx) final_idx[c] = st.S[i][a];
                if (final_w) final_w[c] = ldexp(1.0, i - st.q);
                ++c;
            }
        for (int64_t a = 0; a < st.nE; ++a) {
            if (final_idx) final_idx[c] = st.E[a];
            if (final_w) final_w[c] = 1.0;
            ++c;
        }
        if (final_count) *final_count = (int32_t)c;
        if (halve_calls) *halve_calls = st.halve_calls;
    }
    free(st.E);
    for (int i = 0; i <= mbar; ++i) free(st.S[i]);
    free(cidx); free(cw); free(qrow);
    return rc;
}

int oracle_thinformer_express(const float *Q, const float *K, const float *V, int64_t n, int d, int log2_nout,
                              int mbar, double delta, uint64_t seed, uint32_t head, double *O,
                              int32_t *cache_size, int32_t *final_idx, double *final_w, int32_t *final_count,
                              int64_t *halve_calls)
{
    return oracle_thinformer_express_log(Q, K, V, n, d, log2_nout, mbar, delta, seed, head, O, cache_size,
                                         final_idx, final_w, final_count, halve_calls, NULL, 0);
}

/* Exact causal attention, Eq. (def:att): query t over the pairs 1..t. */
int oracle_exact_causal_attention(const float *Q, const float *K, const float *V, int64_t n, int d, double *O)
{
    int rc = 0;
    for (int64_t t = 0; t < n && rc == 0; ++t) rc = oracle_exact_attention(Q + t * d, K, V, t + 1, 1, d, O + t * d);
    return rc;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
