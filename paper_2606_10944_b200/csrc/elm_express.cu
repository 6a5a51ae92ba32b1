// Offline-Express compression and Thinformer Express in prefill (elm_express_compress, elm_express_prefill).
#include "elm_level.cuh"
#include "elm_prefill_round.cuh"

namespace elm {

// ---------------------------------------------------------------------------------------------
// Offline-Express: the cache a streaming Express run (Algorithm 1, with Subsample, Algorithm 3, and
// Compress2, Algorithm 2, inside, Halve = KH with the failure parameters of Corollary 2) holds after
// n = n_out 4^R points, computed by the equivalent recursion: E = first n_out points; round r
// (thinning factor m = 2r) thins the next three segments of n_out 2^m points each - one stratified
// draw per 2^(m - mbar) points when m > mbar, then Compress2 of depth min(m, mbar) - appends the three
// results to E and halves E twice.  Every Halve call runs through the same level machinery as
// elm_compress; the uniforms' counter words follow the call structure of the streaming run:
//   third word = level i + 64 (4 r + j)    Halve_i inside sibling j in {1, 2, 3} of round r,
//                62 / 63 + 64 (4 r)        the two halvings of E,
//                61 + 64 (4 r + j)         the stratified draws of sibling j (first word = stratum).
// v_max is taken over the whole sequence.
// ---------------------------------------------------------------------------------------------
constexpr int EXPRESS_LANES = 6;       // side streams of the prefill: two per sibling segment
struct ExpressLayout {
    size_t vmax_bits, cnorm, listA, listB, E, T1, Mpair, rdecay, F, F_stride, total;
    // the halvings of E run beside the next round's compression, on a stream and with scratch of their own; E itself
    // alternates between two buffers (round r reads one, its halvings write the other)
    size_t E2, Mpair2, rdecay2, F2;
    // prefill only: the output lists of every Compress2 level of a round; per side stream the cache list
    // of one launch with its weights and lifetimes and the workspace of elm_attend for that list; log2 of
    // the softmax denominators (rounds with Subsample: the tokens that were not kept are merged in afterwards)
    size_t levels, ep_idx, ep_w, ep_birth, ep_death, ep_blk, ws_attend, ep_cap, ep_pad, ep_stride, ws_attend_stride, lse;
    int n_levels;
    // prefill, rounds that take one attention launch: the round's universe and tile table (elm_prefill_round.cuh)
    size_t round;
    RoundBufferLayout rbl;
};
// Tokens per attention launch of the prefill: windows of about 512 tokens (whole strata, at most a segment).
static int64_t prefill_window(const RoundGeom &g)
{
    static const int64_t target = []() {
        const char *e = getenv("ELM_PREFILL_WINDOW");           // tuning aid: a power of two
        const long v = e ? atol(e) : 0;
        return (int64_t)(v >= 64 && (v & (v - 1)) == 0 ? v : 512);
    }();
    int64_t W = (int64_t)1 << g.wlog;
    if (W < target) W = target;
    return W < g.seg ? W : g.seg;
}

// The cache entries some token of a window can see, as runs of the round's point lists, each entry with
// the span of tokens that see it.  In terms of G = the number of kept points of the sibling segment
// that have arrived (a window covers G in [G0, G1)):
//   kind 0   E and the finished siblings: always
//   kind 1   S_i, 1 <= i < q: the output of call c of level i - 1 (u entries) exists from G = (c + 1) A,
//            A = s0 4^(i-1), until the level-i call that consumes it completes at G = (c / 4 + 1) 4 A
//   kind 2   S_0: kept point g exists from its own token (which sees itself) until G = (g / s0 + 1) s0
//   kind 3   S_q: the output of the segment's last call, from G = len0 on
// G = X is reached right after the X-th kept point: at token kept[X - 1] + 1.
struct WindowPieces {
    const int32_t *src[16];
    int64_t src_off[16];
    int64_t first[16];          // kind 1: index of the run's first entry within the sibling's part of the list; kind 2: its g
    int64_t per_call[16];       // kind 1: A
    int32_t dst_off[17];
    int32_t unit[16];           // kind 1: u; kind 2: s0
    float w[16];
    int8_t kind[16];
    int n;
    const int32_t *kept;        // kept points of the round's three siblings (the level-0 input list)
    int64_t kept_off, len0;
    int32_t q;
};
static int32_t window_pieces(const RoundGeom &g, int64_t n_out, int jj, int64_t G0, int64_t G1, const int32_t *E,
                             const int32_t *levels, size_t level_stride, const int32_t *kept, WindowPieces &pc)
{
    int k = 0;
    int32_t at = 0;
    auto piece = [&](const int32_t *src, int64_t off, int64_t count, double wgt, int kind, int64_t first, int64_t unit,
                     int64_t per_call) {
        if (count <= 0) return;
        pc.src[k] = src; pc.src_off[k] = off; pc.w[k] = (float)wgt; pc.dst_off[k] = at;
        pc.kind[k] = (int8_t)kind; pc.first[k] = first; pc.unit[k] = (int32_t)unit; pc.per_call[k] = per_call;
        at += (int32_t)count;
        ++k;
    };
    const int q = g.q;
    piece(E, 0, (1 + jj) * n_out, 1.0, 0, 0, 1, 1);
    for (int i = q - 1; i >= 1; --i) {
        const int64_t A = g.s0 << (2 * (i - 1)), u = (g.s0 << (i - 1)) >> 1;
        const int64_t c_lo = 4 * (G0 / (4 * A)), c_end = G1 / A;
        piece(levels ? levels + (size_t)(i - 1) * level_stride : nullptr, jj * (g.len0 >> i) + c_lo * u, (c_end - c_lo) * u,
              ldexp(1.0, i - q), 1, c_lo * u, u, A);
    }
    if (q >= 1 && g.sub && G1 >= g.len0) piece(E, (1 + jj) * n_out, n_out, 1.0, 3, 0, 1, 1);
    const int64_t g_lo = q >= 1 ? (G0 / g.s0) * g.s0 : 0;
    piece(kept, jj * g.len0 + g_lo, G1 - g_lo, ldexp(1.0, -q), 2, g_lo, g.s0, 1);
    pc.dst_off[k] = at;
    pc.n = k;
    pc.kept = kept;
    pc.kept_off = jj * g.len0;
    pc.len0 = g.len0;
    pc.q = q;
    return at;
}
// Longest cache list any launch of the prefill attends over.
static size_t express_list_cap(const elm_params *p, int mbar)
{
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    size_t cap = (size_t)(4 * n_out);                         // the exact start: causal attention over 4 n_out tokens
    const int R = [&]() { int64_t v = n_out; int r = 0; while (v < (int64_t)p->n_kv) { v *= 4; ++r; } return r; }();
    for (int r = 1; r < R; ++r) {
        const RoundGeom g = round_geom(p, mbar, r);
        const int64_t Wg = prefill_window(g) >> g.wlog;
        for (int jj = 0; jj < 3; ++jj)
            for (int64_t G0 = 0; G0 < g.len0; G0 += Wg) {
                WindowPieces pc;
                const size_t len = (size_t)window_pieces(g, n_out, jj, G0, G0 + Wg, nullptr, nullptr, 0, nullptr, pc);
                if (len > cap) cap = len;
            }
    }
    return cap;
}
static ExpressLayout express_layout(const elm_params *p, int mbar = 0, bool prefill = false)
{
    ExpressLayout L;
    const size_t ts = p->precision == ELM_PREC_FP64_DET ? 8 : 4;
    const size_t BH = (size_t)p->batch * p->kv_heads;
    const size_t n = (size_t)p->n_kv;
    const size_t n_out = (size_t)1 << p->log2_nout;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.vmax_bits = take((BH + 1) * 4);      // + one device status word
    L.cnorm = take(BH * n * ts);
    L.listA = take(BH * n * 4);
    L.listB = take(BH * n * 4);
    L.E = take(BH * n * 4);                // every point list is [BH][n]-strided, like the lists of elm_compress
    L.T1 = take(BH * n * 4);
    L.Mpair = take(BH * (n / 2 + 1) * ts);
    L.rdecay = take(BH * (n / 2 + 1) * ts);
    L.F_stride = 4 * n_out * n_out;        // the first halving of E is one call of 2 n_out pairs
    L.F = take(BH * L.F_stride * ts);
    L.E2 = take(BH * n * 4);
    L.Mpair2 = take(BH * (n / 2 + 1) * ts);       // (indexed with the problem stride n / 2, like Mpair)
    L.rdecay2 = take(BH * (n / 2 + 1) * ts);
    L.F2 = take(BH * L.F_stride * ts);
    L.levels = L.ep_idx = L.ep_w = L.ep_birth = L.ep_death = L.ep_blk = L.ws_attend = L.ep_cap = L.ep_pad = L.ep_stride = 0;
    L.ws_attend_stride = L.lse = 0;
    L.n_levels = 0;
    L.round = 0;
    L.rbl = RoundBufferLayout();
    if (prefill) {
        L.n_levels = mbar < 30 ? mbar : 30;
        L.levels = take((size_t)L.n_levels * BH * n * 4);
        L.ep_cap = express_list_cap(p, mbar);
        L.ep_pad = (L.ep_cap + 127) / 128 * 128;
        // one set per side stream: the launches of a round are spread over EXPRESS_LANES streams
        L.ep_stride = align_up(BH * L.ep_pad * 4, 256);
        L.ep_idx = take(EXPRESS_LANES * L.ep_stride);
        L.ep_w = take(EXPRESS_LANES * L.ep_stride);
        L.ep_birth = take(EXPRESS_LANES * L.ep_stride);
        L.ep_death = take(EXPRESS_LANES * L.ep_stride);
        L.ep_blk = take(EXPRESS_LANES * L.ep_stride);          // two arrays of [BH][ep_pad / 128]
        L.lse = take((size_t)p->batch * p->q_heads * n * 4);
        L.ws_attend_stride = align_up(attend_layout(p, (int32_t)L.ep_cap).total, 256);
        L.ws_attend = take(EXPRESS_LANES * L.ws_attend_stride);
        int R = 0;
        for (size_t v = n_out; v < n; v *= 4) ++R;
        L.rbl = round_buffer_layout(p, mbar, R);
        L.round = take(L.rbl.total);
    }
    L.total = off;
    return L;
}

// The list of one prefill window (see WindowPieces): indices, weights, and for every entry the first
// token that sees it (birth) and the first that does not any more (death); per block of 128 entries the
// largest birth and the smallest death.  Entries beyond the list (up to n_pad) are given the lifetime
// "always": the attention kernel hides them by other means.
__global__ void __launch_bounds__(256) build_window_kernel(WindowPieces pc, int64_t src_stride, int32_t *__restrict__ idx,
                                                           float *__restrict__ w, int n_core, int n_pad,
                                                           int32_t *__restrict__ birth, int32_t *__restrict__ death,
                                                           int32_t *__restrict__ blk_birth, int32_t *__restrict__ blk_death)
{
    __shared__ int32_t sb[8], sd[8];
    const int i = blockIdx.x * 256 + threadIdx.x;
    const int64_t pr = blockIdx.y;
    int32_t bt = 0, dt = 0x7fffffff;
    if (i < n_core) {
        int k = 0;
        while (i >= pc.dst_off[k + 1]) ++k;
        const int64_t o = i - pc.dst_off[k];
        const int32_t *kept = pc.kept + pr * src_stride + pc.kept_off;
        auto token_after = [&](int64_t X) { return X > pc.len0 ? 0x7fffffff : kept[X - 1] + 1; };   // G = X is reached
        idx[pr * n_core + i] = pc.src[k][pr * src_stride + pc.src_off[k] + o];
        w[pr * n_core + i] = pc.w[k];
        if (pc.kind[k] == 1) {
            const int64_t c = (pc.first[k] + o) / pc.unit[k];
            bt = token_after((c + 1) * pc.per_call[k]);
            dt = token_after((c / 4 + 1) * 4 * pc.per_call[k]);
        } else if (pc.kind[k] == 2) {
            const int64_t g = pc.first[k] + o;
            bt = kept[g];
            if (pc.q >= 1) dt = token_after((g / pc.unit[k] + 1) * pc.unit[k]);
        } else if (pc.kind[k] == 3) {
            bt = token_after(pc.len0);
        }
    }
    if (i < n_pad) {
        birth[pr * n_pad + i] = bt;
        death[pr * n_pad + i] = dt;
    }
    int32_t bm = bt, dm = dt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        bm = max(bm, __shfl_xor_sync(0xffffffffu, bm, o));
        dm = min(dm, __shfl_xor_sync(0xffffffffu, dm, o));
    }
    if ((threadIdx.x & 31) == 0) { sb[threadIdx.x >> 5] = bm; sd[threadIdx.x >> 5] = dm; }
    __syncthreads();
    if (threadIdx.x < 2) {
        const int blk = blockIdx.x * 2 + threadIdx.x, h = threadIdx.x * 4;
        if (blk < n_pad / 128) {
            blk_birth[pr * (n_pad / 128) + blk] = max(max(sb[h], sb[h + 1]), max(sb[h + 2], sb[h + 3]));
            blk_death[pr * (n_pad / 128) + blk] = min(min(sd[h], sd[h + 1]), min(sd[h + 2], sd[h + 3]));
        }
    }
}

// Rounds with Subsample: a token that was not kept is in no list, but Algorithm 5 still lets it attend to
// itself with the weight of a point of S_0.  One warp per (head, token): merges that single term into the
// output row, given log2 of the row's denominator over the cache.
template <typename Tin, typename T>
__global__ void __launch_bounds__(256) self_merge_kernel(const Tin *__restrict__ Q, const Tin *__restrict__ K,
                                                         const Tin *__restrict__ V, Tin *__restrict__ O,
                                                         const float *__restrict__ lse, const int32_t *__restrict__ kept,
                                                         int q_heads, int kv_heads, int64_t n, int d, int64_t seg,
                                                         int64_t len0, int wlog, T log2w)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t rel = (int64_t)blockIdx.x * 8 + warp;                   // token within the round's 3 segments
    if (rel >= 3 * seg) return;
    const int bh = blockIdx.y;
    const int64_t prob = (int64_t)(bh / q_heads) * kv_heads + ((int64_t)(bh % q_heads) * kv_heads) / q_heads;
    const int64_t t = seg + rel, jj = rel / seg, stratum = (rel % seg) >> wlog;
    if (kept[prob * n + jj * len0 + stratum] == (int32_t)t) return;        // a kept token is an entry of S_0
    const Tin *q = Q + ((int64_t)bh * n + t) * d, *k = K + (prob * n + t) * d, *v = V + (prob * n + t) * d;
    Tin *o = O + ((int64_t)bh * n + t) * d;
    T dot = 0;
    for (int e = lane; e < d; e += 32) dot += load_as<T>(q, e) * load_as<T>(k, e);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
    const T sc = dot * (T)(1.4426950408889634 / sqrt((double)d)) + log2w;
    const T L = (T)lse[(int64_t)bh * n + t];
    const T M = sc > L ? sc : L;
    const T a = (T)exp2((T)(L - M)), b = (T)exp2((T)(sc - M));
    const T inv = (T)1 / (a + b);
    for (int e = lane; e < d; e += 32) store_from(o, e, (a * load_as<T>(o, e) + b * load_as<T>(v, e)) * inv);
}

// Launch-side state of one side stream of the prefill.
struct PrefillLane {
    int32_t *idx, *birth, *death, *blk_birth, *blk_death;
    float *w;
    unsigned char *ws_attend;
};
static PrefillLane prefill_lane(const ExpressLayout &L, unsigned char *ws, int BH, int lane)
{
    PrefillLane pl;
    pl.idx = reinterpret_cast<int32_t *>(ws + L.ep_idx + lane * L.ep_stride);
    pl.w = reinterpret_cast<float *>(ws + L.ep_w + lane * L.ep_stride);
    pl.birth = reinterpret_cast<int32_t *>(ws + L.ep_birth + lane * L.ep_stride);
    pl.death = reinterpret_cast<int32_t *>(ws + L.ep_death + lane * L.ep_stride);
    pl.blk_birth = reinterpret_cast<int32_t *>(ws + L.ep_blk + lane * L.ep_stride);
    pl.blk_death = pl.blk_birth + (size_t)BH * (L.ep_pad / 128);
    pl.ws_attend = ws + L.ws_attend + lane * L.ws_attend_stride;
    return pl;
}

static RoundBuffers round_buffers(const ExpressLayout &L, unsigned char *ws, int BH, int64_t n_univ)
{
    unsigned char *rw = ws + L.round;
    RoundBuffers rb;
    rb.idx = reinterpret_cast<int32_t *>(rw + L.rbl.idx);
    rb.w = reinterpret_cast<float *>(rw + L.rbl.w);
    rb.birth = reinterpret_cast<int32_t *>(rw + L.rbl.birth);
    rb.death = reinterpret_cast<int32_t *>(rw + L.rbl.death);
    rb.blk_birth = reinterpret_cast<int32_t *>(rw + L.rbl.blk);
    rb.blk_death = rb.blk_birth + (size_t)BH * (n_univ / 128);
    rb.tile_cnt = reinterpret_cast<int32_t *>(rw + L.rbl.tile_cnt);
    rb.tile_blk = reinterpret_cast<int32_t *>(rw + L.rbl.tile_blk);
    rb.item_tab = reinterpret_cast<int32_t *>(rw + L.rbl.item_tab);
    rb.item_cnt = reinterpret_cast<int32_t *>(rw + L.rbl.item_cnt);
    rb.item_cap = L.rbl.item_cap;
    rb.item_ctas = L.rbl.item_ctas;
    rb.ws_attend = rw + L.rbl.ws_attend;
    return rb;
}

// The exact start of Thinformer Express (Algorithm 5) in prefill: token t < rows attends over the tokens 0 .. t.
static int express_attend_start(const void *Q, const void *K, const void *V, void *O, const elm_params *p, const ExpressLayout &L,
                                unsigned char *ws, int rows, cudaStream_t st)
{
    const int BH = p->batch * p->kv_heads;
    const PrefillLane pl = prefill_lane(L, ws, BH, 0);
    if ((size_t)rows > L.ep_cap) return ELM_ERR_WORKSPACE;
    ListPieces pc = {};
    pc.n = 1;
    pc.src[0] = nullptr; pc.src_off[0] = 0; pc.w[0] = 1.f;
    pc.dst_off[0] = 0; pc.dst_off[1] = rows;
    build_list_kernel<<<dim3((unsigned)((rows + 255) / 256), (unsigned)BH), 256, 0, st>>>(pc, p->n_kv, pl.idx, pl.w, rows);
    count_launches(1);
    ELM_CUDA_TRY(cudaGetLastError());
    elm_params pe = *p;
    pe.n_q = rows;
    AttendWindow win;
    win.q_row0 = 0;
    win.n_q_total = p->n_kv;
    win.tail_start = 0;                  // the whole list is the causal tail
    if (L.rbl.total) {
        // (the run has the tile table of the one-launch rounds: pairs of query tiles stop at their own last token)
        const int rc = causal_tile_table(rows, p->batch * p->q_heads, round_buffers(L, ws, BH, 0), win, st);
        if (rc != ELM_OK) return rc;
    }
    return attend_enqueue(Q, K, V, pl.idx, pl.w, rows, &pe, O, pl.ws_attend, st, win);
}

// Attention of the tokens [t0, t0 + rows) over the entries of `pc`, each seen by the tokens of its lifetime.
static int express_attend_window(const void *Q, const void *K, const void *V, void *O, const elm_params *p,
                                 const ExpressLayout &L, unsigned char *ws, const WindowPieces &pc, int64_t t0, int rows,
                                 float *lse, cudaStream_t st, int lane)
{
    const int BH = p->batch * p->kv_heads;
    const int total = pc.dst_off[pc.n];
    const int n_pad = (total + 127) / 128 * 128;
    if ((size_t)total > L.ep_cap) return ELM_ERR_WORKSPACE;
    const PrefillLane pl = prefill_lane(L, ws, BH, lane);
    int32_t *blk_death = pl.blk_birth + (size_t)BH * (n_pad / 128);
    build_window_kernel<<<dim3((unsigned)((n_pad + 255) / 256), (unsigned)BH), 256, 0, st>>>(
        pc, p->n_kv, pl.idx, pl.w, total, n_pad, pl.birth, pl.death, pl.blk_birth, blk_death);
    count_launches(1);
    ELM_CUDA_TRY(cudaGetLastError());
    elm_params pe = *p;
    pe.n_q = rows;
    AttendWindow win;
    win.q_row0 = t0;
    win.n_q_total = p->n_kv;
    win.birth = pl.birth;
    win.death = pl.death;
    win.blk_birth = pl.blk_birth;
    win.blk_death = blk_death;
    win.lse = lse;
    return attend_enqueue(Q, K, V, pl.idx, pl.w, total, &pe, O, pl.ws_attend, st, win);
}

template <typename Tin, typename T>
static int express_impl(const Tin *K, const Tin *V, const elm_params *p, int mbar, uint64_t seed, int32_t *idx_out,
                        float *w_out, unsigned char *ws, cudaStream_t st, uint32_t pbase, const Tin *Q = nullptr,
                        Tin *O = nullptr)
{
    const bool prefill = Q != nullptr;
    const ExpressLayout L = express_layout(p, mbar, prefill);
    const int BH = p->batch * p->kv_heads;
    const int64_t n = p->n_kv;
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    const int R = express_rounds(p);
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
    int32_t *listA = reinterpret_cast<int32_t *>(ws + L.listA);
    int32_t *listB = reinterpret_cast<int32_t *>(ws + L.listB);
    int32_t *E = reinterpret_cast<int32_t *>(ws + L.E);
    int32_t *T1 = reinterpret_cast<int32_t *>(ws + L.T1);
    auto blocks = [](int64_t count) { return (unsigned)((count + 255) / 256); };
    {
        StageTimer t(ELM_STAGE_PREPASS, st, 2);
        ELM_CUDA_TRY(cudaMemsetAsync(c.vmax_bits, 0, (size_t)(BH + 1) * 4, st));
        prepass_kernel<Tin, T><<<dim3(blocks(n), (unsigned)BH), 256, 0, st>>>(K, V, n, p->d, c.cnorm, c.vmax_bits, listA);
        range_kernel<<<dim3(blocks(n_out), (unsigned)BH), 256, 0, st>>>(E, n, 0, 0, n_out);      // exact phase
        count_launches(2);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    int32_t *levels = reinterpret_cast<int32_t *>(ws + L.levels);
    struct SideStreams {                                             // released on every return path
        cudaStream_t s[EXPRESS_LANES] = {};
        cudaEvent_t fork = nullptr, join[EXPRESS_LANES] = {};
        cudaStream_t halve = nullptr;                                // the halvings of E
        cudaEvent_t ready[16] = {}, halved[16] = {};                 // per round: E and the siblings' outputs complete; E halved
        ~SideStreams()
        {
            for (int i = 0; i < EXPRESS_LANES; ++i) {
                if (s[i]) cudaStreamDestroy(s[i]);                   // work already enqueued still completes
                if (join[i]) cudaEventDestroy(join[i]);
            }
            if (fork) cudaEventDestroy(fork);
            if (halve) cudaStreamDestroy(halve);
            for (int i = 0; i < 16; ++i) {
                if (ready[i]) cudaEventDestroy(ready[i]);
                if (halved[i]) cudaEventDestroy(halved[i]);
            }
        }
    } sides;
    cudaStream_t *side = sides.s;
    cudaEvent_t &fork = sides.fork;
    cudaEvent_t *join = sides.join;
    if (prefill && R >= 2) {
        ELM_CUDA_TRY(cudaEventCreateWithFlags(&fork, cudaEventDisableTiming));
        for (int i = 0; i < EXPRESS_LANES; ++i) {
            ELM_CUDA_TRY(cudaStreamCreateWithFlags(&side[i], cudaStreamNonBlocking));
            ELM_CUDA_TRY(cudaEventCreateWithFlags(&join[i], cudaEventDisableTiming));
        }
    }
    // The two halvings of E that end round r (serial chains that keep at most a few dozen SMs busy) run on a stream of
    // their own beside the compression of round r + 1's segments, which does not depend on E; E alternates between
    // two buffers so that round r + 1's segments can deliver their outputs while round r's E is still being read.
    int32_t *Ebuf[2] = {E, reinterpret_cast<int32_t *>(ws + L.E2)};
    LevelCtx<Tin, T> ch = c;
    ch.Mpair = reinterpret_cast<T *>(ws + L.Mpair2);
    ch.rdecay = reinterpret_cast<T *>(ws + L.rdecay2);
    ch.F = reinterpret_cast<T *>(ws + L.F2);
    if (R >= 1) {
        ELM_CUDA_TRY(cudaStreamCreateWithFlags(&sides.halve, cudaStreamNonBlocking));
        for (int r = 0; r < R && r < 16; ++r) {
            ELM_CUDA_TRY(cudaEventCreateWithFlags(&sides.ready[r], cudaEventDisableTiming));
            ELM_CUDA_TRY(cudaEventCreateWithFlags(&sides.halved[r], cudaEventDisableTiming));
        }
    }
    ch.st = sides.halve;
    if (prefill) {
        // Exact phase and round 0 (thinning factor 1: nothing is dropped): each of the first 4 n_out
        // tokens attends over all tokens up to itself (Theorem 3's exact regime).
        const int rc = express_attend_start(Q, K, V, O, p, L, ws, (int)(n < 4 * n_out ? n : 4 * n_out), st);
        if (rc != ELM_OK) return rc;
    }
    for (int r = 0; r < R; ++r) {
        int32_t *const Er = Ebuf[r & 1], *const Enext = Ebuf[(r + 1) & 1];   // this round's E; where its halvings put the next
        const int m = 2 * r, q = m < mbar ? m : mbar;
        const int64_t seg = n_out << m, len0 = n_out << q;
        const double dm = kh_express_delta(p->delta, m);
        // The three sibling segments of the round are thinned together: their point lists are laid
        // side by side, every level holds the calls of all three (call_counter keeps their uniforms
        // apart), and the last level leaves their 3 n_out survivors behind the n_out points of E.
        const int code1 = 64 * (4 * r + 1);                                   // sibling 1; siblings 2, 3 are 64 apart
        if (m > mbar)
            subsample_kernel<<<dim3(blocks(3 * len0), (unsigned)BH), 256, 0, st>>>(listA, n, seg, seg, m - mbar, len0, seed,
                                                                                   (uint32_t)(61 + code1), pbase);
        else
            range_kernel<<<dim3(blocks(3 * seg), (unsigned)BH), 256, 0, st>>>(listA, n, 0, seg, 3 * seg);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
        if (q == 0) {
            copy_list_kernel<<<dim3(blocks(3 * n_out), (unsigned)BH), 256, 0, st>>>(Er, n_out, listA, n, 3 * n_out);
            count_launches(1);
            ELM_CUDA_TRY(cudaGetLastError());
        } else {
            // level i reads list i and writes list i + 1; the prefill keeps every list of the round
            // (the cache of an epoch is made of runs of them), compression alone alternates two
            int32_t *cur = listA, *nxt = listB;
            for (int i = 0; i < q; ++i) {
                const int per = 1 << (2 * (q - 1 - i));                       // calls per sibling
                const int P = (int)((len0 >> i) / per / 2);
                const double dlt = ldexp(dm, 2 * (i + 1 - q)) / (3.0 * (double)q);
                if (prefill) nxt = levels + (size_t)i * BH * n;
                const int rc = run_halve_level<Tin, T>(c, cur, i == q - 1 ? Er + n_out : nxt, n, 3 * per, P, i + code1, dlt, per);
                if (rc != ELM_OK) return rc;
                int32_t *tmp = cur; cur = nxt; nxt = tmp;
            }
        }
        if (prefill && r >= 1) {
            ELM_CUDA_TRY(cudaStreamWaitEvent(st, sides.halved[r - 1], 0));        // this round's E
            // Thinformer Express (Algorithm 5) for the 3 n_out 2^m tokens of this round.  The cache a token
            // sees is E with the finished siblings (weight 1), in every S_i the outputs of level-(i-1)
            // Halve calls that level i has not consumed yet (weight 2^(i-q)), and in S_0 the kept points
            // since the last level-0 call, itself included (weight 2^-q).  It changes with every level-0
            // call, so the tokens are taken in windows: one attention launch per window over every entry
            // that some token of the window sees, each entry carrying the span of tokens that see it.
            // The launches are independent given the round's lists; they are dealt to EXPRESS_LANES
            // streams (each with its own list buffers) between two events.
            const RoundGeom g = round_geom(p, mbar, r);
            float *lse = g.sub ? reinterpret_cast<float *>(ws + L.lse) : nullptr;
            RoundUniverse u;
            if (round_universe(p, mbar, r, u)) {
                // one launch for the round: every entry the round's tokens ever see is gathered once, each pair of
                // query tiles streams the blocks its own tokens see
                const RoundBuffers rb = round_buffers(L, ws, BH, u.n_univ);
                const int rc = express_attend_round(Q, K, V, O, p, u, Er, levels, (size_t)BH * n, listA, n, rb, lse, st);
                if (rc != ELM_OK) return rc;
            } else {
            const int64_t W = prefill_window(g), Wg = W >> g.wlog;
            ELM_CUDA_TRY(cudaEventRecord(fork, st));
            for (int i = 0; i < EXPRESS_LANES; ++i) ELM_CUDA_TRY(cudaStreamWaitEvent(side[i], fork, 0));
            int launch = 0;
            for (int jj = 0; jj < 3; ++jj) {
                for (int64_t G0 = 0; G0 < g.len0; G0 += Wg, ++launch) {
                    const int lane_id = launch % EXPRESS_LANES;
                    WindowPieces pc;
                    window_pieces(g, n_out, jj, G0, G0 + Wg, Er, levels, (size_t)BH * n, listA, pc);
                    const int64_t t0 = (jj + 1) * seg + (G0 << g.wlog);
                    const int rc = express_attend_window(Q, K, V, O, p, L, ws, pc, t0, (int)W, lse, side[lane_id], lane_id);
                    if (rc != ELM_OK) return rc;
                }
            }
            for (int i = 0; i < EXPRESS_LANES; ++i) {
                ELM_CUDA_TRY(cudaEventRecord(join[i], side[i]));
                ELM_CUDA_TRY(cudaStreamWaitEvent(st, join[i], 0));             // the halvings overwrite E
            }
            }
            if (g.sub) {
                // the tokens Subsample dropped still attend to themselves
                const dim3 grid((unsigned)((3 * seg + 7) / 8), (unsigned)(p->batch * p->q_heads));
                self_merge_kernel<Tin, T><<<grid, 256, 0, st>>>(Q, K, V, O, lse, listA, p->q_heads, p->kv_heads, n, p->d, seg,
                                                                g.len0, g.wlog, (T)(-g.q));
                count_launches(1);
                ELM_CUDA_TRY(cudaGetLastError());
            }
        }
        // halve phase: 4 n_out -> 2 n_out -> n_out, on the halving stream: it starts when this round's E (the
        // halvings of the round before, same stream) and the three outputs are there and, in the prefill, read
        const bool last_round = r == R - 1;
        ELM_CUDA_TRY(cudaEventRecord(sides.ready[r], st));
        ELM_CUDA_TRY(cudaStreamWaitEvent(sides.halve, sides.ready[r], 0));
        int rc = run_halve_level<Tin, T>(ch, Er, T1, n, 1, (int)(2 * n_out), (int)(62 + 64 * 4 * r), 0.5 * dm);
        if (rc != ELM_OK) return rc;
        rc = run_halve_level<Tin, T>(ch, T1, last_round ? idx_out : Enext, last_round ? n_out : n, 1, (int)n_out,
                                     (int)(63 + 64 * 4 * r), 0.5 * dm);
        if (rc != ELM_OK) return rc;
        ELM_CUDA_TRY(cudaEventRecord(sides.halved[r], sides.halve));
    }
    if (R >= 1) ELM_CUDA_TRY(cudaStreamWaitEvent(st, sides.halved[R - 1], 0));
    {
        StageTimer t(ELM_STAGE_EMIT, st, 1);
        const int64_t total = (int64_t)BH * n_out;
        emit_kernel<<<blocks(total), 256, 0, st>>>(w_out, idx_out, total, n_out, R == 0);
        count_launches(1);
        ELM_CUDA_TRY(cudaGetLastError());
    }
    return ELM_OK;
}

}  // namespace elm

extern "C" int elm_express_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes)
{
    using namespace elm;
    if (!params || !bytes) return ELM_ERR_NULL;
    const int rc = validate_express(params, mbar);
    if (rc != ELM_OK) return rc;
    *bytes = express_layout(params).total;
    return ELM_OK;
}

extern "C" int elm_express_compress(const void *K, const void *V, const elm_params *params, int32_t mbar, uint64_t seed,
                                    int32_t *idx_out, float *w_out, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    const int rc = validate_express(params, mbar);
    if (rc != ELM_OK) return rc;
    if (!K || !V || !idx_out || !w_out || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)idx_out | (uintptr_t)w_out) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < express_layout(params).total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    if (params->dtype == ELM_F32) {
        return det ? express_impl<float, double>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u)
                   : express_impl<float, float>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u);
    }
    return det ? express_impl<__nv_bfloat16, double>((const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u)
               : express_impl<__nv_bfloat16, float>((const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u);
}

namespace elm {
// what the prefill needs on top of validate_express
static int validate_prefill(const elm_params *p, int32_t mbar)
{
    int rc = validate_express(p, mbar);
    if (rc != ELM_OK) return rc;
    if (p->q_heads < 1 || p->q_heads % p->kv_heads != 0 || (int64_t)p->batch * p->q_heads > 65535) return ELM_ERR_SHAPE;
    if (p->n_q != p->n_kv) return ELM_ERR_SHAPE;                       // one query per token
    const int R = express_rounds(p);
    const int qmax = 2 * (R - 1) < mbar ? 2 * (R - 1) : mbar;            // deepest Compress2 of the run
    if (R >= 2 && qmax > p->log2_nout + 1) return ELM_ERR_SHAPE;          // level-0 calls of at least 2 points
    return ELM_OK;
}
}  // namespace elm

extern "C" int elm_express_prefill_workspace_bytes(const elm_params *params, int32_t mbar, size_t *bytes)
{
    using namespace elm;
    if (!params || !bytes) return ELM_ERR_NULL;
    const int rc = validate_prefill(params, mbar);
    if (rc != ELM_OK) return rc;
    *bytes = express_layout(params, mbar, true).total;
    return ELM_OK;
}

extern "C" int elm_express_prefill(const void *Q, const void *K, const void *V, const elm_params *params, int32_t mbar,
                                   uint64_t seed, void *O, int32_t *idx_out, float *w_out, void *workspace,
                                   size_t workspace_bytes, void *stream)
{
    using namespace elm;
    if (!params) return ELM_ERR_NULL;
    const int rc = validate_prefill(params, mbar);
    if (rc != ELM_OK) return rc;
    if (!Q || !K || !V || !O || !idx_out || !w_out || !workspace) return ELM_ERR_NULL;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O | (uintptr_t)idx_out | (uintptr_t)w_out) & 15) return ELM_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return ELM_ERR_ALIGN;
    if (workspace_bytes < express_layout(params, mbar, true).total) return ELM_ERR_WORKSPACE;
    unsigned char *ws = (unsigned char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const bool det = params->precision == ELM_PREC_FP64_DET;
    typedef __nv_bfloat16 bf;
    if (params->dtype == ELM_F32) {
        return det ? express_impl<float, double>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const float *)Q, (float *)O)
                   : express_impl<float, float>((const float *)K, (const float *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const float *)Q, (float *)O);
    }
    return det ? express_impl<bf, double>((const bf *)K, (const bf *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const bf *)Q, (bf *)O)
               : express_impl<bf, float>((const bf *)K, (const bf *)V, params, mbar, seed, idx_out, w_out, ws, st, 0u, (const bf *)Q, (bf *)O);
}
