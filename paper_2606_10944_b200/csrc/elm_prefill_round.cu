// Thinformer Express (Algorithm 5) in prefill, one attention launch per round.
//
// Within round r the cache of a token is E with the finished siblings (weight 1), in every S_i the outputs of
// level-(i-1) Halve calls that level i has not consumed yet (weight 2^(i-q)), and in S_0 the kept points since
// the last level-0 call, the token itself included (weight 2^-q) - Algorithm 1's wtd_cache() as of that token.
// All of these are entries of lists the round's compression has already written, so the round's "universe"
// (elm_prefill_round.cuh) is gathered once; each entry carries the span of tokens that see it, and each pair
// of 128-query tiles streams the blocks that hold entries its own tokens see.
#include "elm_prefill_round.cuh"

#include <stdlib.h>

#include <algorithm>
#include <deque>
#include <mutex>
#include <queue>
#include <utility>
#include <vector>

#include "elm_attend.cuh"
#include "elm_common.cuh"

namespace elm {
namespace {

constexpr int32_t NEVER = 0x7fffffff;

// One thread per universe entry: row number, weight, first token that sees it (birth) and first that does
// not any more (death); per block of 128 entries the largest birth and the smallest death.  With G = the
// number of a sibling's kept points that have arrived - G = X is reached right after the X-th kept point, at
// token kept[X - 1] + 1:
//   E                       always;  the output of sibling j: from G_j = len0 on (q = 0: from the end of its segment)
//   S_i entry of call c     from G = (c + 1) A until G = (c / 4 + 1) 4 A          (A = s0 4^(i-1))
//   S_0 entry g             from its own token (which sees itself) until G = (g / s0 + 1) s0   (q = 0: for good)
// Padding entries are never seen.
__global__ void __launch_bounds__(256) round_universe_kernel(RoundUniverse u, const int32_t *__restrict__ E,
                                                             const int32_t *__restrict__ levels, int64_t level_stride,
                                                             const int32_t *__restrict__ kept_all, int64_t stride,
                                                             int32_t *__restrict__ idx, float *__restrict__ w,
                                                             int32_t *__restrict__ birth, int32_t *__restrict__ death,
                                                             int32_t *__restrict__ blk_birth, int32_t *__restrict__ blk_death)
{
    __shared__ int32_t sb[8], sd[8];
    const int64_t pos = (int64_t)blockIdx.x * 256 + threadIdx.x;          // n_univ is a multiple of 128
    const int64_t pr = blockIdx.y;
    int32_t bt = NEVER, dt = NEVER, row = 0;
    float wt = 1.f;
    if (pos < u.n_univ) {
        const int32_t *kept = kept_all + pr * stride;
        auto token_after = [&](int64_t jj, int64_t X) { return X > u.len0 ? NEVER : kept[jj * u.len0 + X - 1] + 1; };
        if (pos < u.EP) {
            if (pos < 4 * u.n_out) {
                const int64_t part = pos / u.n_out;
                row = E[pr * stride + pos];
                // (q = 0: no Halve call - the sibling's kept points stay in S_0 to the end of its segment and only
                // then join E, so their copy in E must not be seen before the next sibling begins)
                bt = part == 0 ? 0 : (u.q >= 1 ? token_after(part - 1, u.len0) : (int32_t)((part + 1) * u.seg));
            }
        } else {
            const int64_t jj = (pos - u.EP) / u.SP;
            int64_t o = (pos - u.EP) % u.SP;
            int i = 0;
            while (o >= round_pad128(u.len0 >> i)) { o -= round_pad128(u.len0 >> i); ++i; }
            if (o < (u.len0 >> i)) {
                wt = ldexpf(1.f, i - u.q);
                if (i == 0) {
                    row = kept[jj * u.len0 + o];
                    bt = row;
                    if (u.q >= 1) dt = token_after(jj, (o / u.s0 + 1) * u.s0);
                } else {
                    const int64_t A = u.s0 << (2 * (i - 1)), unit = (u.s0 << (i - 1)) >> 1, c = o / unit;
                    row = levels[(int64_t)(i - 1) * level_stride + pr * stride + jj * (u.len0 >> i) + o];
                    bt = token_after(jj, (c + 1) * A);
                    dt = token_after(jj, (c / 4 + 1) * 4 * A);
                }
            }
        }
        idx[pr * u.n_univ + pos] = row;
        w[pr * u.n_univ + pos] = wt;
        birth[pr * u.n_univ + pos] = bt;
        death[pr * u.n_univ + pos] = dt;
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
        const int64_t blk = (int64_t)blockIdx.x * 2 + threadIdx.x, h = threadIdx.x * 4;
        if (blk < u.n_univ / 128) {
            blk_birth[pr * (u.n_univ / 128) + blk] = max(max(sb[h], sb[h + 1]), max(sb[h + 2], sb[h + 3]));
            blk_death[pr * (u.n_univ / 128) + blk] = min(min(sd[h], sd[h + 1]), min(sd[h + 2], sd[h + 3]));
        }
    }
}

// One thread per pair of query tiles: the blocks of the universe the pair streams
__global__ void round_tiles_kernel(RoundUniverse u, int32_t *__restrict__ tile_cnt, int32_t *__restrict__ tile_blk)
{
    const int tl = blockIdx.x * blockDim.x + threadIdx.x;
    if (tl >= u.tiles) return;
    tile_cnt[tl] = tile_blocks(u, tl, tile_blk + (int64_t)tl * u.cap);
}

// Causal attention over the first `rows` tokens: pair x of query tiles sees the list up to token 256 x + 255
__global__ void causal_tiles_kernel(int tiles, int cap, int32_t *__restrict__ tile_cnt, int32_t *__restrict__ tile_blk)
{
    const int tl = blockIdx.x * blockDim.x + threadIdx.x;
    if (tl >= tiles) return;
    const int cnt = min(cap, 2 * tl + 2);
    tile_cnt[tl] = cnt;
    for (int j = 0; j < cnt; ++j) tile_blk[(int64_t)tl * cap + j] = j;
}

// Which pairs of query tiles each persistent CTA of the attention launch takes.  The pairs of a launch with block
// lists differ in length (cost[x] blocks for pair x of every head), so dealing them out in turn leaves some CTAs
// with 10-17 % more blocks than the mean; here the heads are taken in order (the CTAs then work on one head at a
// time and share its blocks in L2) and, within a head, the pairs from the longest to the shortest, each given to
// the CTA with the least work so far.  Returns false if some CTA would get more than `cap` pairs.
bool balance_items(const std::vector<int> &cost, int heads, int ctas, int cap, std::vector<int32_t> &tab, std::vector<int32_t> &cnt)
{
    const int tiles = (int)cost.size();
    std::vector<int> order(tiles);
    for (int i = 0; i < tiles; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost[a] > cost[b]; });
    typedef std::pair<int64_t, int> Load;                        // (blocks so far, CTA)
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int c = 0; c < ctas; ++c) heap.push(Load(0, c));
    tab.assign((size_t)ctas * cap, 0);
    cnt.assign(ctas, 0);
    for (int h = 0; h < heads; ++h)
        for (int i = 0; i < tiles; ++i) {
            const Load top = heap.top();
            heap.pop();
            const int c = top.second;
            if (cnt[c] >= cap) return false;
            tab[(size_t)c * cap + cnt[c]++] = h * tiles + order[i];
            heap.push(Load(top.first + cost[order[i]] + 1, c));  // + 1: what a pair costs besides its blocks
        }
    return true;
}
// Uploads the table for `cost` and points `win` at it (leaves `win` alone if the table does not fit its buffers).
int upload_item_table(const std::vector<int> &cost, int heads, const RoundBuffers &rb, AttendWindow &win, cudaStream_t st)
{
    const int64_t items = (int64_t)cost.size() * heads;
    const int ctas = (int)std::min<int64_t>(items, device_sm_count());
    if (!rb.item_tab || rb.item_cap < 1 || ctas > rb.item_ctas) return ELM_OK;
    // The table depends on the run's geometry alone: the last few are kept, so that a caller that repeats a run
    // (a serving loop) pays for the dealing once.
    struct Cached {
        std::vector<int> cost;
        int heads, ctas, cap;
        bool fits;
        std::vector<int32_t> tab, cnt;
    };
    static std::mutex mu;
    static std::deque<Cached> cache;
    std::lock_guard<std::mutex> lock(mu);
    const Cached *hit = nullptr;
    for (const Cached &c : cache)
        if (c.heads == heads && c.ctas == ctas && c.cap == rb.item_cap && c.cost == cost) { hit = &c; break; }
    if (!hit) {
        Cached c;
        c.cost = cost; c.heads = heads; c.ctas = ctas; c.cap = rb.item_cap;
        c.fits = balance_items(cost, heads, ctas, rb.item_cap, c.tab, c.cnt);
        cache.push_back(std::move(c));
        if (cache.size() > 16) cache.pop_front();
        hit = &cache.back();
    }
    if (!hit->fits) return ELM_OK;
    // (pageable source: each call returns once its source may change)
    ELM_CUDA_TRY(cudaMemcpyAsync(rb.item_tab, hit->tab.data(), hit->tab.size() * 4, cudaMemcpyHostToDevice, st));
    ELM_CUDA_TRY(cudaMemcpyAsync(rb.item_cnt, hit->cnt.data(), hit->cnt.size() * 4, cudaMemcpyHostToDevice, st));
    win.item_tab = rb.item_tab;
    win.item_cnt = rb.item_cnt;
    win.item_cap = rb.item_cap;
    win.item_ctas = ctas;
    return ELM_OK;
}

bool rounds_enabled()
{
    static const bool on = []() {
        const char *e = getenv("ELM_PREFILL_ROUNDS");                   // tuning aid: 0 forces one launch per window
        return !(e && atoi(e) == 0);
    }();
    return on;
}

}  // namespace

bool round_universe(const elm_params *p, int mbar, int r, RoundUniverse &u)
{
    if (r < 1 || p->dtype != ELM_BF16 || p->precision != ELM_PREC_FP32 || !rounds_enabled()) return false;
    const RoundGeom g = round_geom(p, mbar, r);
    if (g.seg % 256 != 0) return false;
    u.q = g.q; u.wlog = g.wlog; u.sub = g.sub ? 1 : 0;
    u.n_out = (int64_t)1 << p->log2_nout;
    u.len0 = g.len0; u.s0 = g.s0; u.seg = g.seg;
    u.EP = round_pad128(4 * u.n_out);
    u.SP = round_piece_off(u, g.q >= 1 ? g.q : 1);                       // q = 0: the kept points alone
    u.n_univ = u.EP + 3 * u.SP;
    if (u.n_univ > 0x7fffffff / 2) return false;
    u.tiles = (int)(3 * g.seg / 256);
    u.cap = 0;
    u.blocks_total = 0;
    for (int tl = 0; tl < u.tiles; ++tl) {
        const int c = tile_blocks(u, tl, nullptr);
        if (c > u.cap) u.cap = c;
        u.blocks_total += c;
    }
    return true;
}

RoundBufferLayout round_buffer_layout(const elm_params *p, int mbar, int rounds)
{
    RoundBufferLayout L = {};
    size_t n_univ = 0, table = 0, tiles = 0;
    for (int r = 1; r < rounds; ++r) {
        RoundUniverse u;
        if (!round_universe(p, mbar, r, u)) continue;
        if ((size_t)u.n_univ > n_univ) n_univ = (size_t)u.n_univ;
        if ((size_t)u.tiles * u.cap > table) table = (size_t)u.tiles * u.cap;
        if ((size_t)u.tiles > tiles) tiles = (size_t)u.tiles;
    }
    if (n_univ == 0) return L;
    {
        // the exact start (causal attention over 4 n_out tokens) borrows the tile table
        const size_t rows = (size_t)4 << p->log2_nout, st_tiles = (rows + 255) / 256, st_cap = (rows + 127) / 128;
        if (st_tiles > tiles) tiles = st_tiles;
        if (st_tiles * st_cap > table) table = st_tiles * st_cap;
    }
    const size_t BH = (size_t)p->batch * p->kv_heads;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.idx = take(BH * n_univ * 4);
    L.w = take(BH * n_univ * 4);
    L.birth = take(BH * n_univ * 4);
    L.death = take(BH * n_univ * 4);
    L.blk = take(2 * BH * (n_univ / 128) * 4);
    L.tile_cnt = take(tiles * 4);
    L.tile_blk = take(table * 4);
    // per-CTA item lists of the attention launches: room for twice the mean number of pairs per CTA
    L.item_ctas = device_sm_count();
    L.item_cap = (int)(2 * ((tiles * (size_t)p->batch * p->q_heads + L.item_ctas - 1) / L.item_ctas) + 16);
    L.item_tab = take((size_t)L.item_ctas * L.item_cap * 4);
    L.item_cnt = take((size_t)L.item_ctas * 4);
    L.ws_attend = take(attend_layout(p, (int32_t)n_univ).total);
    L.total = off;
    return L;
}

int causal_tile_table(int rows, int heads, const RoundBuffers &rb, AttendWindow &win, cudaStream_t st)
{
    const int tiles = (rows + 255) / 256, cap = (rows + 127) / 128;
    causal_tiles_kernel<<<(unsigned)((tiles + 127) / 128), 128, 0, st>>>(tiles, cap, rb.tile_cnt, rb.tile_blk);
    count_launches(1);
    ELM_CUDA_TRY(cudaGetLastError());
    win.tile_cnt = rb.tile_cnt;
    win.tile_blk = rb.tile_blk;
    win.tile_cap = cap;
    std::vector<int> cost(tiles);
    for (int tl = 0; tl < tiles; ++tl) cost[tl] = std::min(cap, 2 * tl + 2);
    return upload_item_table(cost, heads, rb, win, st);
}

int express_attend_round(const void *Q, const void *K, const void *V, void *O, const elm_params *p, const RoundUniverse &u,
                         const int32_t *E, const int32_t *levels, size_t level_stride, const int32_t *kept, int64_t stride,
                         const RoundBuffers &rb, float *lse, cudaStream_t st)
{
    const int BH = p->batch * p->kv_heads;
    round_universe_kernel<<<dim3((unsigned)((u.n_univ + 255) / 256), (unsigned)BH), 256, 0, st>>>(
        u, E, levels, (int64_t)level_stride, kept, stride, rb.idx, rb.w, rb.birth, rb.death, rb.blk_birth, rb.blk_death);
    round_tiles_kernel<<<(unsigned)((u.tiles + 127) / 128), 128, 0, st>>>(u, rb.tile_cnt, rb.tile_blk);
    count_launches(2);
    ELM_CUDA_TRY(cudaGetLastError());
    elm_params pe = *p;
    pe.n_q = (int32_t)(3 * u.seg);
    AttendWindow win;
    win.q_row0 = u.seg;
    win.n_q_total = p->n_kv;
    win.birth = rb.birth;
    win.death = rb.death;
    win.blk_birth = rb.blk_birth;
    win.blk_death = rb.blk_death;
    win.lse = lse;
    win.tile_cnt = rb.tile_cnt;
    win.tile_blk = rb.tile_blk;
    win.tile_cap = u.cap;
    {
        std::vector<int> cost(u.tiles);
        for (int tl = 0; tl < u.tiles; ++tl) cost[tl] = tile_blocks(u, tl, nullptr);
        const int rc = upload_item_table(cost, p->batch * p->q_heads, rb, win, st);
        if (rc != ELM_OK) return rc;
    }
    return attend_enqueue(Q, K, V, rb.idx, rb.w, (int32_t)u.n_univ, &pe, O, rb.ws_attend, st, win);
}

}  // namespace elm
