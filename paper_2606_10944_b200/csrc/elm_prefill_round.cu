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

constexpr int32_t NEVER = ROUND_NEVER;

// One thread per universe entry (universe_entry in the header): row number, weight, lifetime; per block of 128
// entries the largest birth and the smallest death.
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
        const UniverseEntry e = universe_entry(u, pos, KeptArray{kept, u.len0});
        bt = e.birth;
        dt = e.death;
        wt = e.w;
        if (e.piece == -1) row = E[pr * stride + e.off];
        else if (e.piece == 0) row = kept[e.jj * u.len0 + e.off];
        else if (e.piece > 0) row = levels[(int64_t)(e.piece - 1) * level_stride + pr * stride + e.jj * (u.len0 >> e.piece) + e.off];
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

// Host-only consistency check of the one-launch form's two descriptions of a round (test hook, no CUDA call): the
// lifetimes say which tokens see an entry, the block lists say which blocks a pair of query tiles streams - every
// entry that some token of a pair sees must lie in a block of the pair's list, and a block listed as seen whole must
// hold only entries that every token of the pair sees.  Kept points: the segment's own
// tokens, or (rounds with Subsample) one pseudo-random token per stratum drawn from `seed`.
extern "C" int elm_debug_round_check(const elm_params *params, int32_t mbar, int32_t r, uint64_t seed, int64_t *missing,
                                     int64_t *listed_blocks, int64_t *needed_blocks, int64_t *partly_blocks)
{
    using namespace elm;
    if (!params || !missing || !listed_blocks || !needed_blocks || !partly_blocks) return ELM_ERR_NULL;
    RoundUniverse u;
    if (!round_universe(params, mbar, r, u)) return ELM_ERR_SHAPE;
    std::vector<int32_t> kept((size_t)3 * u.len0);
    uint64_t state = seed * 6364136223846793005ull + 1442695040888963407ull;
    for (int64_t jj = 0; jj < 3; ++jj)
        for (int64_t g = 0; g < u.len0; ++g) {
            state = state * 6364136223846793005ull + 1442695040888963407ull;
            const int64_t within = u.wlog ? (int64_t)((state >> 33) % ((uint64_t)1 << u.wlog)) : 0;
            kept[(size_t)(jj * u.len0 + g)] = (int32_t)((jj + 1) * u.seg + (g << u.wlog) + within);
        }
    const KeptArray kept_of = {kept.data(), u.len0};
    std::vector<UniverseEntry> entries((size_t)u.n_univ);
    for (int64_t pos = 0; pos < u.n_univ; ++pos) entries[(size_t)pos] = universe_entry(u, pos, kept_of);
    *missing = *listed_blocks = *needed_blocks = *partly_blocks = 0;
    // (the attention kernel finds a row's visible columns by bisection: births and deaths must not decrease within a block)
    for (int64_t pos = 1; pos < u.n_univ; ++pos)
        if (pos % 128 != 0 && (entries[(size_t)pos].birth < entries[(size_t)pos - 1].birth ||
                               entries[(size_t)pos].death < entries[(size_t)pos - 1].death))
            ++*missing;
    std::vector<int32_t> list((size_t)u.cap);
    std::vector<char> in_list((size_t)(u.n_univ / 128)), needed((size_t)(u.n_univ / 128));
    for (int tl = 0; tl < u.tiles; ++tl) {
        const int cnt = tile_blocks(u, tl, list.data());
        if (cnt > u.cap) return ELM_ERR_WORKSPACE;
        std::fill(in_list.begin(), in_list.end(), 0);
        std::fill(needed.begin(), needed.end(), 0);
        const int64_t T0 = u.seg + (int64_t)tl * 256, T1 = T0 + 256;       // the pair's tokens
        for (int j = 0; j < cnt; ++j) {
            const int32_t b = list[(size_t)j] & ~TILE_BLK_PARTLY;
            if (b < 0 || b >= u.n_univ / 128 || in_list[(size_t)b]) return ELM_ERR_SHAPE;   // out of range or twice
            in_list[(size_t)b] = 1;
            if (!(list[(size_t)j] & TILE_BLK_PARTLY)) {
                // said to be seen whole: every one of its entries must be seen by every token of the pair
                for (int64_t pos = (int64_t)b * 128; pos < (int64_t)b * 128 + 128; ++pos) {
                    const UniverseEntry &e = entries[(size_t)pos];
                    if (!(e.birth <= T0 && e.death >= T1)) ++*missing;
                }
            } else {
                ++*partly_blocks;
            }
        }
        for (int64_t pos = 0; pos < u.n_univ; ++pos) {
            const UniverseEntry &e = entries[(size_t)pos];
            if (e.birth < e.death && e.birth < T1 && e.death > T0) {
                needed[(size_t)(pos / 128)] = 1;
                if (!in_list[(size_t)(pos / 128)]) ++*missing;
            }
        }
        *listed_blocks += cnt;
        for (size_t b = 0; b < needed.size(); ++b) *needed_blocks += needed[b];
    }
    return ELM_OK;
}
