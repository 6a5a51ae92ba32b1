// Thinformer Express (Algorithm 5) in prefill, one attention launch per round: geometry of a round and the
// list ("universe") of every cache entry the round's tokens ever see.
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <cuda_runtime.h>

#include "../../include/elm.h"

namespace elm {

// Geometry of round r of an Express run (thinning factor m = 2r): Compress2 depth q = min(m, mbar), one
// point kept per 2^wlog tokens (Subsample, when m > mbar), `seg` tokens and len0 kept points per sibling
// segment, s0 kept points per level-0 Halve call.
struct RoundGeom {
    int m, q, wlog;
    bool sub;
    int64_t seg, len0, s0;
};
inline RoundGeom round_geom(const elm_params *p, int mbar, int r)
{
    RoundGeom g;
    const int64_t n_out = (int64_t)1 << p->log2_nout;
    g.m = 2 * r;
    g.q = g.m < mbar ? g.m : mbar;
    g.sub = g.m > mbar;
    g.wlog = g.m - g.q;
    g.seg = n_out << g.m;
    g.len0 = n_out << g.q;
    g.s0 = g.q >= 1 ? (n_out << 2) >> g.q : g.len0;        // q = 0: no Halve call, S_0 only grows
    return g;
}

// The universe of a round, per attention problem: every entry of E and of the three siblings' point lists,
// laid out as
//   [0, EP)                          E and, behind it, the three siblings' outputs (4 n_out entries, padded)
//   EP + jj SP + off(i) ...          sibling jj, piece i: i = 0 its kept points (the entries of S_0), 1 <= i < q
//                                    the outputs of its level-(i-1) Halve calls (the entries of S_i),
//                                    len0 / 2^i entries each, every piece padded to a multiple of 128,
//                                    off(i) = sum over i' < i of the padded lengths
// so that a block of 128 entries never mixes pieces.  Each entry carries the span of tokens that see it
// (comment at round_universe_kernel); a pair of 128-query tiles streams only the blocks that hold entries
// some of its 256 tokens see (tile_blocks).
struct RoundUniverse {
    int q, wlog, sub;
    int64_t n_out, len0, s0, seg;
    int64_t EP, SP, n_univ;
    int tiles, cap;                  // pairs of query tiles in the round; most blocks any of them streams
    int64_t blocks_total;            // blocks streamed by all pairs of one head
};
__host__ __device__ inline int64_t round_pad128(int64_t x) { return (x + 127) / 128 * 128; }
__host__ __device__ inline int64_t round_piece_off(const RoundUniverse &u, int i)
{
    int64_t off = 0;
    for (int k = 0; k < i; ++k) off += round_pad128(u.len0 >> k);
    return off;
}
// Blocks of the universe that tile pair `tl` (tokens seg + 256 tl ... of every head) streams; returns their
// number, writes them to out[] if out is not null.  With G = the number of the sibling's kept points that
// have arrived, the pair's tokens live through G in [G0, G1]:
//   E and the finished siblings, plus the sibling's own output once G reaches len0 (rounds with Subsample:
//   the last kept point may come before the sibling's last token),
//   of S_i, 1 <= i < q, the outputs of level-(i-1) calls c_lo .. c_end - 1: call c (u entries) exists from
//   G = (c + 1) A, A = s0 4^(i-1), until the level-i call that consumes it completes at G = (c / 4 + 1) 4 A,
//   of S_0 the kept points from the start of the running level-0 call up to the pair's last token.
// A listed block carries TILE_BLK_PARTLY unless all of its 128 entries are seen by every token of the pair, whatever
// the problem (with Subsample the kept points differ between problems: the test is then conservative) - the
// attention kernel takes such a block without looking at any lifetime.
constexpr int32_t TILE_BLK_PARTLY = 1 << 30;
__host__ __device__ inline int tile_blocks(const RoundUniverse &u, int tl, int32_t *out)
{
    const int64_t t_all = (int64_t)tl * 256;
    const int64_t jj = t_all / u.seg, t_rel = t_all % u.seg;
    const int64_t G0 = t_rel >> u.wlog, G1 = ((t_rel + 255) >> u.wlog) + 1;
    // an entry born when G reaches X is seen by the pair's first token iff X <= G0; one that dies when G reaches Y is
    // seen by the pair's last token iff Y >= G_keep (the G1-th kept point is the last token itself without Subsample,
    // and may come earlier with it)
    const int64_t G_keep = u.sub ? G1 + 1 : G1;
    int n = 0;
    // blocks of the universe entries [a, b), which belong to the piece that starts at `base` and has `len` entries;
    // born(e) / dies(e): the G at which entry e of the piece appears / disappears (dies < 0: never)
    auto run = [&](int64_t a, int64_t b, int64_t base, int64_t len, auto born, auto dies) {
        if (b <= a) return;
        for (int64_t blk = a / 128; blk <= (b - 1) / 128; ++blk) {
            const int64_t lo = blk * 128 - base, hi = lo + 127;
            bool whole = lo >= 0 && hi < len && born(hi) <= G0;
            if (whole) {
                const int64_t d = dies(lo);
                whole = d < 0 || d >= G_keep;
            }
            if (out) out[n] = (int32_t)blk | (whole ? 0 : TILE_BLK_PARTLY);
            ++n;
        }
    };
    // E and the finished siblings (always there for this sibling's tokens); its own output only behind its last kept point
    const int64_t e_seen = (1 + jj) * u.n_out;
    run(0, e_seen + ((u.q >= 1 && u.sub && G1 >= u.len0) ? u.n_out : 0), 0, e_seen,
        [&](int64_t) { return (int64_t)0; }, [&](int64_t) { return (int64_t)-1; });
    const int64_t base = u.EP + jj * u.SP;
    for (int i = u.q - 1; i >= 1; --i) {
        const int64_t A = u.s0 << (2 * (i - 1)), unit = (u.s0 << (i - 1)) >> 1;
        // call c's output is born when G reaches (c + 1) A, right after that kept point: without Subsample the
        // G1-th kept point is the pair's last token, so what is born there belongs to the next pair
        const int64_t c_lo = 4 * (G0 / (4 * A)), c_end = (u.sub ? G1 : G1 - 1) / A;
        const int64_t b0 = base + round_piece_off(u, i);
        run(b0 + c_lo * unit, b0 + c_end * unit, b0, u.len0 >> i,
            [&](int64_t e) { return (e / unit + 1) * A; }, [&](int64_t e) { return (e / unit / 4 + 1) * 4 * A; });
    }
    const int64_t g_lo = u.q >= 1 ? (G0 / u.s0) * u.s0 : 0;
    // kept point g is born at its own token: before the pair iff its stratum lies before the pair's first
    run(base + g_lo, base + G1, base, u.len0, [&](int64_t e) { return e + 1; },
        [&](int64_t e) { return u.q >= 1 ? (e / u.s0 + 1) * u.s0 : (int64_t)-1; });
    return n;
}

// Entry `pos` of the universe: which row of K / V it is (through `row_of`), its weight, the first token that sees it
// (birth) and the first that does not any more (death).  With G = the number of a sibling's kept points that have
// arrived - G = X is reached right after the X-th kept point, at token kept(jj, X - 1) + 1:
//   E                       always;  the output of sibling j: from G_j = len0 on (q = 0: from the end of its segment)
//   S_i entry of call c     from G = (c + 1) A until G = (c / 4 + 1) 4 A          (A = s0 4^(i-1))
//   S_0 entry g             from its own token (which sees itself) until G = (g / s0 + 1) s0   (q = 0: until the
//                           sibling's segment ends)
// Padding entries are never seen.  `kept(jj, g)` is the token of kept point g of sibling jj; piece = -1 for E,
// -2 for padding, else the level i, with `off` the entry's index within the sibling's piece (within E for piece -1).
constexpr int32_t ROUND_NEVER = 0x7fffffff;
// kept(jj, g) over an array that holds the three siblings' kept points one after the other
struct KeptArray {
    const int32_t *kept;
    int64_t len0;
    __host__ __device__ int32_t operator()(int64_t jj, int64_t g) const { return kept[jj * len0 + g]; }
};
struct UniverseEntry {
    int piece;
    int64_t jj, off;
    int32_t birth, death;
    float w;
};
template <class Kept>
__host__ __device__ inline UniverseEntry universe_entry(const RoundUniverse &u, int64_t pos, Kept kept)
{
    UniverseEntry e = {-2, 0, 0, ROUND_NEVER, ROUND_NEVER, 1.f};
    auto token_after = [&](int64_t jj, int64_t X) { return X > u.len0 ? ROUND_NEVER : (int32_t)(kept(jj, X - 1) + 1); };
    if (pos < u.EP) {
        if (pos < 4 * u.n_out) {
            const int64_t part = pos / u.n_out;
            e.piece = -1;
            e.off = pos;
            // (q = 0: no Halve call - the sibling's kept points stay in S_0 to the end of its segment and only then
            // join E, so their copy in E must not be seen before the next sibling begins)
            e.birth = part == 0 ? 0 : (u.q >= 1 ? token_after(part - 1, u.len0) : (int32_t)((part + 1) * u.seg));
        }
        return e;
    }
    e.jj = (pos - u.EP) / u.SP;
    int64_t o = (pos - u.EP) % u.SP;
    int i = 0;
    while (o >= round_pad128(u.len0 >> i)) { o -= round_pad128(u.len0 >> i); ++i; }
    if (o >= (u.len0 >> i)) return e;                         // padding behind the piece
    e.piece = i;
    e.off = o;
    e.w = 1.f;
    for (int k = 0; k < u.q - i; ++k) e.w *= 0.5f;           // 2^(i - q)
    if (i == 0) {
        e.birth = (int32_t)kept(e.jj, o);
        // (q = 0: no Halve call; the points leave S_0 for E when the sibling's segment ends)
        e.death = u.q >= 1 ? token_after(e.jj, (o / u.s0 + 1) * u.s0) : (int32_t)((e.jj + 2) * u.seg);
    } else {
        const int64_t A = u.s0 << (2 * (i - 1)), unit = (u.s0 << (i - 1)) >> 1, c = o / unit;
        e.birth = token_after(e.jj, (c + 1) * A);
        e.death = token_after(e.jj, (c / 4 + 1) * 4 * A);
    }
    return e;
}

// Does round r of the prefill take the one-launch form?  (bf16 inputs in fp32 mode - the tensor-core attention
// kernel - and segments that are whole pairs of query tiles.)  Fills `u` if so.
bool round_universe(const elm_params *p, int mbar, int r, RoundUniverse &u);

// Device buffers of the one-launch form (sized by round_buffer_bytes for the largest universe of the run)
struct RoundBuffers {
    int32_t *idx, *birth, *death, *blk_birth, *blk_death, *tile_cnt, *tile_blk;
    int32_t *item_tab, *item_cnt;        // [item_ctas][item_cap], [item_ctas]: the pairs each persistent CTA takes
    int item_cap, item_ctas;
    float *w;
    unsigned char *ws_attend;
};
struct RoundBufferLayout {
    size_t idx, w, birth, death, blk, tile_cnt, tile_blk, item_tab, item_cnt, ws_attend, total;
    int item_cap, item_ctas;
};
// Largest universe / tile table over the rounds of the run that take the one-launch form (total = 0: none does)
RoundBufferLayout round_buffer_layout(const elm_params *p, int mbar, int rounds);

// Causal attention over the first `rows` tokens of each of `heads` heads (the exact start): fills the tile table so
// that a pair of query tiles streams the list only up to its own last token, deals the pairs to the CTAs by
// length, and points `win` at both.
struct AttendWindow;
int causal_tile_table(int rows, int heads, const RoundBuffers &rb, AttendWindow &win, cudaStream_t st);

// Attention of the round's 3 seg tokens over the universe: builds the universe from E (stride `stride`
// per problem), the level lists (`levels` + (i - 1) level_stride: outputs of level i - 1) and the kept
// points (`kept`), the tile table, then one gather and one attention launch on `st`.
int express_attend_round(const void *Q, const void *K, const void *V, void *O, const elm_params *p, const RoundUniverse &u,
                         const int32_t *E, const int32_t *levels, size_t level_stride, const int32_t *kept, int64_t stride,
                         const RoundBuffers &rb, float *lse, cudaStream_t st);

}  // namespace elm
