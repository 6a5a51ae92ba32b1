"""Host logic of the prefill's one-launch-per-round form (no GPU): the two descriptions of an Express round - the
lifetime of every entry of the round's list, and the blocks of 128 entries each pair of 128-query tiles streams -
must agree: whatever a token of a pair sees lies in a block of the pair's list.  The library rebuilds both on the
host (elm_debug_round_check) for kept points drawn from a seed."""
import pytest

import paper_2606_10944_b200 as elm

# log2_nout, mbar, rounds R (n = n_out 4^R), head dim
RUNS = [
    (6, 4, 3, 64),       # level-0 calls of 64 and 16 points
    (6, 0, 4, 64),       # mbar = 0: strata of 4, 16 and 64 tokens, no Halve call inside a segment
    (6, 1, 5, 128),      # strata up to 128 tokens, Compress2 of depth 1
    (7, 3, 4, 128),      # odd mbar
    (8, 6, 3, 128),
    (9, 7, 4, 128),      # the paper's proportions (mbar = log2 n_out - 2)
    (6, 0, 6, 64),       # strata of 1024 tokens: a pair of query tiles lies inside one stratum
    (11, 9, 3, 128),     # cfg5's prefill
]


@pytest.mark.parametrize("log2_nout,mbar,R,d", RUNS)
def test_every_visible_entry_lies_in_a_listed_block(log2_nout, mbar, R, d):
    n = (1 << log2_nout) * 4 ** R
    checked = 0
    for r in range(1, R):
        for seed in (1, 2):
            res = elm.debug_round_check(1, 2, 1, n, d, log2_nout, mbar, r, seed=seed)
            if res is None:                      # segments shorter than a pair of query tiles: taken in windows
                assert (1 << log2_nout) * 4 ** r % 256 != 0
                continue
            missing, listed, needed, partly = res
            assert missing == 0, (r, seed, res)
            # the lists are tight: at most one block in twenty holds nothing the pair sees
            assert needed <= listed <= needed * 1.05 + 1, (r, seed, res)
            assert 0 < partly <= listed
            checked += 1
    assert checked >= 2


def test_most_blocks_of_cfg5_are_listed_as_seen_whole():
    """cfg5's prefill (level-0 calls of 512 and 2048 points): only the blocks around a pair's own tokens can be partly
    visible - the kernel looks at lifetimes for about one block in twenty."""
    n = 2048 * 4 ** 3
    for r in (1, 2):
        missing, listed, needed, partly = elm.debug_round_check(1, 32, 8, n, 128, 11, 9, r)
        assert missing == 0 and partly <= 0.08 * listed


def test_rounds_of_other_storage_or_precision_are_taken_in_windows():
    n = 64 * 4 ** 3
    assert elm.debug_round_check(1, 2, 1, n, 64, 6, 4, 2, dtype_code=0) is None              # fp32 storage
    assert elm.debug_round_check(1, 2, 1, n, 64, 6, 4, 2, precision="fp64") is None
    assert elm.debug_round_check(1, 2, 1, n, 64, 6, 4, 0) is None                            # round 0 is exact
