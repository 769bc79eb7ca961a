"""Pins for the token-budget selection of the CPU oracle (Sec. 3.1, 3.2): brute force by
numpy's lexicographic sort, crafted ties, k = 1, k = n, all-equal scores, zeros of both
signs, NaN.  No GPU needed."""
import numpy as np
import pytest

import oracle


def _brute(scores, n, k):
    """k-1 best of blocks [0, n-1) by (score desc, index asc) + block n-1, ascending."""
    s = scores[: n - 1].astype(np.float64)
    s = np.where(np.isnan(s), -np.inf, s)
    nan_last = np.isnan(scores[: n - 1]).astype(np.int64)
    order = np.lexsort((np.arange(n - 1), -s, nan_last))     # last key is the primary one
    return sorted(list(order[: max(0, k - 1)]) + [n - 1])


@pytest.mark.parametrize("seed", range(6))
def test_random_scores_against_lexsort(seed):
    r = np.random.default_rng(seed)
    B, Hkv, b, max_blocks, max_sel = 3, 2, 16, 40, 12
    lens = np.array([40 * 16, 17 * 16 - 5, 3], np.int32)
    sc = r.normal(size=(B, Hkv, max_blocks)).astype(np.float32)
    if seed % 2:
        sc = np.round(sc * 2) / 2                # many exact ties
    budget = [16 * 7, 16 * 12, 16 * 100, 5][seed % 4]
    idx, cnt = oracle.select(sc, lens, b, budget, max_sel)
    for i in range(B):
        n = -(-int(lens[i]) // b)
        k = min(max(1, budget // b), n, max_sel)
        for h in range(Hkv):
            want = _brute(sc[i, h], n, k)
            assert cnt[i, h] == len(want) == k
            assert list(idx[i, h, :k]) == want
            assert np.all(idx[i, h, k:] == -1)


def test_crafted_ties_prefer_lower_index():
    sc = np.array([[[1.0, 5.0, 5.0, 5.0, 0.0, 5.0, 9.0, 123.0]]], np.float32)
    lens = [8 * 4]                                # n = 8, block 7 forced, its score ignored
    idx, cnt = oracle.select(sc, lens, 4, 4 * 4, 8)
    assert list(idx[0, 0, :4]) == [1, 2, 6, 7] and cnt[0, 0] == 4
    idx, cnt = oracle.select(sc, lens, 4, 4 * 1, 8)          # k = 1: only the last block
    assert list(idx[0, 0]) == [7] + [-1] * 7 and cnt[0, 0] == 1
    idx, cnt = oracle.select(sc, lens, 4, 4 * 8, 8)          # k = n: everything
    assert list(idx[0, 0]) == list(range(8))
    idx, cnt = oracle.select(sc, lens, 4, 4 * 50, 8)         # budget beyond the sequence
    assert list(idx[0, 0]) == list(range(8))
    idx, cnt = oracle.select(sc, lens, 4, 0, 8)              # budget below one block -> k = 1
    assert cnt[0, 0] == 1 and idx[0, 0, 0] == 7


def test_all_equal_scores_take_the_first_blocks():
    sc = np.full((1, 1, 10), 0.25, np.float32)
    idx, cnt = oracle.select(sc, [10 * 8], 8, 8 * 4, 6)
    assert list(idx[0, 0]) == [0, 1, 2, 9, -1, -1]


def test_signed_zeros_tie_and_nan_ranks_last():
    sc = np.array([[[-0.0, 0.0, -1.0, np.nan, -0.0, 7.0]]], np.float32)
    idx, _ = oracle.select(sc, [6], 1, 3, 6)                 # n = 6, k = 3
    assert list(idx[0, 0, :3]) == [0, 1, 5]                  # -0 at index 0 ties with +0 at 1
    sc = np.array([[[np.nan, -np.inf, np.nan, -3.0, 0.0]]], np.float32)
    idx, _ = oracle.select(sc, [5], 1, 4, 5)                 # candidates 0..3, k-1 = 3
    assert list(idx[0, 0, :4]) == [0, 1, 3, 4]               # -3, -inf, then the first NaN
    idx, _ = oracle.select(sc, [5], 1, 3, 5)
    assert list(idx[0, 0, :3]) == [1, 3, 4]


def test_partial_tail_and_single_block():
    sc = np.arange(8, dtype=np.float32).reshape(1, 1, 8)
    idx, cnt = oracle.select(sc, [33], 8, 16, 4)             # n = 5 (tail of 1 token), k = 2
    assert list(idx[0, 0, :2]) == [3, 4] and cnt[0, 0] == 2
    idx, cnt = oracle.select(sc, [5], 8, 64, 4)              # n = 1
    assert list(idx[0, 0]) == [0, -1, -1, -1] and cnt[0, 0] == 1
    idx, cnt = oracle.select(sc, [0], 8, 64, 4)              # empty sequence
    assert cnt[0, 0] == 0 and np.all(idx == -1)


def test_positive_scaling_never_changes_the_selection():
    r = np.random.default_rng(9)
    sc = r.normal(size=(2, 2, 64)).astype(np.float32)
    a = oracle.select(sc, [64 * 8, 50 * 8], 8, 8 * 9, 16)
    b = oracle.select(sc * np.float32(0.125), [64 * 8, 50 * 8], 8, 8 * 9, 16)   # exact scaling
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# ---- threshold method (Sec. 3.1): blocks whose softmax score exceeds tau, plus the last block ----
def _softmax64(x):
    x = x.astype(np.float64)
    e = np.exp(x - x.max())
    return e / e.sum()


@pytest.mark.parametrize("seed", range(4))
def test_threshold_selection_against_numpy_softmax(seed):
    r = np.random.default_rng(100 + seed)
    B, Hkv, b, max_blocks, max_sel = 2, 2, 16, 60, 60
    lens = np.array([60 * 16, 23 * 16 + 5], np.int32)
    sc = (r.normal(size=(B, Hkv, max_blocks)) * 2.0).astype(np.float32)
    tau = [0.002, 0.006, 0.02, 0.5][seed]
    idx, cnt, probs = oracle.select_threshold(sc, lens, b, tau, max_sel)
    for i in range(B):
        n = -(-int(lens[i]) // b)
        for h in range(Hkv):
            p = _softmax64(sc[i, h, : n - 1])
            assert np.allclose(probs[i, h, : n - 1], p, rtol=1e-12) and abs(p.sum() - 1.0) < 1e-12
            want = sorted([j for j in range(n - 1) if p[j] > tau] + [n - 1])
            assert list(idx[i, h, : cnt[i, h]]) == want
            assert np.all(idx[i, h, cnt[i, h]:] == -1)


def test_threshold_closed_forms_and_truncation():
    # equal scores: every block has probability 1/(n-1)
    sc = np.zeros((1, 1, 9), np.float32)
    idx, cnt, _ = oracle.select_threshold(sc, [9 * 4], 4, 0.124, 9)       # 1/8 > 0.124: all
    assert list(idx[0, 0]) == list(range(9))
    idx, cnt, _ = oracle.select_threshold(sc, [9 * 4], 4, 0.125, 9)       # 1/8 > 1/8 is false: last only
    assert list(idx[0, 0, :1]) == [8] and cnt[0, 0] == 1
    # one dominant block
    sc[0, 0, 3] = 30.0
    idx, cnt, _ = oracle.select_threshold(sc, [9 * 4], 4, 0.5, 9)
    assert list(idx[0, 0, :2]) == [3, 8] and cnt[0, 0] == 2
    # the last block's own score plays no role, and a shift of all scores changes nothing
    sc2 = sc + np.float32(5.0)
    sc2[0, 0, 8] = 1e9
    a = oracle.select_threshold(sc2, [9 * 4], 4, 0.5, 9)
    assert np.array_equal(a[0], idx)
    # more blocks pass than fit: the highest-scoring max_sel-1 are kept (ties: lower index)
    sc3 = np.array([[[1, 3, 2, 3, 0, 1, 9]]], np.float32)
    idx, cnt, _ = oracle.select_threshold(sc3, [7 * 4], 4, 1e-6, 4)       # all six pass, room for three
    assert list(idx[0, 0]) == [1, 2, 3, 6] and cnt[0, 0] == 4
    # a single block: nothing to normalise over
    idx, cnt, _ = oracle.select_threshold(sc3, [3], 4, 0.1, 4)
    assert list(idx[0, 0]) == [0, -1, -1, -1] and cnt[0, 0] == 1


# ---- selection for several query tokens: the blocks holding the query tokens are forced ----------

def test_multi_token_selection_with_one_token_is_the_single_token_selection():
    r = np.random.default_rng(11)
    sc = r.normal(size=(3, 2, 40)).astype(np.float32)
    lens = np.array([40 * 16, 17 * 16 - 5, 3], np.int32)
    for budget, max_sel in [(16 * 7, 12), (16 * 100, 40), (0, 4)]:
        a = oracle.select(sc, lens, 16, budget, max_sel)
        m = oracle.select_multi(sc, lens, 16, budget, 1, max_sel)
        assert np.array_equal(a[0], m[0]) and np.array_equal(a[1], m[1])


@pytest.mark.parametrize("T", [2, 5, 8])
def test_multi_token_selection_against_lexsort_with_forced_blocks(T):
    r = np.random.default_rng(20 + T)
    B, Hkv, b, max_blocks, max_sel = 5, 2, 16, 40, 12
    # 640: the T tokens sit in the last block; 16*17+3: they straddle two blocks (for T > 3);
    # 16*9: exactly at a block end; 4: shorter than a block; 2: shorter than T for T > 2
    lens = np.array([640, 16 * 17 + 3, 16 * 9, 4, 2], np.int32)
    sc = np.round(r.normal(size=(B, Hkv, max_blocks)).astype(np.float32) * 3) / 3
    for budget in (16 * 7, 16 * 2, 16, 16 * 100):
        idx, cnt = oracle.select_multi(sc, lens, b, budget, T, max_sel)
        for i in range(B):
            L = int(lens[i])
            n = -(-L // b)
            jf = max(0, L - T) // b
            forced = list(range(jf, n))
            k = min(max(1, budget // b), n, max_sel)
            need = min(max(0, k - len(forced)), jf)
            for h in range(Hkv):
                order = np.lexsort((np.arange(jf), -sc[i, h, :jf].astype(np.float64)))
                want = sorted(list(order[:need]) + forced)
                assert cnt[i, h] == len(want)
                assert list(idx[i, h, :len(want)]) == want
                assert np.all(idx[i, h, len(want):] == -1)
                # every query token's own block is there
                for t in range(T):
                    pos = L - T + t
                    if pos >= 0:
                        assert pos // b in want


# ---- threshold selection for several query tokens ----------------------------------------------------

def test_threshold_multi_with_one_token_is_the_single_token_routine():
    r = np.random.default_rng(321)
    B, Hkv, b, max_blocks = 3, 2, 16, 50
    lens = np.array([50 * 16, 31 * 16 + 7, 16], np.int32)
    sc = (r.normal(size=(B, Hkv, max_blocks)) * 2.0).astype(np.float32)
    for tau in (0.004, 0.03):
        for max_sel in (50, 7):
            a = oracle.select_threshold(sc, lens, b, tau, max_sel)
            m = oracle.select_threshold_multi(sc, lens, b, tau, 1, max_sel)
            assert np.array_equal(a[0], m[0]) and np.array_equal(a[1], m[1])
            assert np.allclose(a[2], m[2], rtol=0, atol=0)


@pytest.mark.parametrize("T", [2, 5, 8])
def test_threshold_multi_against_numpy_softmax_and_forced_range(T):
    r = np.random.default_rng(400 + T)
    B, Hkv, b, max_blocks, max_sel = 4, 2, 16, 40, 40
    # the T tokens inside one block; straddling two blocks; exactly filling a block's end; fewer tokens than T
    lens = np.array([40 * 16, 21 * 16 + 2, 30 * 16, 3], np.int32)
    sc = (r.normal(size=(B, Hkv, max_blocks)) * 2.0).astype(np.float32)
    tau = 0.03
    idx, cnt, probs = oracle.select_threshold_multi(sc, lens, b, tau, T, max_sel)
    for i in range(B):
        L = int(lens[i])
        n = -(-L // b)
        jf = max(0, L - T) // b
        forced = list(range(jf, n))
        for h in range(Hkv):
            got = list(idx[i, h, : cnt[i, h]])
            if jf:
                p = _softmax64(sc[i, h, :jf])
                assert np.allclose(probs[i, h, :jf], p, rtol=1e-12)
                want = sorted([j for j in range(jf) if p[j] > tau] + forced)
            else:
                want = forced
            assert got == want and np.all(idx[i, h, cnt[i, h]:] == -1)
    # the forced blocks' own scores play no role
    sc2 = sc.copy()
    for i in range(B):
        jf = max(0, int(lens[i]) - T) // b
        sc2[i, :, jf:] = 1e9
    idx2, cnt2, _ = oracle.select_threshold_multi(sc2, lens, b, tau, T, max_sel)
    assert np.array_equal(idx2, idx) and np.array_equal(cnt2, cnt)


def test_threshold_multi_truncation_keeps_the_best_beside_the_forced_blocks():
    # blocks of 4 tokens, L = 30: n = 8 blocks; T = 3 tokens at positions 27..29: jf = 6, forced {6, 7}
    sc = np.array([[[1, 3, 2, 3, 0, 1, 9, 9]]], np.float32)
    idx, cnt, _ = oracle.select_threshold_multi(sc, [30], 4, 1e-6, 3, 4)     # all six pass, room for two
    assert list(idx[0, 0]) == [1, 3, 6, 7] and cnt[0, 0] == 4               # (ties: the lower index first)
    idx, cnt, _ = oracle.select_threshold_multi(sc, [30], 4, 0.9, 3, 4)      # nothing passes: the forced only
    assert list(idx[0, 0, :2]) == [6, 7] and cnt[0, 0] == 2
