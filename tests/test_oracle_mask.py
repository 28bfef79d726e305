"""Pins for the mask oracle (Sec. 3.3, Eq. 3 TopK and Eq. 4 threshold): brute
force by a full Python sort, closed-form counts, nesting and degenerate
thresholds."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O

RATIO, COUNT, THR = O.MODE_TOPK_RATIO, O.MODE_TOPK_COUNT, O.MODE_THRESHOLD
DIAG, SINK = O.FORCE_DIAG, O.FORCE_SINK


def brute_topk(s, i, ki, flags):
    """Give forced blocks the best possible rank, sort every causal block by
    (forced first, score descending, index ascending), keep the first ki
    (all forced ones if there are more of them)."""
    n = i + 1
    forced = [j for j in range(n) if (j == i and flags & DIAG) or (j == 0 and flags & SINK)]
    others = [j for j in range(n) if j not in forced and not math.isnan(float(s[j]))]
    others = sorted(others, key=lambda j: (-float(s[j]), j))
    return sorted(forced + others[:max(ki - len(forced), 0)])


def random_scores(rng, nb, hq=1, quantise=None):
    s = rng.random((hq, nb, nb)).astype(np.float32)
    if quantise:
        s = (np.floor(s * quantise) / quantise).astype(np.float32)   # many exact ties
    return s


def test_keep_count_closed_forms():
    assert [O.keep_count(n, RATIO, 1, 2) for n in (1, 2, 3, 4, 5)] == [1, 1, 2, 2, 3]
    assert [O.keep_count(n, RATIO, 1, 10) for n in (1, 10, 11, 2048)] == [1, 1, 2, 205]
    assert O.keep_count(7, RATIO, 1, 1) == 7 and O.keep_count(7, RATIO, 3, 1) == 7
    assert O.keep_count(2048, RATIO, 1, 20) == 103                    # ceil(102.4)
    assert [O.keep_count(n, COUNT, k=3) for n in (1, 2, 3, 9)] == [1, 2, 3, 3]
    # exact rational: 3/10 of 10 is 3, never 4 as a float ceil(0.3*10) could give
    assert O.keep_count(10, RATIO, 3, 10) == 3


@pytest.mark.parametrize("flags", [0, DIAG, DIAG | SINK, SINK])
@pytest.mark.parametrize("quantise", [None, 4])
def test_topk_matches_full_sort(flags, quantise):
    rng = np.random.default_rng(10 + flags)
    S = random_scores(rng, 48, quantise=quantise)[0]
    for (num, den) in [(1, 2), (1, 4), (1, 10), (1, 1), (2, 3)]:
        for i in range(48):
            ki = O.keep_count(i + 1, RATIO, num, den)
            got = O.select_row(S[i], i, RATIO, keep_num=num, keep_den=den, flags=flags)
            assert got == brute_topk(S[i], i, ki, flags)
            nf = len({j for j in ([i] if flags & DIAG else []) + ([0] if flags & SINK else [])})
            assert len(got) == max(ki, nf)
            assert got == sorted(set(got)) and all(0 <= j <= i for j in got)
    for k in (0, 1, 5, 100):
        for i in range(48):
            assert O.select_row(S[i], i, COUNT, k=k, flags=flags) == brute_topk(S[i], i, min(k, i + 1), flags)


def test_topk_ties_go_to_lower_index():
    s = np.array([0.2, 0.5, 0.5, 0.5, 0.1, 0.5, 0.3], np.float32)      # row i = 6
    assert O.select_row(s, 6, COUNT, k=3, flags=0) == [1, 2, 3]
    assert O.select_row(s, 6, COUNT, k=3, flags=DIAG) == [1, 2, 6]      # diagonal takes one of the 3 places
    assert O.select_row(s, 6, COUNT, k=4, flags=DIAG | SINK) == [0, 1, 2, 6]
    assert O.select_row(s, 6, COUNT, k=1, flags=DIAG | SINK) == [0, 6]  # forced blocks exceed k
    z = np.array([0.0, -0.0, 0.0, -0.0], np.float32)                   # +0 and -0 are equal
    assert O.select_row(z, 3, COUNT, k=2, flags=0) == [0, 1]


def test_topk_nesting_and_full_ratio():
    rng = np.random.default_rng(3)
    S = random_scores(rng, 40)[0]
    for i in range(40):
        prev = set()
        for k in range(0, i + 2):
            cur = set(O.select_row(S[i], i, COUNT, k=k, flags=DIAG))
            assert prev <= cur
            prev = cur
        assert O.select_row(S[i], i, RATIO, keep_num=1, keep_den=1, flags=DIAG) == list(range(i + 1))


def test_nan_scores_never_selected_unless_forced():
    s = np.array([np.nan, 0.3, np.nan, 0.1, np.nan], np.float32)
    assert O.select_row(s, 4, COUNT, k=4, flags=0) == [1, 3]
    assert O.select_row(s, 4, COUNT, k=2, flags=DIAG) == [1, 4]
    assert O.select_row(s, 4, THR, threshold=-np.inf, flags=SINK) == [0, 1, 3]


def test_threshold_is_the_strict_bitmap_or_forced():
    rng = np.random.default_rng(4)
    S = random_scores(rng, 32, quantise=8)[0]
    for thr in (0.0, 0.125, 0.5, 0.875):
        for flags in (0, DIAG, DIAG | SINK):
            for i in range(32):
                bitmap = S[i, : i + 1] > np.float32(thr)                # Eq. 4
                if flags & DIAG:
                    bitmap[i] = True
                if flags & SINK:
                    bitmap[0] = True
                assert O.select_row(S[i], i, THR, threshold=thr, flags=flags) == np.flatnonzero(bitmap).tolist()
    # strictness: a score equal to the threshold is not kept
    assert O.select_row(np.array([0.5, 0.25], np.float32), 1, THR, threshold=0.5, flags=0) == []


def test_threshold_degenerate_and_nesting():
    rng = np.random.default_rng(5)
    S = random_scores(rng, 24)[0]
    for i in range(24):
        assert O.select_row(S[i], i, THR, threshold=-np.inf, flags=DIAG) == list(range(i + 1))
        assert O.select_row(S[i], i, THR, threshold=np.inf, flags=DIAG) == [i]
        assert O.select_row(S[i], i, THR, threshold=1.0, flags=DIAG | SINK) == sorted({0, i})
        a = set(O.select_row(S[i], i, THR, threshold=0.3, flags=DIAG))
        b = set(O.select_row(S[i], i, THR, threshold=0.6, flags=DIAG))
        assert b <= a


def test_threshold_compares_in_fp32():
    # 0.1 as fp32 is larger than the double 0.1: in fp32 they are equal -> not kept
    s = np.array([np.float32(0.1)], np.float32)
    assert O.select_row(s, 0, THR, threshold=0.1, flags=0) == []


def test_block_mask_csr_layout_and_row_ids():
    rng = np.random.default_rng(6)
    scores = [random_scores(rng, 3, hq=2), random_scores(rng, 5, hq=2)]
    row_ptr, col = O.block_mask(scores, COUNT, k=2, flags=DIAG)
    assert row_ptr.shape == (2 * 3 + 2 * 5 + 1,) and row_ptr[0] == 0 and row_ptr[-1] == len(col)
    # row id of (b, h, i) = Hq*off_b + h*nb_b + i
    r = 2 * 3 + 1 * 5 + 4
    assert col[row_ptr[r]:row_ptr[r + 1]].tolist() == O.select_row(scores[1][1, 4], 4, COUNT, k=2, flags=DIAG)
    counts = np.diff(row_ptr)
    want = [min(2, i + 1) for _h in range(2) for i in range(3)] + [min(2, i + 1) for _h in range(2) for i in range(5)]
    assert counts.tolist() == want
    fp, fc = O.full_causal_lists([0, 5, 12], 4, 2)
    assert np.diff(fp).tolist() == [1, 2, 1, 2, 1, 2, 1, 2] and fc[:3].tolist() == [0, 0, 1]


def test_dense_tail_keeps_the_last_query_blocks_whole():
    """Sec. 4: sparsity in the context, dense on the question.  Closed forms: the last `dense_tail` rows of every
    (sequence, head) list all their causal blocks, the other rows are untouched; a tail as long as the sequence gives
    the full causal lists; a tail of zero changes nothing."""
    rng = np.random.default_rng(7)
    scores = [random_scores(rng, 6, hq=2), random_scores(rng, 2, hq=2), random_scores(rng, 9, hq=2)]
    base_rp, base_col = O.block_mask(scores, COUNT, k=2, flags=DIAG)
    rp0, col0 = O.block_mask(scores, COUNT, k=2, flags=DIAG, dense_tail=0)
    assert np.array_equal(rp0, base_rp) and np.array_equal(col0, base_col)
    rp, col = O.block_mask(scores, COUNT, k=2, flags=DIAG, dense_tail=3)
    r = 0
    for nb in (6, 2, 9):
        for _h in range(2):
            for i in range(nb):
                got = col[rp[r]:rp[r + 1]].tolist()
                if i >= nb - 3:
                    assert got == list(range(i + 1))
                else:
                    assert got == base_col[base_rp[r]:base_rp[r + 1]].tolist()
                r += 1
    frp, fcol = O.block_mask(scores, THR, threshold=2.0, flags=0, dense_tail=9)
    wrp, wcol = O.full_causal_lists([0, 6 * 4, 8 * 4, 17 * 4], 4, 2)
    assert np.array_equal(frp, wrp) and np.array_equal(fcol, wcol)
