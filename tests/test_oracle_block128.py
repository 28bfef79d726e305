"""Pins for 128-token gate blocks: the rule that rewrites 128-token block lists as 64-token lists (block j -> 2j, 2j + 1;
row 2i of the diagonal block keeps 2i only) must select exactly the (query, key) pairs the 128-token lists select under
the causal mask.  Checked on the oracle alone: attention at B = 128 on the lists equals attention at B = 64 on the
rewritten lists, and the pair sets themselves are compared by brute force."""
import math

import numpy as np

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W


def expand_reference(cu, hq, rp128, col128):
    """The rule, written with python sets, independent of any kernel."""
    lens = np.diff(np.asarray(cu, dtype=np.int64))
    rp64, col64 = [0], []
    base128 = 0
    for S in lens:
        nb128, nb64 = (S + 127) // 128, (S + 63) // 64
        for h in range(hq):
            for i64 in range(nb64):
                src = base128 + h * nb128 + i64 // 2
                want = set()
                for j in col128[rp128[src]:rp128[src + 1]]:
                    for jj in (2 * int(j), 2 * int(j) + 1):
                        if jj <= i64:
                            want.add(jj)
                col64.extend(sorted(want))
                rp64.append(len(col64))
        base128 += hq * nb128
    return np.asarray(rp64, dtype=np.int64), np.asarray(col64, dtype=np.int64)


def pairs(cu, hq, B, rp, col):
    """All (head, query token, key token) triples the lists select under the causal mask."""
    out = set()
    lens = np.diff(np.asarray(cu, dtype=np.int64))
    base = 0
    for b, S in enumerate(lens):
        nb = (S + B - 1) // B
        for h in range(hq):
            for i in range(nb):
                r = base + h * nb + i
                for j in col[rp[r]:rp[r + 1]]:
                    for tq in range(i * B, min((i + 1) * B, S)):
                        for tk in range(int(j) * B, min((int(j) + 1) * B, S)):
                            if tk <= tq:
                                out.add((b, h, tq, tk))
        base += hq * nb
    return out


def random_lists(rng, cu, hq, B):
    lens = np.diff(np.asarray(cu, dtype=np.int64))
    rp, col = [0], []
    for S in lens:
        nb = (S + B - 1) // B
        for h in range(hq):
            for i in range(nb):
                keep = {i} if rng.random() < 0.8 else set()             # some rows without their diagonal block
                keep |= {int(j) for j in range(i + 1) if rng.random() < 0.4}
                col.extend(sorted(keep))
                rp.append(len(col))
    return np.asarray(rp, dtype=np.int64), np.asarray(col, dtype=np.int64)


def test_expansion_rule_selects_the_same_pairs():
    rng = np.random.default_rng(31)
    cu = np.array([0, 130, 130, 449, 513, 577], dtype=np.int64)       # ragged: 64-token tails, an empty sequence, one token over
    rp128, col128 = random_lists(rng, cu, 2, 128)
    rp64, col64 = expand_reference(cu, 2, rp128, col128)
    assert pairs(cu, 2, 128, rp128, col128) == pairs(cu, 2, 64, rp64, col64)
    # closed form of the lengths: 2 per off-diagonal entry, 1 (even row) or 2 (odd row) for the diagonal entry
    lens = np.diff(cu)
    r64 = 0
    base128 = 0
    for S in lens:
        nb128, nb64 = (S + 127) // 128, (S + 63) // 64
        for h in range(2):
            for i64 in range(nb64):
                src = base128 + h * nb128 + i64 // 2
                ent = col128[rp128[src]:rp128[src + 1]]
                n = 2 * int((ent < i64 // 2).sum()) + (int((ent == i64 // 2).sum()) * (2 if i64 % 2 else 1))
                assert rp64[r64 + 1] - rp64[r64] == n
                r64 += 1
        base128 += 2 * nb128


def test_attention_at_128_equals_attention_on_expanded_lists():
    rng = np.random.default_rng(32)
    lens = [200, 65, 384]
    w = W.make_small(seed=515, seqlens=lens, hq=2, hkv=1)
    rp128, col128 = random_lists(rng, w.cu_seqlens, 2, 128)
    rp64, col64 = expand_reference(w.cu_seqlens, 2, rp128, col128)
    sc = 1 / math.sqrt(128)
    o128, lse128 = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp128, col128, 2, 1, 128, sc)
    o64, lse64 = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp64, col64, 2, 1, 64, sc)
    np.testing.assert_allclose(o128, o64, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse128, lse64, rtol=1e-12, atol=1e-14)


def test_gate_at_128_pools_pairs_of_64_blocks():
    """A 128-token average is the mean of its two 64-token averages when both are full (a relation between two block
    sizes of the same oracle routine, through a different path: pool at 64, then average pairs by hand)."""
    w = W.make_small(seed=516, seqlens=[512], hq=2, hkv=1)
    p64 = O.pool_avg(w.q, w.cu_seqlens, 64)[0]
    p128 = O.pool_avg(w.q, w.cu_seqlens, 128)[0]
    np.testing.assert_allclose(p128, 0.5 * (p64[:, 0::2] + p64[:, 1::2]), rtol=1e-13, atol=1e-15)
