"""Pins of the oracle's chunked-prefill routines: a chunk (the last S_q positions of each sequence, starting on a block
boundary) must reproduce the corresponding rows of the whole problem, which the other oracle tests pin; plus a
single-query case written out by hand."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W


def make_chunk(w, starts):
    """Full workload -> (q_chunk bits, cu_q): the queries from `starts[b]` (tokens) to the end of each sequence."""
    cu = w.cu_seqlens
    parts, cu_q = [], [0]
    for b, st in enumerate(starts):
        parts.append(w.q[cu[b] + st:cu[b + 1]])
        cu_q.append(cu_q[-1] + int(cu[b + 1] - cu[b] - st))
    return np.concatenate(parts, axis=0), np.asarray(cu_q, dtype=np.int32)


@pytest.fixture(scope="module")
def case():
    lens, starts = [200, 64, 333, 130], [128, 0, 192, 130]         # the last sequence contributes no query
    w = W.make_small(seed=4242, seqlens=lens, hq=4, hkv=2, q_gain=2.0)
    qc, cu_q = make_chunk(w, starts)
    return w, lens, starts, qc, cu_q


def test_chunk_offsets_and_validation(case):
    w, lens, starts, qc, cu_q = case
    assert O.chunk_offsets(cu_q, w.cu_seqlens, 64).tolist() == [2, 0, 3, 3]
    with pytest.raises(ValueError):
        O.chunk_offsets([0, 100], [0, 200], 64)                     # starts at token 100: not a block boundary
    with pytest.raises(ValueError):
        O.chunk_offsets([0, 300], [0, 200], 64)


@pytest.mark.parametrize("theta", [0.0, 10000.0])
def test_chunk_gate_scores_are_rows_of_the_whole(case, theta):
    w, lens, starts, qc, cu_q = case
    wk3 = W.make_gate_weights(7, 2, 3 * 128)
    full = O.gate_scores_ex(w.q, w.k, w.wq, wk3, w.cu_seqlens, 64, pool_k=7, rope_theta=theta)
    part = O.gate_scores_chunk(qc, w.k, w.wq, wk3, cu_q, w.cu_seqlens, 64, pool_k=7, rope_theta=theta)
    offs = O.chunk_offsets(cu_q, w.cu_seqlens, 64)
    for b, st in enumerate(starts):
        off = int(offs[b])
        assert part[b].shape == (4, full[b].shape[1] - off, full[b].shape[2])
        np.testing.assert_array_equal(part[b], full[b][:, off:, :])


def test_chunk_lists_and_attention_are_rows_of_the_whole(case):
    w, lens, starts, qc, cu_q = case
    full_s = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 64)
    part_s = O.gate_scores_chunk(qc, w.k, w.wq, w.wk, cu_q, w.cu_seqlens, 64)
    kw = dict(keep_num=1, keep_den=2, flags=3)
    rp_f, col_f = O.block_mask(full_s, O.MODE_TOPK_RATIO, **kw)
    rp_c, col_c = O.block_mask_chunk(part_s, O.MODE_TOPK_RATIO, **kw)
    assert len(rp_c) == len(rp_f)
    r = 0
    offs = O.chunk_offsets(cu_q, w.cu_seqlens, 64)
    for b, (S, st) in enumerate(zip(lens, starts)):
        nb = (S + 63) // 64
        for h in range(4):
            for i in range(nb):
                got = col_c[rp_c[r]:rp_c[r + 1]].tolist()
                want = col_f[rp_f[r]:rp_f[r + 1]].tolist() if i >= int(offs[b]) else []
                assert got == want, (b, h, i)
                r += 1
    sc = 1 / math.sqrt(128)
    o_f, lse_f = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp_f, col_f, 4, 2, 64, sc)
    o_c, lse_c = O.sparse_attention_chunk(qc, w.k, w.v, cu_q, w.cu_seqlens, rp_c, col_c, 4, 2, 64, sc)
    for b, st in enumerate(starts):
        k0, k1 = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        q0, q1 = int(cu_q[b]), int(cu_q[b + 1])
        np.testing.assert_allclose(o_c[q0:q1], o_f[k0 + st:k1], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(lse_c[:, q0:q1], lse_f[:, k0 + st:k1], rtol=1e-12, atol=1e-14)


def test_single_query_chunk_by_hand():
    """One query at the last position of a 130-token sequence, lists {0, 2} of its row (block 2): it sees tokens 0..63
    and 128..129; softmax and weighted sum written out with python floats."""
    w = W.make_small(seed=4243, seqlens=[130], hq=1, hkv=1)
    qc = w.q[129:130]
    rp = np.array([0, 0, 0, 2]); col = np.array([0, 2])
    sc = 0.25
    o, lse = O.sparse_attention_chunk(qc, w.k, w.v, [0, 1], [0, 130], rp, col, 1, 1, 64, sc)
    qf = O.bf16_bits_to_f64(qc[0, 0]); kf = O.bf16_bits_to_f64(w.k[:, 0]); vf = O.bf16_bits_to_f64(w.v[:, 0])
    keys = list(range(64)) + [128, 129]
    logits = [sc * sum(float(a) * float(b) for a, b in zip(qf, kf[t])) for t in keys]
    mx = max(logits)
    e = [math.exp(x - mx) for x in logits]
    z = sum(e)
    want = [sum(e[n] * float(vf[t][c]) for n, t in enumerate(keys)) / z for c in range(128)]
    np.testing.assert_allclose(o[0, 0], want, rtol=1e-12, atol=1e-15)
    assert lse[0, 0] == pytest.approx(mx + math.log(z), rel=1e-13)
