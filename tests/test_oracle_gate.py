"""Pins for the gate oracle (Sec. 3.1, Eq. 1): closed forms, invariants and a
loop-level brute force on tiny inputs.  None of these re-uses the oracle's own
code path to produce the expected value."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W


def bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def small(seed, seqlens, hq, hkv, **kw):
    return W.make_small(seed, seqlens, hq, hkv, **kw)


def test_bf16_conversion_exact():
    vals = np.array([0.0, 1.0, -2.5, 0.15625, 3.0e38, -1.0e-30], dtype=np.float32)
    b = bits(vals)
    back = O.bf16_bits_to_f64(b)
    # bf16 keeps 8 significant bits: representable values survive, others move by < 2^-8 relative
    assert back[0] == 0.0 and back[1] == 1.0 and back[2] == -2.5 and back[3] == 0.15625
    assert np.all(np.abs(back - vals.astype(np.float64)) <= np.abs(vals) * 2.0 ** -8)
    assert O.bf16_bits_to_f64(np.array([0x3F80, 0xC000, 0x7F80], np.uint16)).tolist() == [1.0, -2.0, np.inf]


def test_pool_constant_block_and_ragged_tail():
    B, d = 4, 8
    # sequence of 10 tokens -> blocks of 4, 4, 2 tokens; token t holds the value t in every channel
    x = np.repeat(np.arange(10, dtype=np.float32)[:, None, None], d, axis=2)
    p = O.pool_avg(bits(x), [0, 10], B)[0]
    assert p.shape == (1, 3, d)
    np.testing.assert_array_equal(p[0, :, 0], [1.5, 5.5, 8.5])      # tail averages its 2 valid tokens
    c = np.full((8, 2, d), 0.75, np.float32)
    np.testing.assert_array_equal(O.pool_avg(bits(c), [0, 8], B)[0], np.full((2, 2, d), 0.75))


def test_pool_respects_sequence_boundaries():
    B, d = 4, 4
    x = np.zeros((9, 1, d), np.float32)
    x[:5] = 1.0          # sequence 0: 5 tokens of ones; sequence 1: 4 tokens of zeros
    p = O.pool_avg(bits(x), [0, 5, 9], B)
    np.testing.assert_array_equal(p[0][0, :, 0], [1.0, 1.0])         # tail block of seq 0 does not read seq 1
    np.testing.assert_array_equal(p[1][0, :, 0], [0.0])


def test_project_identity_and_single_entry_matrices():
    r = np.random.default_rng(0)
    pooled = r.standard_normal((2, 5, 6))
    eye = np.stack([np.eye(6)] * 2)
    np.testing.assert_array_equal(O.project(pooled, eye), pooled)
    # W[h] with a single 1 at (c0, o0): out[..., o0] = pooled[..., c0]; a transposed W would read channel o0
    Wm = np.zeros((2, 6, 3))
    Wm[0, 4, 1] = 1.0
    Wm[1, 2, 0] = 1.0
    out = O.project(pooled, Wm)
    np.testing.assert_array_equal(out[0, :, 1], pooled[0, :, 4])
    np.testing.assert_array_equal(out[1, :, 0], pooled[1, :, 2])
    assert np.count_nonzero(out[0, :, [0, 2]]) == 0


def test_pool_then_project_commutes_with_project_then_pool():
    # linearity: averaging the per-token projections equals projecting the average
    w = small(1, [24], 3, 1, block=8, head_dim=16, gate_dim=5)
    qf = O.bf16_bits_to_f64(w.q)                                     # [T, H, d]
    per_token = np.einsum("thc,hco->tho", qf, w.wq.astype(np.float64))
    avg_of_proj = per_token.reshape(3, 8, 3, 5).mean(axis=1).transpose(1, 0, 2)
    proj_of_avg = O.project(O.pool_avg(w.q, w.cu_seqlens, 8)[0], w.wq)
    np.testing.assert_allclose(proj_of_avg, avg_of_proj, rtol=0, atol=1e-12)


def test_logits_closed_form_rank_one():
    # Q block i constant x_i*e_0, K block j constant y_j*e_0, Wq = E(0->2), Wk = E(0->2):
    # logit = x_i*y_j/sqrt(dg); softmax over j<=i in closed form.
    B, d, dg, nb = 2, 4, 9, 4
    xs = np.array([1.0, -2.0, 0.5, 3.0])
    ys = np.array([0.25, 1.0, -1.5, 2.0])
    q = np.zeros((nb * B, 1, d), np.float32)
    k = np.zeros((nb * B, 1, d), np.float32)
    q[:, 0, 0] = np.repeat(xs, B)
    k[:, 0, 0] = np.repeat(ys, B)
    wq = np.zeros((1, d, dg), np.float32)
    wk = np.zeros((1, d, dg), np.float32)
    wq[0, 0, 2] = 1.0
    wk[0, 0, 2] = 1.0
    s = O.gate_scores(bits(q), bits(k), wq, wk, [0, nb * B], B)[0]
    assert s.shape == (1, nb, nb) and s.dtype == np.float32
    for i in range(nb):
        e = [math.exp(xs[i] * ys[j] / 3.0) for j in range(i + 1)]
        for j in range(nb):
            want = e[j] / sum(e) if j <= i else 0.0
            assert abs(float(s[0, i, j]) - want) <= 1e-7


def test_scores_brute_force_loops_gqa():
    # explicit loops over every index of Eq. 1 on a tiny GQA layer (2 KV heads, G = 2, ragged tail)
    w = small(2, [7, 5], 4, 2, block=2, head_dim=4, gate_dim=3, w_std=1.0)
    got = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 2)
    qf, kf = O.bf16_bits_to_f64(w.q), O.bf16_bits_to_f64(w.k)
    for b in range(2):
        s0, s1 = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        nb = (s1 - s0 + 1) // 2
        for h in range(4):
            g = h // 2
            for i in range(nb):
                logits = []
                for j in range(i + 1):
                    tq = range(s0 + 2 * i, min(s0 + 2 * i + 2, s1))
                    tk = range(s0 + 2 * j, min(s0 + 2 * j + 2, s1))
                    acc = 0.0
                    for o in range(3):
                        a = sum(sum(qf[t, h, c] for t in tq) / len(tq) * float(w.wq[h, c, o]) for c in range(4))
                        bb = sum(sum(kf[t, g, c] for t in tk) / len(tk) * float(w.wk[g, c, o]) for c in range(4))
                        acc += a * bb
                    logits.append(acc / math.sqrt(3.0))
                mx = max(logits)
                den = sum(math.exp(x - mx) for x in logits)
                for j in range(i + 1):
                    assert abs(float(got[b][h, i, j]) - math.exp(logits[j] - mx) / den) <= 2e-7
                assert np.all(got[b][h, i, i + 1:] == 0)


@pytest.mark.parametrize("zero", ["wq", "wk", "constk"])
def test_uniform_rows_when_logits_are_constant(zero):
    w = small(3, [40], 2, 1, block=4, head_dim=8, gate_dim=8, w_std=1.0)
    wq, wk, k = w.wq.copy(), w.wk.copy(), w.k.copy()
    if zero == "wq":
        wq[:] = 0
    elif zero == "wk":
        wk[:] = 0
    else:
        k[:] = k[0:1]                                                # every key identical -> pooled K constant
    s = O.gate_scores(w.q, k, wq, wk, w.cu_seqlens, 4)[0]
    for i in range(10):
        np.testing.assert_allclose(s[:, i, : i + 1], 1.0 / (i + 1), rtol=1e-6)


def test_rows_sum_to_one_row0_is_one_shape_and_shift_invariance():
    w = small(4, [640], 4, 2)
    s = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 64)[0]
    assert s.shape == (4, 10, 10)                                    # [seq/B, seq/B] per head
    assert s.size * 4096 == 4 * 640 * 640                            # 1/4096 of the attention map at B = 64
    np.testing.assert_allclose(s.astype(np.float64).sum(axis=2), 1.0, atol=1e-6)
    assert np.all(s[:, 0, 0] == 1.0)
    assert np.all(np.triu(s, 1) == 0) and np.all(s[:, np.tril_indices(10)[0], np.tril_indices(10)[1]] > 0)
    # a constant added to every logit of a row leaves the softmax unchanged
    L = np.random.default_rng(0).standard_normal((2, 6, 6))
    shift = np.arange(6.0)[None, :, None] * 3.0
    np.testing.assert_allclose(O.causal_softmax_rows(L + shift), O.causal_softmax_rows(L), atol=1e-15)


def test_gqa_head_mapping_is_h_div_g():
    # make KV head 1's keys all zero: query heads 2,3 (G = 2) must see uniform rows, heads 0,1 must not
    w = small(5, [32], 4, 2, block=4, head_dim=8, gate_dim=8, w_std=1.0)
    k = w.k.copy()
    k[:, 1, :] = 0
    s = O.gate_scores(w.q, k, w.wq, w.wk, w.cu_seqlens, 4)[0]
    for i in range(8):
        np.testing.assert_allclose(s[2:, i, : i + 1], 1.0 / (i + 1), rtol=1e-6)
    assert np.abs(s[0, 7, :8] - 1 / 8).max() > 1e-3 and np.abs(s[1, 7, :8] - 1 / 8).max() > 1e-3


def test_flatten_roundtrip_layout():
    w = small(6, [10, 4, 7], 3, 1, block=4, head_dim=8, gate_dim=8)
    s = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 4)
    flat = O.flatten_scores(s)
    assert flat.size == 3 * (9 + 1 + 4)
    # sequence 1 starts after Hq * nb_0^2 entries, laid out [h][i][j]
    assert flat[3 * 9] == s[1][0, 0, 0] and flat[3 * 9 + 3 * 1 + 1 * 4 + 2 + 0] == s[2][1, 1, 0]
    back = O.unflatten_scores(flat, w.cu_seqlens, 4, 3)
    for a, b in zip(s, back):
        np.testing.assert_array_equal(a, b)
