"""Pins of the oracle's AttnGate variants (Sec. 3.1: composed avg/max/min pooling, block-level RoPE with theta / B).

Each check compares the oracle with something other than itself: a closed form, an invariant, a textbook rotation, or
a brute-force evaluation written in a different way."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W


def _bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _rand_bits(rng, shape):
    return _bits(rng.standard_normal(shape))


def test_pool_compose_avg_alone_is_pool_avg():
    rng = np.random.default_rng(1)
    x = _rand_bits(rng, (150, 3, 8))
    cu = [0, 70, 150]
    a = O.pool_compose(x, cu, 16, O.POOL_AVG)
    b = O.pool_avg(x, cu, 16)
    for u, v in zip(a, b):
        np.testing.assert_array_equal(u, v)


def test_pool_compose_brute_force_and_order():
    """avg | max | min concatenated in that order; ragged tail pools the tokens it has (python loops per element)."""
    rng = np.random.default_rng(2)
    T, H, d, B = 37, 2, 4, 8
    x = _rand_bits(rng, (T, H, d))
    xf = O.bf16_bits_to_f64(x)
    got = O.pool_compose(x, [0, T], B, O.POOL_AVG | O.POOL_MAX | O.POOL_MIN)[0]
    nb = (T + B - 1) // B
    assert got.shape == (H, nb, 3 * d)
    for h in range(H):
        for i in range(nb):
            toks = range(i * B, min((i + 1) * B, T))
            for c in range(d):
                vals = [xf[t, h, c] for t in toks]
                assert got[h, i, c] == pytest.approx(sum(vals) / len(vals), rel=1e-15, abs=1e-15)
                assert got[h, i, d + c] == max(vals)
                assert got[h, i, 2 * d + c] == min(vals)
    # a subset keeps the order of the remaining parts
    mm = O.pool_compose(x, [0, T], B, O.POOL_MAX | O.POOL_MIN)[0]
    np.testing.assert_array_equal(mm[..., :d], got[..., d:2 * d])
    np.testing.assert_array_equal(mm[..., d:], got[..., 2 * d:])


def test_pool_compose_invariants():
    rng = np.random.default_rng(3)
    x = _rand_bits(rng, (64, 2, 8))
    p = O.pool_compose(x, [0, 64], 16, 7)[0]
    avg, mx, mn = p[..., :8], p[..., 8:16], p[..., 16:]
    assert np.all(mx >= avg) and np.all(avg >= mn)
    const = _bits(np.full((32, 1, 4), 0.75))
    pc = O.pool_compose(const, [0, 32], 16, 7)[0]
    np.testing.assert_array_equal(pc, np.full((1, 2, 12), 0.75))
    with pytest.raises(ValueError):
        O.pool_compose(x, [0, 64], 16, 0)
    with pytest.raises(ValueError):
        O.pool_compose(x, [0, 64], 16, 8)


def test_gate_scores_ex_reduces_to_eq1():
    """Defaults are Eq. 1; a K matrix whose max and min rows are zero reads only the average part."""
    rng = np.random.default_rng(4)
    T, Hq, Hkv, d, dg, B = 96, 4, 2, 8, 8, 16
    q, k = _rand_bits(rng, (T, Hq, d)), _rand_bits(rng, (T, Hkv, d))
    wq = rng.standard_normal((Hq, d, dg)).astype(np.float32)
    wk = rng.standard_normal((Hkv, d, dg)).astype(np.float32)
    base = O.gate_scores(q, k, wq, wk, [0, T], B)
    same = O.gate_scores_ex(q, k, wq, wk, [0, T], B)
    np.testing.assert_array_equal(base[0], same[0])
    wk3 = np.zeros((Hkv, 3 * d, dg), dtype=np.float32)
    wk3[:, :d] = wk
    ext = O.gate_scores_ex(q, k, wq, wk3, [0, T], B, pool_k=7)
    np.testing.assert_array_equal(base[0], ext[0])
    # and a matrix that reads only the max part equals Eq. 1 evaluated on the max-pooled K
    wkm = np.zeros((Hkv, 3 * d, dg), dtype=np.float32)
    wkm[:, d:2 * d] = wk
    got = O.gate_scores_ex(q, k, wq, wkm, [0, T], B, pool_k=7)[0]
    kf = O.bf16_bits_to_f64(k).reshape(T // B, B, Hkv, d).max(axis=1).transpose(1, 0, 2)      # [Hkv, nb, d]
    gq = O.project(O.pool_avg(q, [0, T], B)[0], wq)
    gk = np.einsum("hic,hco->hio", kf, wk.astype(np.float64))
    want = O.causal_softmax_rows(O.gate_logits(gq, gk)).astype(np.float32)
    np.testing.assert_array_equal(got, want)


def test_block_rope_is_a_plane_rotation():
    """dg = 2: one pair, frequency theta'^0 = 1, so block i is rotated by i radians (textbook 2-D rotation)."""
    g = np.zeros((1, 5, 2))
    g[..., 0] = 1.0
    r = O.block_rope(g, 10000.0, 64)
    for i in range(5):
        assert r[0, i, 0] == pytest.approx(math.cos(i), abs=1e-15)
        assert r[0, i, 1] == pytest.approx(math.sin(i), abs=1e-15)
    g2 = np.zeros((1, 3, 2))
    g2[..., 1] = 1.0
    r2 = O.block_rope(g2, 10000.0, 64)
    assert r2[0, 1, 0] == pytest.approx(-math.sin(1.0), abs=1e-15)
    assert r2[0, 1, 1] == pytest.approx(math.cos(1.0), abs=1e-15)


def test_block_rope_uses_theta_over_block():
    """dg = 4: the second pair has frequency (theta / B)^(-1/2); theta = 6400, B = 64 gives 0.1, so block 10 turns 1 rad."""
    g = np.zeros((1, 11, 4))
    g[..., 1] = 1.0                                  # first element of the second pair (1, 3)
    r = O.block_rope(g, 6400.0, 64)
    assert r[0, 10, 1] == pytest.approx(math.cos(1.0), abs=1e-14)
    assert r[0, 10, 3] == pytest.approx(math.sin(1.0), abs=1e-14)
    assert r[0, 10, 0] == 0.0 and r[0, 10, 2] == 0.0


def test_block_rope_invariants():
    rng = np.random.default_rng(5)
    g = rng.standard_normal((3, 9, 16))
    r = O.block_rope(g, 500000.0, 64)
    np.testing.assert_array_equal(r[:, 0], g[:, 0])                                   # position 0 is not rotated
    np.testing.assert_allclose((r ** 2).sum(-1), (g ** 2).sum(-1), rtol=1e-13)       # norms are kept
    # relative property: with the same vector at every position, <rope(a, i), rope(b, j)> depends on i - j only
    a, b = rng.standard_normal(16), rng.standard_normal(16)
    ra = O.block_rope(np.tile(a, (1, 9, 1)), 500000.0, 64)[0]
    rb = O.block_rope(np.tile(b, (1, 9, 1)), 500000.0, 64)[0]
    L = ra @ rb.T
    for off in range(-8, 9):
        diag = np.diagonal(L, offset=off)
        np.testing.assert_allclose(diag, diag[0], rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.diagonal(L), a @ b, atol=1e-12)                    # offset 0: the plain dot product


def test_gate_scores_ex_rope_closed_form_on_constant_input():
    """Identical tokens: every block pools and projects to the same vectors u (queries) and v (keys), so the logit of
    (i, j) is the rotary form sum_c (u_c v_c + u_c' v_c') cos((i-j) f_c) + (u_c v_c' - u_c' v_c) sin((i-j) f_c),
    written out here from the rotation, and the score row is its softmax over j <= i."""
    rng = np.random.default_rng(6)
    T, d, dg, B, theta = 80, 4, 4, 8, 800.0
    tok_q, tok_k = rng.standard_normal(d), rng.standard_normal(d)
    q = _bits(np.tile(tok_q, (T, 1, 1)))
    k = _bits(np.tile(tok_k, (T, 1, 1)))
    wq = rng.standard_normal((1, d, dg)).astype(np.float32)
    wk = rng.standard_normal((1, d, dg)).astype(np.float32)
    got = O.gate_scores_ex(q, k, wq, wk, [0, T], B, rope_theta=theta)[0][0]
    u = O.bf16_bits_to_f64(q[0, 0]) @ wq[0].astype(np.float64)
    v = O.bf16_bits_to_f64(k[0, 0]) @ wk[0].astype(np.float64)
    half = dg // 2
    f = [(theta / B) ** (-2.0 * c / dg) for c in range(half)]
    nb = T // B
    for i in range(nb):
        logits = []
        for j in range(i + 1):
            acc = 0.0
            for c in range(half):
                ang = (i - j) * f[c]
                acc += (u[c] * v[c] + u[c + half] * v[c + half]) * math.cos(ang)
                acc += (u[c] * v[c + half] - u[c + half] * v[c]) * math.sin(ang)
            logits.append(acc / math.sqrt(dg))
        mx = max(logits)
        e = [math.exp(x - mx) for x in logits]
        want = np.array([x / sum(e) for x in e])
        np.testing.assert_allclose(got[i, : i + 1], want, rtol=2e-7, atol=0)
        assert np.all(got[i, i + 1:] == 0)
    # no RoPE when theta is 0
    np.testing.assert_array_equal(O.gate_scores_ex(q, k, wq, wk, [0, T], B, rope_theta=0.0)[0], O.gate_scores(q, k, wq, wk, [0, T], B)[0])
