"""GPU parity of seer_gate_scores_ex (Sec. 3.1: composed avg/max/min pooling, block-level RoPE) against the oracle.

Tolerance as for the plain gate: |x - ref| <= 1e-3 |ref| on every causal entry (absolute 1e-33 below 1e-30)."""
import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rt():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests must run on a B200")
    from paper_2410_13276_b200 import binding as B
    from paper_2410_13276_b200.prefill import Prefill
    ctx = B.Context(0)
    yield B, Prefill, ctx
    ctx.close()


def check_scores(got_flat, ref_list, w):
    got = O.unflatten_scores(got_flat, w.cu_seqlens, w.block, w.num_q_heads)
    for g, r in zip(got, ref_list):
        nb = r.shape[-1]
        il = np.tril_indices(nb)
        gg, rr = g[:, il[0], il[1]].astype(np.float64), r[:, il[0], il[1]].astype(np.float64)
        tol = np.where(np.abs(rr) < 1e-30, 1e-33, 1e-3 * np.abs(rr))
        bad = np.abs(gg - rr) > tol
        assert not bad.any(), f"{bad.sum()} scores off, worst rel {np.max(np.abs(gg - rr) / np.maximum(np.abs(rr), 1e-300)):.3e}"


def run_case(rt, w, pool_q, pool_k, theta, seed, gain=1.0):
    import torch
    B, Prefill, ctx = rt
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    nq, nk = bin(pool_q).count("1"), bin(pool_k).count("1")
    wq = (W.make_gate_weights(seed, w.num_q_heads, nq * 128) * np.float32(gain)).astype(np.float32)
    wk = W.make_gate_weights(seed + 1, w.num_kv_heads, nk * 128)
    opt = B.seer_gate_options(pool_q, pool_k, theta)
    p.gate_ex(opt, torch.from_numpy(wq).cuda(), torch.from_numpy(wk).cuda())
    assert p.status() == 0
    ref = O.gate_scores_ex(w.q, w.k, wq, wk, w.cu_seqlens, 64, pool_q=pool_q, pool_k=pool_k, rope_theta=theta)
    check_scores(p.scores_host(), ref, w)
    return p


CASES = [
    # (seqlens, hq, hkv, pool_q, pool_k, theta)
    ([64], 1, 1, 1, 7, 0.0),
    ([200], 4, 2, 1, 7, 500000.0),            # the paper's best pooling + block RoPE, ragged tail
    ([130, 0, 777, 64, 65], 6, 2, 7, 7, 10000.0),
    ([1500, 333], 5, 1, 2, 4, 0.0),           # max on Q, min on K
    ([4099], 8, 4, 3, 6, 500000.0),           # avg+max on Q, max+min on K, 65 blocks
    ([1], 2, 1, 5, 1, 500000.0),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"q{c[3]}k{c[4]}t{int(c[5])}_{sum(c[0])}")
def test_gate_variants_small(rt, case):
    seqlens, hq, hkv, pq, pk, theta = case
    w = W.make_small(seed=300 + pq * 8 + pk, seqlens=seqlens, hq=hq, hkv=hkv)
    run_case(rt, w, pq, pk, theta, seed=7000 + pq * 8 + pk)


def test_gate_variants_defaults_equal_plain_gate(rt):
    """avg on both, no RoPE: the same scores, bit for bit, as seer_gate_scores."""
    import torch
    B, Prefill, ctx = rt
    w = W.make_small(seed=310, seqlens=[777, 130], hq=4, hkv=2)
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.scores.zero_()                                  # entries above the diagonal are never written
    p.gate()
    plain = p.scores_host().copy()
    p.scores.zero_()
    p.gate_ex(B.seer_gate_options(1, 1, 0.0), p.wq, p.wk)
    assert p.status() == 0
    assert np.array_equal(p.scores_host(), plain)


def test_gate_variants_large_logits_with_rope(rt):
    """Large logits (gain on Wq) at a few thousand positions: the rotation angle has to be exact enough for the 1e-3 bound."""
    w = W.make_small(seed=311, seqlens=[64 * 300], hq=2, hkv=1, q_gain=3.0)
    run_case(rt, w, 1, 7, 500000.0, seed=7100, gain=6.0)


def test_gate_variants_reduced_twin(rt):
    """c3's reduced twin (32 / 8 heads) with the paper's best pooling and block RoPE."""
    w = W.make_workload("c3s")
    run_case(rt, w, 1, 7, 500000.0, seed=7200)


def test_gate_variants_rejects_bad_options(rt):
    import torch
    B, Prefill, ctx = rt
    w = W.make_small(seed=312, seqlens=[128], hq=2, hkv=1)
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    for opt in [B.seer_gate_options(0, 1, 0.0), B.seer_gate_options(1, 8, 0.0), B.seer_gate_options(1, 1, -1.0),
                B.seer_gate_options(1, 1, float("nan"))]:
        with pytest.raises(B.SeerError) as e:
            p.gate_ex(opt, p.wq, p.wk)
        assert e.value.status == 1
