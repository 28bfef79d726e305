"""GPU parity of seer_attn_block_max (Sec. 3.2, Eq. 2 on the listed blocks) against the oracle.

The probabilities are those of the block-sparse softmax the lists define; the lse fed to the call is the GPU attention
kernel's own.  Tolerance: |x - ref| <= 1e-2 |ref| + 1e-7 (bf16 operands, fp32 accumulation, lse within its own bound)."""
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


def run(rt, w, params, rows=None):
    B, Prefill, ctx = rt
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx, want_lse=True)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.run(params)
    got = p.block_max().cpu().numpy()
    assert p.status() == 0
    rp = p.row_ptr.cpu().numpy().astype(np.int64)
    col = p.col_idx.cpu().numpy()[: rp[-1]]
    ref = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, w.num_q_heads, w.num_kv_heads, 64,
                                  1.0 / np.sqrt(128.0), rows=rows)
    sel = ~np.isnan(ref)
    assert sel.any()
    g, r = got[: rp[-1]][sel].astype(np.float64), ref[sel]
    assert np.all(np.abs(g - r) <= 1e-2 * np.abs(r) + 1e-7), f"worst rel {np.max(np.abs(g - r) / np.maximum(r, 1e-30)):.3e}"
    return p


@pytest.mark.parametrize("cfg", [dict(seed=400, seqlens=[64], hq=1, hkv=1), dict(seed=401, seqlens=[200], hq=4, hkv=2),
                                 dict(seed=402, seqlens=[130, 0, 777, 64, 65], hq=6, hkv=2),
                                 dict(seed=403, seqlens=[1500, 333], hq=5, hkv=1)], ids=lambda c: f"s{c['seed']}")
@pytest.mark.parametrize("keep", [(1, 1), (1, 3)], ids=["dense", "third"])
def test_block_max_small(rt, cfg, keep):
    B, Prefill, ctx = rt
    w = W.make_small(**cfg)
    run(rt, w, B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=keep[0], keep_den=keep[1], flags=3))


def test_block_max_dense_lists_are_the_eq2_map(rt):
    """Full causal lists: the values are the max-pooled dense causal attention map of Eq. 2."""
    B, Prefill, ctx = rt
    w = W.make_small(seed=404, seqlens=[300], hq=2, hkv=1)
    p = run(rt, w, B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=1, flags=1))
    gt = O.maxpool_attention_map(w.q, w.k, w.cu_seqlens, 2, 1, 64, 1.0 / np.sqrt(128.0))[0]
    rp = p.row_ptr.cpu().numpy(); col = p.col_idx.cpu().numpy(); got = p.bmax.cpu().numpy()
    nb = 5
    for h in range(2):
        for i in range(nb):
            r = h * nb + i
            for q_ in range(rp[r], rp[r + 1]):
                ref = gt[h, i, col[q_]]
                assert abs(got[q_] - ref) <= 1e-2 * ref + 1e-7


def test_block_max_reduced_twin_sampled_rows(rt):
    B, Prefill, ctx = rt
    w = W.make_workload("c3s")
    p0 = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    rows = list(range(0, int(p0.rows), 97))[:200]
    run(rt, w, B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=10, flags=3), rows=rows)
