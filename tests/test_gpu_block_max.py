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


IMPLS = [0, 1]   # 0: the tcgen05 pipeline without V, 1: the mma.sync kernel


def run(rt, w, params, rows=None, impl=0):
    B, Prefill, ctx = rt
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx, want_lse=True)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.run(params)
    B.seer_set_attn_impl(ctx, impl)
    try:
        got = p.block_max().cpu().numpy()
    finally:
        B.seer_set_attn_impl(ctx, 0)
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
@pytest.mark.parametrize("impl", IMPLS)
def test_block_max_small(rt, cfg, keep, impl):
    B, Prefill, ctx = rt
    w = W.make_small(**cfg)
    run(rt, w, B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=keep[0], keep_den=keep[1], flags=3), impl=impl)


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


@pytest.mark.parametrize("impl", IMPLS)
def test_block_max_reduced_twin_sampled_rows(rt, impl):
    B, Prefill, ctx = rt
    w = W.make_workload("c3s")
    p0 = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    rows = list(range(0, int(p0.rows), 97))[:200]
    run(rt, w, B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=10, flags=3), rows=rows, impl=impl)


def hand_lists(rt, w, rp, col, impl):
    """Attention and block maxima on lists given by hand; returns (values, status, oracle values)."""
    B, Prefill, ctx = rt
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx, want_lse=True)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.set_lists(rp, col)
    p.status()                                           # (reads and clears the device status)
    B.seer_set_attn_impl(ctx, impl)
    try:
        p.attn()
        st_attn = p.status()
        got = p.block_max().cpu().numpy()[: len(col)]
        st = p.status()
    finally:
        B.seer_set_attn_impl(ctx, 0)
    return got, st_attn, st


@pytest.mark.parametrize("impl", IMPLS)
def test_block_max_unsorted_odd_and_empty_lists(rt, impl):
    w = W.make_small(410, [256 + 37], 2, 1)             # five blocks, the last one ragged
    # head 0: rows with lists [], [1, 0], [2], [3, 0, 1], [4, 2, 0]; head 1: [0], [], [0, 1, 2], [], [4]
    rp = np.array([0, 0, 2, 3, 6, 9, 10, 10, 13, 13, 14], np.int64)
    col = np.array([1, 0, 2, 3, 0, 1, 4, 2, 0, 0, 0, 1, 2, 4], np.int32)
    got, st_attn, st = hand_lists(rt, w, rp, col, impl)
    assert st_attn == 0 and st == 0
    ref = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, 2, 1, 64, 1.0 / np.sqrt(128.0))
    assert np.all(np.abs(got - ref) <= 1e-2 * np.abs(ref) + 1e-7)


@pytest.mark.parametrize("impl", IMPLS)
def test_block_max_flags_out_of_range_entries_and_reports_zero(rt, impl):
    w = W.make_small(411, [192], 1, 1)
    rp = np.array([0, 1, 3, 5], np.int64)
    col = np.array([0, 0, 5, -3, 2], np.int32)          # row 1 lists block 5 (> i), row 2 lists block -3
    got, st_attn, st = hand_lists(rt, w, rp, col, impl)
    assert st_attn == 5 and st == 5                     # SEER_ERR_INVALID_INDEX from both calls
    good_rp = np.array([0, 1, 2, 3], np.int64)
    good_col = np.array([0, 0, 2], np.int32)
    ref = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, good_rp, good_col, 1, 1, 64, 1.0 / np.sqrt(128.0))
    assert got[2] == 0.0 and got[3] == 0.0
    assert np.all(np.abs(got[[0, 1, 4]] - ref) <= 1e-2 * np.abs(ref) + 1e-7)
