"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times (whole GPU path, default
attention kernel).  The oracle cannot run attention in full at these sizes, so it checks (a) the gate scores of every
head, one head at a time, (b) the block lists of every head, rebuilt from the GPU's own scores (bit-exact), (c) attention
on a stratified sample of rows of every (sequence, head) (the first two query blocks, the last, the longest and the
shortest list, eight seeded-random ones) with the GPU's lists fed to both, (d) properties that hold at any size (list
lengths in closed form, ordering, range), and (e) every output row against the independent mma.sync kernel."""
import json
import math
import os

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "thresholds.json")


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


def golden_threshold(name):
    with open(GOLDEN) as f:
        return float.fromhex(json.load(f)[name]["threshold_hex"])


def check_workload(rt, name, specs, sample_heads=None, rows_per_head=8, all_rows=False):
    B, Prefill, ctx = rt
    w = W.make_workload(name)
    G = w.num_q_heads // w.num_kv_heads
    if sample_heads is None:
        sample_heads = list(range(w.num_q_heads))
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.gate()
    gpu_scores = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 64, w.num_q_heads)   # per sequence [Hq, nb, nb] views
    # (a) gate scores, head by head, against the oracle run on that head alone
    for h in sample_heads:
        g = h // G
        ref = O.gate_scores(np.ascontiguousarray(w.q[:, h:h + 1]), np.ascontiguousarray(w.k[:, g:g + 1]),
                            w.wq[h:h + 1], w.wk[g:g + 1], w.cu_seqlens, 64)
        got = [s[h:h + 1] for s in gpu_scores]
        for r, x in zip(ref, got):
            il = np.tril_indices(r.shape[-1])
            rr, xx = r[:, il[0], il[1]].astype(np.float64), x[:, il[0], il[1]].astype(np.float64)
            assert np.all(np.abs(xx - rr) <= np.where(rr < 1e-30, 1e-33, 1e-3 * rr)), (name, h)
    nbs = [int(n) for n in w.num_blocks]
    for spec in specs:
        params = B.make_mask_params(spec.mode, keep_num=spec.keep_num, keep_den=spec.keep_den, k=spec.k,
                                    threshold=spec.threshold or 0.0, flags=spec.flags)
        p.mask(params)
        p.o.fill_(float("nan"))
        p.attn()
        assert p.status() == 0
        rp, col = p.lists_host()
        # the banded gate + mask call (no score matrix) gives the same lists, bit for bit
        p.row_ptr.fill_(-1)
        p.gate_mask(params)
        assert p.status() == 0
        rp_f, col_f = p.lists_host()
        assert np.array_equal(rp_f, rp) and np.array_equal(col_f, col), name
        p.ws_fused = None
        # (d) properties at any size
        counts = np.diff(rp)
        assert rp[0] == 0 and rp[-1] == len(col) == int(p.nnz.item())
        base = 0
        for nb in nbs:
            i_of_row = np.tile(np.arange(nb), w.num_q_heads)
            c = counts[base:base + w.num_q_heads * nb]
            if spec.mode == W.MODE_TOPK_RATIO:
                nf = np.where(i_of_row == 0, 1, bin(spec.flags & 3).count("1"))
                ki = np.clip(-((-spec.keep_num * (i_of_row + 1)) // spec.keep_den), 1, i_of_row + 1)
                assert np.array_equal(c, np.maximum(ki, nf))
            assert np.all(c >= 1) and np.all(c <= i_of_row + 1)
            base += w.num_q_heads * nb
        row_of = np.repeat(np.arange(len(counts)), counts)
        same_row = row_of[1:] == row_of[:-1]
        assert np.all(col[1:][same_row] > col[:-1][same_row])            # ascending, unique
        assert np.all(col >= 0)
        # (b) lists of the sampled heads, rebuilt by the oracle from the GPU's scores: bit-exact
        base = 0
        for b, nb in enumerate(nbs):
            for h in sample_heads:
                s = gpu_scores[b][h:h + 1]
                orp, ocol = O.block_mask([s], spec.mode, keep_num=spec.keep_num, keep_den=spec.keep_den, k=spec.k,
                                         threshold=spec.threshold or 0.0, flags=spec.flags)
                r0 = base + h * nb
                assert np.array_equal(np.diff(rp[r0:r0 + nb + 1]), np.diff(orp)), (name, h)
                assert np.array_equal(col[rp[r0]:rp[r0 + nb]], ocol), (name, h)
            base += w.num_q_heads * nb
        # (c) attention on a stratified sample of rows with the GPU's lists
        rows = None if all_rows else W.sample_rows(w.cu_seqlens, w.num_q_heads, rp, seed=11,
                                                   per_head_random=rows_per_head, heads=sample_heads)
        o_ref, lse_ref = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp, col, w.num_q_heads, w.num_kv_heads, 64,
                                            1 / math.sqrt(128), rows=rows)
        done = ~np.isnan(o_ref[..., 0])
        assert done.sum() > 0
        x, r = p.o_host()[done].astype(np.float64), o_ref[done]
        err = np.abs(x - r)
        assert np.all(err <= 2e-2 + 1e-2 * np.abs(r)), (name, err.max())
        rms = np.sqrt((err ** 2).sum(-1)) / np.maximum(np.sqrt((r ** 2).sum(-1)), 1e-30)
        assert rms.max() <= 1e-2, (name, rms.max())
        lg, lr = p.lse_host().T[done].astype(np.float64), lse_ref.T[done]
        assert np.all(np.abs(lg - lr) <= 2e-3 + 1e-3 * np.abs(lr))
        assert not np.isnan(p.o_host()).any()                            # every row was written


def test_c3_128k_topk_bench_configuration(rt):
    specs = [W.MaskSpec(W.MODE_TOPK_RATIO, 1, 10, flags=W.FORCE_DIAG | W.FORCE_SINK),
             W.MaskSpec(W.MODE_TOPK_RATIO, 1, 2, flags=W.FORCE_DIAG | W.FORCE_SINK)]
    check_workload(rt, "c3", specs)


def test_c1_full_size_every_row(rt):
    """The smallest workload: the oracle runs the whole of it (every head, every attention row)."""
    check_workload(rt, "c1", [W.make_workload("c1").masks[0]], all_rows=True)


@pytest.mark.parametrize("name", ["c2", "c4", "c5"])
def test_threshold_workloads_full_size(rt, name):
    w_spec = W.make_workload(name + "s").masks[0]            # same mask recipe as the full-size workload
    spec = W.MaskSpec(W.MODE_THRESHOLD, threshold=golden_threshold(name), flags=w_spec.flags)
    check_workload(rt, name, [spec])


def full_size_params(B, name):
    if name == "c3":
        return B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=10, flags=3)
    w_spec = W.make_workload(name + "s").masks[0]
    return B.make_mask_params(B.SEER_THRESHOLD, threshold=golden_threshold(name), flags=w_spec.flags)


@pytest.mark.parametrize("name", ["c3", "c2", "c4", "c5"])
def test_full_size_all_rows_cross_check(rt, name):
    """Every output row of the full-size workloads, not a sample: the tcgen05 kernel against the independent mma.sync
    kernel (different tiling, layout and softmax scheme; itself checked against the oracle on the small cases) on the
    same lists.  Both round P and o to bf16, so the bound is the attention tolerance between two results of that kind."""
    import torch
    B, Prefill, ctx = rt
    w = W.make_workload(name)
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    B.seer_set_attn_impl(ctx, 0)
    p.run(full_size_params(B, name))
    assert p.status() == 0
    o_tc = p.o.float().clone()
    lse_tc = p.lse.clone()
    B.seer_set_attn_impl(ctx, 1)
    try:
        p.o.fill_(float("nan"))
        p.attn()
        assert p.status() == 0
    finally:
        B.seer_set_attn_impl(ctx, 0)
    o_mma = p.o.float()
    assert not torch.isnan(o_mma).any() and not torch.isnan(o_tc).any()
    err = (o_tc - o_mma).abs()
    assert bool((err <= 2e-2 + 1e-2 * o_mma.abs()).all()), float(err.max())
    rms = err.pow(2).sum(-1).sqrt() / o_mma.pow(2).sum(-1).sqrt().clamp_min(1e-30)
    assert float(rms.max()) <= 2e-2, float(rms.max())
    assert bool(((lse_tc - p.lse).abs() <= 2e-3 + 1e-3 * p.lse.abs()).all())
