"""GPU parity with 128-token gate blocks (shape.block = 128): gate scores and lists against the oracle at B = 128, the
expanded 64-token lists against the rule written with python sets (bit-exact), and the attention that runs on them
against the oracle's attention at B = 128 on the 128-token lists."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W
from test_oracle_block128 import expand_reference

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


CASES = [
    # (seqlens, hq, hkv, mask kwargs)
    ([128], 1, 1, dict(mode=O.MODE_TOPK_RATIO, keep_num=1, keep_den=2, flags=3)),
    ([130, 0, 777, 64, 65, 1], 6, 2, dict(mode=O.MODE_TOPK_RATIO, keep_num=1, keep_den=3, flags=3)),
    ([4099], 8, 4, dict(mode=O.MODE_THRESHOLD, threshold=0.03, flags=1)),
    ([1500, 333, 2048], 4, 1, dict(mode=O.MODE_TOPK_COUNT, k=4, flags=3)),
    ([9000], 2, 2, dict(mode=O.MODE_THRESHOLD, threshold=0.02, flags=0)),      # rows may lose their diagonal block
]


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_block128_whole_path(rt, ci):
    B, Prefill, ctx = rt
    lens, hq, hkv, kw = CASES[ci]
    w = W.make_small(seed=88_000 + ci, seqlens=lens, hq=hq, hkv=hkv, q_gain=2.0, block=128)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True, block=128)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                                k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw["flags"])
    p.o.fill_(float("nan"))
    p.run(params)
    assert p.status() == 0
    # gate at B = 128
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 128, hq)
    ref = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 128)
    for g, r in zip(got, ref):
        il = np.tril_indices(r.shape[-1])
        gg, rr = g[:, il[0], il[1]].astype(np.float64), r[:, il[0], il[1]].astype(np.float64)
        assert np.all(np.abs(gg - rr) <= np.where(rr < 1e-30, 1e-33, 1e-3 * rr))
    # lists at B = 128: the oracle's mask on the GPU's scores
    rp, col = p.lists_host()
    orp, ocol = O.block_mask(got, kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                             k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw["flags"])
    assert np.array_equal(rp, orp) and np.array_equal(col, ocol)
    # expanded lists: bit-exact against the rule
    rp64, col64 = p.lists64_host()
    erp, ecol = expand_reference(w.cu_seqlens, hq, rp, col)
    assert np.array_equal(rp64, erp) and np.array_equal(col64, ecol)
    assert int(p.nnz64.item()) == len(ecol)
    # attention against the oracle at B = 128 on the 128-token lists
    o_ref, lse_ref = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp, col, hq, hkv, 128, 1 / math.sqrt(128))
    x = p.o_host().astype(np.float64)
    empty = np.isneginf(lse_ref.T)                       # tokens whose row lists nothing visible (no diagonal block)
    err = np.abs(x - o_ref)
    assert np.all(err[~empty] <= 2e-2 + 1e-2 * np.abs(o_ref[~empty]))
    lg = p.lse_host().T.astype(np.float64)
    assert np.all(np.abs(lg[~empty] - lse_ref.T[~empty]) <= 2e-3 + 1e-3 * np.abs(lse_ref.T[~empty]))
    assert np.all(x[empty] == 0) and np.all(np.isneginf(lg[empty]))
    # gate + mask in one call gives the same lists
    p.row_ptr.fill_(-1); p.row_ptr64.fill_(-1)
    p.gate_mask(params, band_bytes=0)
    rp2, col2 = p.lists_host()
    rp642, col642 = p.lists64_host()
    assert np.array_equal(rp2, rp) and np.array_equal(col2, col) and np.array_equal(rp642, rp64) and np.array_equal(col642, col64)


def test_block128_rope_uses_theta_over_128(rt):
    import torch
    B, Prefill, ctx = rt
    lens, hq, hkv = [3000, 130], 4, 2
    w = W.make_small(seed=88_100, seqlens=lens, hq=hq, hkv=hkv, block=128)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False, block=128)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    wq = W.make_gate_weights(15, hq, 128)
    wk = W.make_gate_weights(16, hkv, 3 * 128)
    opt = B.seer_gate_options(1, 7, 500000.0)
    p.gate_ex(opt, torch.from_numpy(wq).cuda(), torch.from_numpy(wk).cuda())
    assert p.status() == 0
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 128, hq)
    ref = O.gate_scores_ex(w.q, w.k, wq, wk, w.cu_seqlens, 128, pool_q=1, pool_k=7, rope_theta=500000.0)
    for g, r in zip(got, ref):
        il = np.tril_indices(r.shape[-1])
        gg, rr = g[:, il[0], il[1]].astype(np.float64), r[:, il[0], il[1]].astype(np.float64)
        assert np.all(np.abs(gg - rr) <= np.where(rr < 1e-30, 1e-33, 1e-3 * rr))


def test_block128_unsupported_calls_and_capacity(rt):
    import torch
    B, Prefill, ctx = rt
    w = W.make_small(seed=88_200, seqlens=[1000], hq=2, hkv=1, block=128)
    p = Prefill(w.cu_seqlens, 2, 1, ctx=ctx, want_lse=True, block=128)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=1, flags=1)
    p.gate(); p.mask(params)
    with pytest.raises(B.SeerError) as e:
        B.seer_sparse_attn(ctx, p.shape, p.q, p.k, p.v, p.row_ptr, p.col_idx, p.o, p.lse)
    assert e.value.status == 2                             # SEER_ERR_UNSUPPORTED
    with pytest.raises(B.SeerError) as e:
        B.seer_expand_block_lists(ctx, p.attn_shape, p.row_ptr, p.col_idx, p.row_ptr64, p.col_idx64)
    assert e.value.status == 2                             # a 64-token shape has nothing to expand
    # dense causal lists: 8 blocks of 128 -> 36 entries; 16 rows of 64 -> 136 entries
    assert int(p.nnz.item()) == 2 * 36 and int(p.nnz64.item()) == 2 * 136
    small = torch.empty(100, dtype=torch.int32, device="cuda")
    B.seer_expand_block_lists(ctx, p.shape, p.row_ptr, p.col_idx, p.row_ptr64, small, 100, p.nnz64)
    assert p.status() == 4                                 # SEER_ERR_CAPACITY
    assert int(p.nnz64.item()) == 2 * 136
