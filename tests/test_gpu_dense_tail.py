"""seer_mask_params.dense_tail_blocks ("sparsity in the context, dense on the question", Sec. 4): the last query blocks
of every sequence keep all their causal blocks.  Lists bit-exact against the oracle's mask builder on the GPU's scores,
through the separate calls, the one-call gate + mask, 128-token blocks and a chunk."""
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


@pytest.mark.parametrize("mode,kw", [(O.MODE_TOPK_RATIO, dict(keep_num=1, keep_den=5)), (O.MODE_TOPK_COUNT, dict(k=2)),
                                     (O.MODE_THRESHOLD, dict(threshold=0.05))])
@pytest.mark.parametrize("blk", [64, 128])
@pytest.mark.parametrize("tail", [0, 1, 3, 1000])
def test_dense_tail_lists(rt, mode, kw, blk, tail):
    B, Prefill, ctx = rt
    lens, hq, hkv = [1500, 64, 0, 2100, 130], 4, 2
    w = W.make_small(seed=66_000 + blk, seqlens=lens, hq=hq, hkv=hkv, q_gain=2.0, block=blk)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False, block=blk)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(mode, keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1), k=kw.get("k", 0),
                                threshold=kw.get("threshold", 0.0), flags=3, dense_tail=tail)
    p.gate(); p.mask(params)
    assert p.status() == 0
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, blk, hq)
    orp, ocol = O.block_mask(got, mode, flags=3, dense_tail=tail, **kw)
    rp, col = p.lists_host()
    assert np.array_equal(rp, orp) and np.array_equal(col, ocol)
    p.row_ptr.fill_(-1)
    p.gate_mask(params, band_bytes=0)
    rp2, col2 = p.lists_host()
    assert np.array_equal(rp2, orp) and np.array_equal(col2, ocol)
    if tail == 1000:                                      # everything dense: the full causal lists, in closed form
        frp, fcol = O.full_causal_lists(w.cu_seqlens, blk, hq)
        assert np.array_equal(rp, frp) and np.array_equal(col, fcol)


def test_dense_tail_with_a_chunk_and_validation(rt):
    B, Prefill, ctx = rt
    lens, starts, hq, hkv = [1000, 700], [640, 0], 2, 1
    w = W.make_small(seed=66_500, seqlens=lens, hq=hq, hkv=hkv)
    cu_q = np.array([0, 360, 360 + 700], dtype=np.int32)
    qc = np.concatenate([w.q[640:1000], w.q[1000:1700]], axis=0)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False, cu_seqlens_q=cu_q)
    p.set_inputs(qc, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(B.SEER_TOPK_COUNT, k=2, flags=1, dense_tail=2)
    p.scores.fill_(float("nan"))
    p.gate(); p.mask(params)
    assert p.status() == 0
    offs = O.chunk_offsets(cu_q, w.cu_seqlens, 64)
    s = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 64, hq)
    rows = [s[b][:, int(offs[b]):, :] for b in range(2)]
    orp, ocol = O.block_mask_chunk(rows, O.MODE_TOPK_COUNT, k=2, flags=1, dense_tail=2)
    rp, col = p.lists_host()
    assert np.array_equal(rp, orp) and np.array_equal(col, ocol)
    bad = B.make_mask_params(B.SEER_TOPK_COUNT, k=2, flags=1, dense_tail=-1)
    with pytest.raises(B.SeerError) as e:
        p.mask(bad)
    assert e.value.status == 1
