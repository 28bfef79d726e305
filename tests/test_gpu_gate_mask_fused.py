"""seer_gate_block_mask (gate and mask in one call, scores held one band at a time) against the two separate calls and
the oracle.

The banded call runs the same kernels on the same projected vectors, so its lists must equal those of
seer_gate_scores / seer_gate_scores_ex + seer_block_mask bit for bit, whatever the band size: bands of whole sequences,
of whole heads and of 64-row tile runs are all forced here by the scratch size.  The lists are also compared with the
oracle's mask builder applied to the scores the GPU gate produced (bit-exact)."""
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


def mask_params(B, kw):
    return B.make_mask_params(kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1), k=kw.get("k", 0),
                              threshold=kw.get("threshold", 0.0), flags=kw.get("flags", 3))


def band_sizes(lens, hq):
    """Scratch sizes that force each kind of band for the longest sequence: tile runs, single heads, two heads, all."""
    nb = max((n + 63) // 64 for n in lens)
    return [0, 3 * 64 * nb * 4 + 16, nb * nb * 4 + 16, 2 * nb * nb * 4 + 64, hq * nb * nb * 4 + 16, 1 << 26]


SHAPES = [
    # (seqlens, hq, hkv)
    ([64], 1, 1),
    ([4099], 8, 4),                              # 65 blocks: two 64-row tiles per head, ragged tail
    ([130, 0, 777, 64, 65], 6, 2),               # packed, an empty sequence, odd block counts (unaligned score offsets)
    ([9000, 333, 2048], 4, 1),                   # 141 blocks: three tiles per head
    ([1], 2, 1),
    ([100] * 37, 3, 3),                          # many short sequences: whole-sequence bands gather several
]
MODES = [
    dict(mode=O.MODE_TOPK_RATIO, keep_num=1, keep_den=4, flags=3),
    dict(mode=O.MODE_TOPK_COUNT, k=3, flags=1),
    dict(mode=O.MODE_THRESHOLD, threshold=0.02, flags=3),
]


@pytest.mark.parametrize("si", range(len(SHAPES)))
@pytest.mark.parametrize("mi", range(len(MODES)))
def test_fused_equals_separate_calls(rt, si, mi):
    B, Prefill, ctx = rt
    lens, hq, hkv = SHAPES[si]
    kw = MODES[mi]
    w = W.make_small(seed=77_000 + 10 * si + mi, seqlens=lens, hq=hq, hkv=hkv, q_gain=3.0)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = mask_params(B, kw)
    p.gate()
    p.mask(params)
    assert p.status() == 0
    rp0, col0 = p.lists_host()
    nnz0 = int(p.nnz.item())
    # the oracle's mask on the GPU's scores
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 64, hq)
    orp, ocol = O.block_mask(got, kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                             k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw.get("flags", 3))
    assert np.array_equal(rp0, orp) and np.array_equal(col0, ocol)
    for band in band_sizes(lens, hq):
        p.row_ptr.fill_(-7)
        p.col_idx.fill_(-7)
        p.nnz.fill_(-7)
        p.scores.fill_(float("nan"))           # the fused call must not depend on the score matrix
        p.gate_mask(params, band_bytes=band)
        assert p.status() == 0, (lens, band)
        rp1, col1 = p.lists_host()
        assert np.array_equal(rp1, rp0), (lens, hq, hkv, kw, band)
        assert np.array_equal(col1, col0), (lens, hq, hkv, kw, band)
        assert int(p.nnz.item()) == nnz0


def test_fused_with_gate_options(rt):
    """Composed pooling and block RoPE go through the same banded path."""
    import torch
    B, Prefill, ctx = rt
    lens, hq, hkv = [3000, 200], 4, 2
    w = W.make_small(seed=78_001, seqlens=lens, hq=hq, hkv=hkv)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    wq = torch.from_numpy(W.make_gate_weights(5, hq, 128)).cuda()
    wk = torch.from_numpy(W.make_gate_weights(6, hkv, 3 * 128)).cuda()
    opt = B.seer_gate_options(1, 7, 500000.0)
    params = mask_params(B, MODES[0])
    p.gate_ex(opt, wq, wk)
    p.mask(params)
    rp0, col0 = p.lists_host()
    for band in band_sizes(lens, hq):
        p.row_ptr.fill_(0)
        p.col_idx.fill_(-1)
        p.gate_mask(params, band_bytes=band, options=opt, wq=wq, wk=wk)
        assert p.status() == 0
        rp1, col1 = p.lists_host()
        assert np.array_equal(rp1, rp0) and np.array_equal(col1, col0), band


def test_fused_capacity_and_workspace_errors(rt):
    import torch
    B, Prefill, ctx = rt
    lens, hq, hkv = [2000], 2, 1
    w = W.make_small(seed=78_002, seqlens=lens, hq=hq, hkv=hkv)
    params = mask_params(B, dict(mode=O.MODE_THRESHOLD, threshold=0.0, flags=3))
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.gate_mask(params, band_bytes=0)
    assert p.status() == 0
    nnz = int(p.nnz.item())
    small = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False, col_capacity=nnz - 1)
    small.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    small.gate_mask(params, band_bytes=0)      # several bands: the overflow is seen in a later band
    assert small.status() == 4                     # SEER_ERR_CAPACITY
    assert int(small.nnz.item()) == nnz          # the count is still the true one
    # a workspace that holds the projected vectors but not 64 rows of scores
    need = B.seer_gate_mask_workspace_bytes(p.shape, 0)
    assert need > B.seer_workspace_bytes(p.shape)
    ws = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SeerError) as e:
        B.seer_gate_block_mask(ctx, p.shape, None, p.q, p.k, p.wq, p.wk, params, p.row_ptr, p.col_idx, p.col_capacity,
                               p.nnz, ws)
    assert e.value.status == 3                    # SEER_ERR_WORKSPACE


def test_fused_empty_batch(rt):
    B, Prefill, ctx = rt
    p = Prefill([0, 0, 0], 2, 1, ctx=ctx, want_lse=False)
    params = mask_params(B, MODES[0])
    p.row_ptr.fill_(5)
    p.gate_mask(params, band_bytes=0)
    assert p.status() == 0
    assert int(p.row_ptr[0].item()) == 0 and int(p.nnz.item()) == 0
