"""Seeded random shapes through the whole GPU path (gate -> mask -> attention -> max-pooled map), each checked against
the oracle: gate scores within 1e-3 relative, lists bit-exact (oracle mask on the GPU's own scores), attention within
the stated tolerance with the GPU's lists fed to both, the max-pooled map within 1e-2 relative.

Shapes: 1-4 packed sequences of 0-700 tokens (ragged tails, empty sequences, single tokens), 1-3 KV heads, group sizes
1, 2, 4, 5, every mask mode with random parameters and flags."""
import math

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


def draw_case(seed):
    rng = np.random.default_rng(900_000 + seed)
    nseq = int(rng.integers(1, 5))
    lens = [int(x) for x in rng.choice([0, 1, 63, 64, 65, 127, 128, 200, 333, 512, 700], size=nseq)]
    if sum(lens) == 0:
        lens[0] = 64
    hkv = int(rng.integers(1, 4))
    group = int(rng.choice([1, 2, 4, 5]))
    mode = int(rng.integers(0, 3))
    flags = int(rng.choice([1, 3]))
    kw = dict(mode=mode, flags=flags)
    if mode == O.MODE_TOPK_RATIO:
        kw.update(keep_num=int(rng.integers(1, 4)), keep_den=int(rng.integers(3, 9)))
    elif mode == O.MODE_TOPK_COUNT:
        kw.update(k=int(rng.integers(0, 6)))
    else:
        kw.update(threshold=float(rng.choice([0.0, 0.05, 0.2, 0.5, 1.0])))
    gain = float(rng.choice([1.0, 3.0]))
    return lens, hkv * group, hkv, kw, gain


@pytest.mark.parametrize("seed", range(48))
def test_random_shape_whole_path(rt, seed):
    B, Prefill, ctx = rt
    lens, hq, hkv, kw, gain = draw_case(seed)
    w = W.make_small(seed=910_000 + seed, seqlens=lens, hq=hq, hkv=hkv, q_gain=gain)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                                k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw["flags"])
    p.o.fill_(float("nan"))
    p.run(params)
    bmax = p.block_max().cpu().numpy()
    assert p.status() == 0, (lens, hq, hkv, kw)
    # gate
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 64, hq)
    ref = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 64)
    for g, r in zip(got, ref):
        il = np.tril_indices(r.shape[-1])
        gg, rr = g[:, il[0], il[1]].astype(np.float64), r[:, il[0], il[1]].astype(np.float64)
        assert np.all(np.abs(gg - rr) <= np.where(rr < 1e-30, 1e-33, 1e-3 * rr)), (lens, hq, hkv)
    # lists: the oracle's mask on the GPU's scores, bit-exact
    rp, col = p.lists_host()
    orp, ocol = O.block_mask(got, kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                             k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw["flags"])
    assert np.array_equal(rp, orp) and np.array_equal(col, ocol), (lens, hq, hkv, kw)
    # attention and the max-pooled map with the GPU's lists
    o_ref, lse_ref = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp, col, hq, hkv, 64, 1 / math.sqrt(128))
    x, r = p.o_host().astype(np.float64), o_ref
    err = np.abs(x - r)
    assert np.all(err <= 2e-2 + 1e-2 * np.abs(r)), (lens, hq, hkv, kw, float(err.max()))
    rms = np.sqrt((err ** 2).sum(-1)) / np.maximum(np.sqrt((r ** 2).sum(-1)), 1e-30)
    assert rms.max() <= 1e-2
    lg, lr = p.lse_host().astype(np.float64), lse_ref
    fin = np.isfinite(lr)
    assert np.all(np.abs(lg[fin] - lr[fin]) <= 2e-3 + 1e-3 * np.abs(lr[fin])) and np.all(lg[~fin] == lr[~fin])
    bref = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, hq, hkv, 64, 1 / math.sqrt(128))
    assert np.all(np.abs(bmax[: len(col)] - bref) <= 1e-2 * bref + 1e-7), (lens, hq, hkv, kw)
