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


@pytest.mark.parametrize("seed", range(40))
def test_random_shape_all_features(rt, seed):
    """Seeded random combinations of everything the library offers on one problem: block 64 or 128, composed pooling
    and block RoPE in the gate, every mask mode with random flags and a dense tail, the one-call gate + mask with a random
    band size, the list expansion for 128-token blocks, attention and (at block 64) the max-pooled map; each against
    the oracle as in the tests of the single features."""
    import torch
    from test_oracle_block128 import expand_reference
    B, Prefill, ctx = rt
    rng = np.random.default_rng(777_000 + seed)
    blk = int(rng.choice([64, 128]))
    nseq = int(rng.integers(1, 4))
    lens = [int(x) for x in rng.choice([1, 63, 64, 65, 127, 128, 129, 200, 333, 512, 700, 1000], size=nseq)]
    hkv = int(rng.integers(1, 3))
    hq = hkv * int(rng.choice([1, 2, 4, 5]))
    mode = int(rng.integers(0, 3))
    kw = dict(keep_num=int(rng.integers(1, 3)), keep_den=int(rng.integers(2, 7)), k=int(rng.integers(0, 6)),
              threshold=float(rng.choice([0.0, 0.02, 0.1, 0.5])), flags=int(rng.choice([0, 1, 2, 3])))
    tail = int(rng.choice([0, 0, 1, 2]))
    pq, pk = int(rng.choice([1, 3, 7])), int(rng.choice([1, 6, 7]))
    theta = float(rng.choice([0.0, 10000.0, 500000.0]))
    w = W.make_small(seed=778_000 + seed, seqlens=lens, hq=hq, hkv=hkv, q_gain=float(rng.choice([1.0, 3.0])), block=blk)
    wq = W.make_gate_weights(seed, hq, bin(pq).count("1") * 128)
    wk = W.make_gate_weights(seed + 1, hkv, bin(pk).count("1") * 128)
    wq_d, wk_d = torch.from_numpy(wq).cuda(), torch.from_numpy(wk).cuda()
    opt = B.seer_gate_options(pq, pk, theta)
    params = B.make_mask_params(mode, dense_tail=tail, **kw)
    what = (blk, lens, hq, hkv, mode, kw, tail, pq, pk, theta)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True, block=blk)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.o.fill_(float("nan"))
    try:
        p.gate_ex(opt, wq_d, wk_d); p.mask(params); p.attn()
    finally:
        B.seer_set_attn_impl(ctx, 0)
    assert p.status() == 0, what
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, blk, hq)
    ref = O.gate_scores_ex(w.q, w.k, wq, wk, w.cu_seqlens, blk, pool_q=pq, pool_k=pk, rope_theta=theta)
    for g, r in zip(got, ref):
        il = np.tril_indices(r.shape[-1])
        gg, rr = g[:, il[0], il[1]].astype(np.float64), r[:, il[0], il[1]].astype(np.float64)
        assert np.all(np.abs(gg - rr) <= np.where(rr < 1e-30, 1e-33, 1e-3 * rr)), what
    rp, col = p.lists_host()
    orp, ocol = O.block_mask(got, mode, dense_tail=tail, **kw)
    assert np.array_equal(rp, orp) and np.array_equal(col, ocol), what
    if blk == 128:
        rp64, col64 = p.lists64_host()
        erp, ecol = expand_reference(w.cu_seqlens, hq, rp, col)
        assert np.array_equal(rp64, erp) and np.array_equal(col64, ecol), what
    o_ref, lse_ref = O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp, col, hq, hkv, blk, 1 / math.sqrt(128))
    x = p.o_host().astype(np.float64)
    assert np.all(np.abs(x - o_ref) <= 2e-2 + 1e-2 * np.abs(o_ref)), what
    lg, fin = p.lse_host().astype(np.float64), np.isfinite(lse_ref)
    assert np.all(np.abs(lg[fin] - lse_ref[fin]) <= 2e-3 + 1e-3 * np.abs(lse_ref[fin])) and np.all(np.isneginf(lg[~fin])), what
    p.row_ptr.fill_(-1)
    p.gate_mask(params, band_bytes=int(rng.choice([0, 20000, 1 << 20])), options=opt, wq=wq_d, wk=wk_d)
    rp2, col2 = p.lists_host()
    assert p.status() == 0 and np.array_equal(rp2, rp) and np.array_equal(col2, col), what
    if blk == 64:
        bm = p.block_max().cpu().numpy()[:len(col)]
        bref = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, hq, hkv, 64, 1 / math.sqrt(128))
        assert np.all(np.abs(bm - bref) <= 1e-2 * np.abs(bref) + 1e-30), what


@pytest.mark.parametrize("seed", range(24))
def test_random_lists_on_data_that_moves_the_softmax_references(rt, seed):
    """Random lists (odd lengths, rows without their diagonal block, empty rows) on inputs built to exceed the running
    softmax references again and again: key norms that grow along the sequence, a few huge outlier keys, queries of very
    different scales, strongly negative logits followed by a late positive block.  Both attention kernels against
    the oracle."""
    B, Prefill, ctx = rt
    rng = np.random.default_rng(555_000 + seed)
    lens = [int(rng.integers(300, 2500)) for _ in range(int(rng.integers(1, 3)))]
    hq = int(rng.choice([1, 2]))
    w = W.make_small(seed=556_000 + seed, seqlens=lens, hq=hq, hkv=1)
    T = int(w.cu_seqlens[-1])
    kf, qf = W.bf16_bits_to_f32(w.k).copy(), W.bf16_bits_to_f32(w.q).copy()
    kind = int(rng.integers(0, 4))
    if kind == 0:
        kf *= np.linspace(0.2, float(rng.choice([8.0, 20.0])), T, dtype=np.float32)[:, None, None]
    elif kind == 1:
        kf[rng.choice(T, size=8, replace=False)] *= 40.0
    elif kind == 2:
        qf *= np.exp(rng.normal(0, 1.5, size=(T, 1, 1))).astype(np.float32)
    else:
        kf[:] = -np.abs(kf); qf[:] = np.abs(qf); kf[T - 70:] = np.abs(kf[T - 70:]) * 3
    k, q = W.f32_to_bf16_bits(kf), W.f32_to_bf16_bits(qf)
    rp, col = [0], []
    for S in lens:
        for _h in range(hq):
            for i in range((S + 63) // 64):
                keep = {i} if rng.random() < 0.9 else set()
                keep |= {int(j) for j in range(i + 1) if rng.random() < 0.5}
                col.extend(sorted(keep)); rp.append(len(col))
    rp, col = np.asarray(rp, np.int64), np.asarray(col, np.int32)
    p = Prefill(w.cu_seqlens, hq, 1, ctx=ctx, want_lse=True)
    p.set_inputs(q, k, w.v, w.wq, w.wk)
    p.set_lists(rp, col)
    o_ref, lse_ref = O.sparse_attention(q, k, w.v, w.cu_seqlens, rp, col, hq, 1, 64, 1 / math.sqrt(128))
    fin = np.isfinite(lse_ref)
    try:
        for impl in (0, 1):
            B.seer_set_attn_impl(ctx, impl)
            p.o.fill_(float("nan"))
            p.attn()
            assert p.status() == 0, (seed, impl)
            x, lg = p.o_host().astype(np.float64), p.lse_host().astype(np.float64)
            assert np.all(np.abs(x - o_ref) <= 2e-2 + 1e-2 * np.abs(o_ref)), (seed, impl, kind)
            assert np.all(np.abs(lg[fin] - lse_ref[fin]) <= 2e-3 + 1e-3 * np.abs(lse_ref[fin])), (seed, impl, kind)
            assert np.all(np.isneginf(lg[~fin]))
    finally:
        B.seer_set_attn_impl(ctx, 0)
