"""Chunked prefill on the GPU (shape.cu_seqlens_q_host: the queries are the last S_q positions of each sequence).

Checked (a) against the oracle's chunk routines: score rows within 1e-3 relative, lists bit-exact (oracle mask on the
GPU's own score rows), attention within the stated tolerance with the GPU's lists fed to both; and (b) against the GPU's
own run of the whole problem, of which a chunk's results must be the matching rows, bit for bit (same kernels, same
arithmetic, same lists)."""
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


def make_chunk(w, starts):
    cu = w.cu_seqlens
    parts, cu_q = [], [0]
    for b, st in enumerate(starts):
        parts.append(w.q[cu[b] + st:cu[b + 1]])
        cu_q.append(cu_q[-1] + int(cu[b + 1] - cu[b] - st))
    q = np.concatenate(parts, axis=0) if sum(len(x) for x in parts) else np.zeros((0,) + w.q.shape[1:], np.uint16)
    return q, np.asarray(cu_q, dtype=np.int32)


CASES = [
    # (seqlens, chunk starts in tokens, hq, hkv, block, mask kwargs)
    ([512], [448], 2, 1, 64, dict(mode=O.MODE_TOPK_RATIO, keep_num=1, keep_den=2, flags=3)),            # the last block alone
    ([200, 64, 333, 130], [128, 0, 192, 130], 4, 2, 64, dict(mode=O.MODE_TOPK_RATIO, keep_num=1, keep_den=3, flags=3)),
    ([4099, 700], [2048, 640], 8, 4, 64, dict(mode=O.MODE_THRESHOLD, threshold=0.03, flags=1)),
    ([5000], [4992], 6, 2, 64, dict(mode=O.MODE_TOPK_COUNT, k=5, flags=3)),                               # 8 tokens against 4992 cached
    ([3000, 1000], [1024, 768], 4, 1, 128, dict(mode=O.MODE_TOPK_RATIO, keep_num=1, keep_den=2, flags=3)),
]


def rel_ok(got, ref):
    gg, rr = got.astype(np.float64), ref.astype(np.float64)
    return np.all(np.abs(gg - rr) <= np.where(rr < 1e-30, 1e-33, 1e-3 * rr))


@pytest.mark.parametrize("ci", range(len(CASES)))
@pytest.mark.parametrize("impl", [0, 1])
def test_chunk_against_oracle_and_whole_run(rt, ci, impl):
    B, Prefill, ctx = rt
    lens, starts, hq, hkv, blk, kw = CASES[ci]
    w = W.make_small(seed=99_000 + ci, seqlens=lens, hq=hq, hkv=hkv, q_gain=2.0, block=blk)
    qc, cu_q = make_chunk(w, starts)
    params = B.make_mask_params(kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                                k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw["flags"])
    B.seer_set_attn_impl(ctx, impl)
    try:
        full = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True, block=blk)
        full.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
        full.run(params)
        part = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True, block=blk, cu_seqlens_q=cu_q)
        part.set_inputs(qc, w.k, w.v, w.wq, w.wk)
        part.scores.fill_(float("nan"))
        part.o.fill_(float("nan"))
        part.run(params)
        assert full.status() == 0 and part.status() == 0
    finally:
        B.seer_set_attn_impl(ctx, 0)
    offs = O.chunk_offsets(cu_q, w.cu_seqlens, blk)
    s_full = O.unflatten_scores(full.scores_host(), w.cu_seqlens, blk, hq)
    s_part = O.unflatten_scores(part.scores_host(), w.cu_seqlens, blk, hq)
    ref = O.gate_scores_chunk(qc, w.k, w.wq, w.wk, cu_q, w.cu_seqlens, blk)
    rows_part = []
    for b in range(len(lens)):
        off = int(offs[b])
        nb = s_full[b].shape[-1]
        rows = s_part[b][:, off:, :]
        rows_part.append(rows)
        for i in range(off, nb):
            assert np.array_equal(rows[:, i - off, :i + 1], s_full[b][:, i, :i + 1])          # (b) rows of the whole run
            assert rel_ok(rows[:, i - off, :i + 1], ref[b][:, i - off, :i + 1])                 # (a) the oracle
    # lists
    rp, col = part.lists_host()
    orp, ocol = O.block_mask_chunk(rows_part, kw["mode"], keep_num=kw.get("keep_num", 1), keep_den=kw.get("keep_den", 1),
                                   k=kw.get("k", 0), threshold=kw.get("threshold", 0.0), flags=kw["flags"])
    assert np.array_equal(rp, orp) and np.array_equal(col, ocol)
    rp_f, col_f = full.lists_host()
    r = 0
    for b, S in enumerate(lens):
        nb = (S + blk - 1) // blk
        for h in range(hq):
            for i in range(nb):
                want = col_f[rp_f[r]:rp_f[r + 1]] if i >= int(offs[b]) else col_f[:0]
                assert np.array_equal(col[rp[r]:rp[r + 1]], want)
                r += 1
    # attention
    o_part, lse_part = part.o_host(), part.lse_host()
    o_full, lse_full = full.o_host(), full.lse_host()
    for b, st in enumerate(starts):
        k0, k1 = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        q0, q1 = int(cu_q[b]), int(cu_q[b + 1])
        assert np.array_equal(o_part[q0:q1], o_full[k0 + st:k1])
        assert np.array_equal(lse_part[:, q0:q1], lse_full[:, k0 + st:k1])
    assert not np.isnan(o_part).any()
    o_ref, lse_ref = O.sparse_attention_chunk(qc, w.k, w.v, cu_q, w.cu_seqlens, rp, col, hq, hkv, blk, 1 / math.sqrt(128))
    err = np.abs(o_part.astype(np.float64) - o_ref)
    assert np.all(err <= 2e-2 + 1e-2 * np.abs(o_ref))
    assert np.all(np.abs(lse_part.astype(np.float64) - lse_ref) <= 2e-3 + 1e-3 * np.abs(lse_ref))
    # gate + mask in one call (small bands), and the max-pooled map on the kept blocks
    part.row_ptr.fill_(-1)
    part.gate_mask(params, band_bytes=0)
    rp2, col2 = part.lists_host()
    assert part.status() == 0 and np.array_equal(rp2, rp) and np.array_equal(col2, col)
    if blk == 64:
        bm_part = part.block_max().cpu().numpy()[:len(col)]
        bm_full = full.block_max().cpu().numpy()[:len(col_f)]
        r = 0
        for b, S in enumerate(lens):
            nb = (S + 63) // 64
            for h in range(hq):
                for i in range(nb):
                    if i >= int(offs[b]):
                        assert np.array_equal(bm_part[rp[r]:rp[r + 1]], bm_full[rp_f[r]:rp_f[r + 1]])
                    r += 1


def test_chunk_with_rope_and_pooling_options(rt):
    import torch
    B, Prefill, ctx = rt
    lens, starts, hq, hkv = [3000, 130], [1984, 64], 4, 2
    w = W.make_small(seed=99_100, seqlens=lens, hq=hq, hkv=hkv)
    qc, cu_q = make_chunk(w, starts)
    wq = W.make_gate_weights(25, hq, 2 * 128)
    wk = W.make_gate_weights(26, hkv, 3 * 128)
    opt = B.seer_gate_options(3, 7, 500000.0)                   # avg+max on Q, all three on K, block RoPE
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=False, cu_seqlens_q=cu_q)
    p.set_inputs(qc, w.k, w.v, w.wq, w.wk)
    p.gate_ex(opt, torch.from_numpy(wq).cuda(), torch.from_numpy(wk).cuda())
    assert p.status() == 0
    got = O.unflatten_scores(p.scores_host(), w.cu_seqlens, 64, hq)
    ref = O.gate_scores_chunk(qc, w.k, wq, wk, cu_q, w.cu_seqlens, 64, pool_q=3, pool_k=7, rope_theta=500000.0)
    offs = O.chunk_offsets(cu_q, w.cu_seqlens, 64)
    for b in range(2):
        off = int(offs[b])
        for i in range(off, got[b].shape[-1]):
            assert rel_ok(got[b][:, i, :i + 1], ref[b][:, i - off, :i + 1])


def test_chunk_shape_validation(rt):
    import torch
    B, Prefill, ctx = rt
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    for cu_q, want in (([0, 300], 1), ([0, 100], 2), ([5, 64], 1)):       # more queries than keys; unaligned start; cu_q[0] != 0
        s = B.make_shape([0, 200], 2, 1, cu_seqlens_q=cu_q)
        assert B.seer_mask_rows(s) == -1
        with pytest.raises(B.SeerError) as e:
            B.seer_gate_scores(ctx, s, buf, buf, buf, buf, buf, buf)
        assert e.value.status == want
    s = B.make_shape([0, 200], 2, 1, cu_seqlens_q=[0, 72])               # starts at token 128
    assert B.seer_mask_rows(s) == 2 * 4
    with pytest.raises(B.SeerError) as e:
        B.seer_gate_scores_static(s, buf, buf, buf, buf, buf)
    assert e.value.status == 2


@pytest.mark.parametrize("seed", list(range(24)) + [345])
def test_random_chunks_equal_rows_of_the_whole_run(rt, seed):
    """Seeded random packed batches, chunk starts and mask modes: scores, lists, o and lse of the chunk equal the matching
    rows of the GPU's whole-problem run exactly (that run is what the other tests hold against the oracle)."""
    B, Prefill, ctx = rt
    rng = np.random.default_rng(123_000 + seed)
    blk = int(rng.choice([64, 64, 128]))
    nseq = int(rng.integers(1, 4))
    lens = [int(x) for x in rng.choice([1, 64, 65, 200, 333, 512, 700, 1300], size=nseq)]
    starts = []
    for S in lens:
        nb = (S + blk - 1) // blk
        c = int(rng.integers(0, nb + 1))                     # nb: the sequence contributes no query
        starts.append(S if c == nb else c * blk)
    hkv = int(rng.integers(1, 3)); hq = hkv * int(rng.choice([1, 2, 4]))
    mode = int(rng.integers(0, 3))
    params = B.make_mask_params(mode, keep_num=1, keep_den=int(rng.integers(2, 6)), k=int(rng.integers(0, 5)),
                                threshold=float(rng.choice([0.0, 0.05, 0.3])), flags=int(rng.choice([0, 1, 3])),
                                dense_tail=int(rng.choice([0, 0, 1])))
    w = W.make_small(seed=124_000 + seed, seqlens=lens, hq=hq, hkv=hkv, q_gain=2.0, block=blk)
    qc, cu_q = make_chunk(w, starts)
    full = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True, block=blk)
    full.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    full.run(params)
    part = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True, block=blk, cu_seqlens_q=cu_q)
    if qc.shape[0] == 0:
        qc = np.zeros((1,) + w.q.shape[1:], np.uint16)       # a buffer to point at; no query is read
    part.set_inputs(qc, w.k, w.v, w.wq, w.wk)
    part.o.fill_(float("nan"))
    part.run(params)
    assert full.status() == 0 and part.status() == 0, (lens, starts, blk)
    offs = O.chunk_offsets(cu_q, w.cu_seqlens, blk)
    rp, col = part.lists_host()
    rp_f, col_f = full.lists_host()
    s_full = O.unflatten_scores(full.scores_host(), w.cu_seqlens, blk, hq)
    s_part = O.unflatten_scores(part.scores_host(), w.cu_seqlens, blk, hq)
    r = 0
    for b, S in enumerate(lens):
        nb = (S + blk - 1) // blk
        for h in range(hq):
            for i in range(nb):
                if i >= int(offs[b]):
                    assert np.array_equal(s_part[b][h, i, :i + 1], s_full[b][h, i, :i + 1]), (lens, starts, b, h, i)
                    assert np.array_equal(col[rp[r]:rp[r + 1]], col_f[rp_f[r]:rp_f[r + 1]]), (lens, starts, b, h, i)
                else:
                    assert rp[r + 1] == rp[r]
                r += 1
    o_part, lse_part = part.o_host(), part.lse_host()
    o_full, lse_full = full.o_host(), full.lse_host()
    for b, st in enumerate(starts):
        k0, k1 = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        q0, q1 = int(cu_q[b]), int(cu_q[b + 1])
        assert np.array_equal(o_part[q0:q1], o_full[k0 + st:k1]), (lens, starts, blk)
        assert np.array_equal(lse_part[:, q0:q1], lse_full[:, k0 + st:k1])
