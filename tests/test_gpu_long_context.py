"""One 655 360-token sequence with 32 / 8 heads: q and o have 2.68e9 elements, more than 2^31, so every token / head /
element offset in the kernels must be 64-bit (nothing else in the suite reaches that size).  Inputs are drawn on the
device (seeded); gate and mask go through the one-call path (no 13 GB score matrix).  Checked: list lengths in closed
form for all 327 680 rows, attention and lse of sampled rows at both ends of the tensors against the oracle, the lists of
the last rows of one head against the oracle's gate + TopK, and that every output row was written."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_655k_tokens_beyond_2_31_elements():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests must run on a B200")
    from paper_2410_13276_b200 import binding as B
    from paper_2410_13276_b200.prefill import Prefill
    T, hq, hkv = 655360, 32, 8
    gen = torch.Generator(device="cuda")
    gen.manual_seed(20241)

    def draw(heads):
        out = torch.empty((T, heads, 128), dtype=torch.bfloat16, device="cuda")
        for s in range(0, T, 65536):
            out[s:s + 65536] = torch.randn((min(65536, T - s), heads, 128), generator=gen, device="cuda").to(torch.bfloat16)
        return out

    q, k, v = draw(hq), draw(hkv), draw(hkv)
    assert q.numel() > 2 ** 31
    wq_h, wk_h = W.make_gate_weights(1, hq, 128), W.make_gate_weights(2, hkv, 128)
    nb = T // 64
    cap = int(hq * (nb * (nb + 1) // 2) * 0.11) + hq * nb * 3
    ctx = B.Context(0)
    try:
        p = Prefill([0, T], hq, hkv, ctx=ctx, want_lse=True, col_capacity=cap)
        p.q, p.k, p.v = q, k, v
        p.wq, p.wk = torch.from_numpy(wq_h).cuda(), torch.from_numpy(wk_h).cuda()
        p.scores = None
        params = B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=10, flags=3)
        p.o.fill_(float("nan"))
        p.gate_mask(params, band_bytes=1 << 30)
        p.attn()
        assert p.status() == 0
        rp = p.row_ptr.cpu().numpy().astype(np.int64)
        i = np.tile(np.arange(nb), hq)
        want = np.maximum(np.clip(-((-(i + 1)) // 10), 1, i + 1), np.where(i == 0, 1, 2))
        assert np.array_equal(np.diff(rp), want) and int(p.nnz.item()) == int(rp[-1])
        assert not bool(torch.isnan(p.o).any())                       # every row written
        # sampled rows, the last ones beyond element 2^31 of q / o
        rows = [5, 7 * nb + nb // 2, 16 * nb + 3 * nb // 4, 30 * nb + nb - 1, 31 * nb + nb - 2, 31 * nb + nb - 1]
        col = np.zeros(int(rp[-1]), dtype=np.int32)
        for r in rows:
            col[rp[r]:rp[r + 1]] = p.col_idx[rp[r]:rp[r + 1]].cpu().numpy()
        kb = k.view(torch.int16).cpu().numpy().view(np.uint16)
        vb = v.view(torch.int16).cpu().numpy().view(np.uint16)
        qb = np.zeros((T, hq, 128), dtype=np.uint16)
        for r in rows:
            h, ii = divmod(r, nb)
            qb[ii * 64:(ii + 1) * 64, h] = q[ii * 64:(ii + 1) * 64, h].view(torch.int16).cpu().numpy().view(np.uint16)
        o_ref, lse_ref = O.sparse_attention(qb, kb, vb, [0, T], rp, col, hq, hkv, 64, 1 / math.sqrt(128), rows=rows)
        for r in rows:
            h, ii = divmod(r, nb)
            sl = slice(ii * 64, (ii + 1) * 64)
            x, ref = p.o[sl, h].float().cpu().numpy().astype(np.float64), o_ref[sl, h]
            assert np.all(np.abs(x - ref) <= 2e-2 + 1e-2 * np.abs(ref)), r
            lg, lr = p.lse[h, sl].cpu().numpy().astype(np.float64), lse_ref[h, sl]
            assert np.all(np.abs(lg - lr) <= 2e-3 + 1e-3 * np.abs(lr)), r
        # lists of the last rows of the last head against the oracle's gate + TopK; scores this long are nearly uniform, so
        # only blocks whose oracle score clears the selection boundary by the gate tolerance are required to agree
        h = hq - 1
        qh = q[:, h:h + 1].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        sc = O.gate_scores(qh, np.ascontiguousarray(kb[:, hkv - 1:hkv]), wq_h[h:h + 1], wk_h[hkv - 1:hkv], [0, T], 64)[0][0]
        for ii in range(nb - 8, nb):
            r = h * nb + ii
            got = set(p.col_idx[rp[r]:rp[r + 1]].cpu().numpy().tolist())
            row = sc[ii, :ii + 1].astype(np.float64)
            kth = np.sort(row)[::-1][len(got) - 1]
            sure_in = set(np.flatnonzero(row > kth * (1 + 4e-3)).tolist()) | {0, ii}
            sure_out = set(np.flatnonzero(row < kth * (1 - 4e-3)).tolist()) - {0, ii}
            assert sure_in <= got and not (sure_out & got), ii
    finally:
        ctx.close()
