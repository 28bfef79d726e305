"""The bounded waits of the tcgen05 attention kernel, exercised without faulting anything (needs a B200).

seer_debug_lost_wait makes exactly one wait run out: the first stream of CTA 0 never issues the V copy of one of its
tiles, so the MMA issuer's wait for that copy expires after the (shortened) limit.  What must then hold: the device
status is SEER_ERR_TIMEOUT, the kernel has returned (the call and the poll come back), every row that does not belong
to the stream that lost its copy equals the normal run bit for bit, and the context goes on working: the next call
without the hook gives the normal result (so the tensor memory of the aborted CTA was freed and no barrier is left
half-armed).
"""
import numpy as np
import pytest

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
    B.seer_debug_lost_wait(ctx, 2_000_000, -1)
    ctx.close()


@pytest.mark.parametrize("lost_tile", [0, 3])
def test_a_lost_copy_raises_timeout_and_the_context_survives(rt, lost_tile):
    import torch
    B, Prefill, ctx = rt
    hq, hkv, S = 8, 2, 4096
    w = W.make_small(seed=4242, seqlens=[S], hq=hq, hkv=hkv)
    p = Prefill(w.cu_seqlens, hq, hkv, ctx=ctx, want_lse=True)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=2, flags=B.SEER_FORCE_DIAG | B.SEER_FORCE_SINK)
    p.gate(); p.mask(params)
    p.attn(dynamic=False); torch.cuda.synchronize()
    assert p.status() == 0
    o_ref, lse_ref = p.o.clone(), p.lse.clone()

    # rows (head, query block) of the first stream of CTA 0: work items 0, 2 * grid, ... in the kernel's order
    # (KV head, query block from the last to the first, head within the group), two streams per CTA
    nb = S // 64
    rows = hq * nb
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    grid = min(sms, (rows + 1) // 2)
    group = hq // hkv
    lost_rows = set()
    for wi in range(0, rows, 2 * grid):
        g, rem = divmod(wi, nb * group)
        lost_rows.add((g * group + rem % group, nb - 1 - rem // group))

    B.seer_debug_lost_wait(ctx, 2_000, lost_tile)                  # 2 ms instead of 2 s
    try:
        p.o.fill_(float("nan")); p.lse.fill_(float("nan"))
        p.attn(dynamic=False)                                      # static deal: the rows of the stream that loses its copy are known
        status = B.seer_poll_device_status(ctx)                    # synchronises: the kernel has returned
    finally:
        B.seer_debug_lost_wait(ctx, 2_000_000, -1)
    assert B.STATUS_NAMES[status] == "SEER_ERR_TIMEOUT"
    o_bad, lse_bad = p.o.clone(), p.lse.clone()
    keep = torch.ones((hq, nb), dtype=torch.bool)
    for h, i in lost_rows:
        keep[h, i] = False
    keep_tok = keep.repeat_interleave(64, dim=1).cuda()            # [hq, S]
    assert torch.equal(o_bad.permute(1, 0, 2)[keep_tok], o_ref.permute(1, 0, 2)[keep_tok]), "a row of another stream changed"
    assert torch.equal(lse_bad[keep_tok], lse_ref[keep_tok])
    # the item that lost its copy cannot have been written
    h0, i0 = 0, nb - 1
    assert torch.isnan(o_bad[i0 * 64:(i0 + 1) * 64, h0].float()).all()

    # the context still works and the result is the normal one
    p.o.fill_(float("nan")); p.lse.fill_(float("nan"))
    p.attn(); torch.cuda.synchronize()                             # (with the work counter: the same result bit for bit)
    assert p.status() == 0
    assert torch.equal(p.o, o_ref) and torch.equal(p.lse, lse_ref)


def test_lost_wait_hook_rejects_a_zero_limit(rt):
    B, _, ctx = rt
    with pytest.raises(B.SeerError):
        B.seer_debug_lost_wait(ctx, 0, -1)
