"""seer_gate_scores_static: the gate for callers that may not allocate device memory (a server whose pool owns all of
HBM, a plugin that must not call cudaMalloc inside someone else's allocator).  It takes no context and no workspace;
its intermediates sit in a fixed array inside the library that every call on the device shares.

The checks: through the C ABI, calls in a row (different shapes, so a later call finds an earlier call's leftovers in
the array) must give the same scores as seer_gate_scores and as the CPU oracle, within the gate tolerance of the other
GPU tests (1e-3 relative); from the second call on the free device memory must be exactly what it was before the call;
the largest shape that fits (10922 (head, block) pairs of 768 bytes) must be accepted and the next one refused.  The
file sorts last so that a run stopping at the first failure has already run everything else; it also passes on its own
in a fresh process."""
import ctypes as C

import numpy as np
import pytest

from paper_2410_13276_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _scores_both_ways(B, Prefill, ctx, w, check_memory):
    import torch
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, ctx=ctx)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    p.gate()
    ref = p.scores_host().copy()
    out = torch.full_like(p.scores, float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.seer_gate_scores_static(p.shape, p.q, p.k, p.wq, p.wk, out)
    torch.cuda.synchronize()
    if check_memory:                     # (the first call on a device may load the library's image lazily)
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
    return ref, out[: ref.size].cpu().numpy(), p


def _check(ref, got, w):
    from oracle import seer_oracle as O
    refs = O.unflatten_scores(ref, w.cu_seqlens, 64, w.num_q_heads)
    gots = O.unflatten_scores(got, w.cu_seqlens, 64, w.num_q_heads)
    for r, g in zip(refs, gots):
        il = np.tril_indices(r.shape[-1])
        rr, gg = r[:, il[0], il[1]].astype(np.float64), g[:, il[0], il[1]].astype(np.float64)
        assert np.all(np.abs(gg - rr) <= 1e-3 * np.abs(rr))


def test_static_gate_matches_workspace_gate_on_two_calls_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests must run on a B200")
    from paper_2410_13276_b200 import binding as B
    from paper_2410_13276_b200.prefill import Prefill
    ctx = B.Context(0)
    try:
        big = W.make_small(301, [2048, 700], 8, 2)          # fills more of the array
        small = W.make_small(302, [130, 0, 65], 6, 3)       # then a smaller, ragged batch over the leftovers
        from oracle import seer_oracle as O
        for n, w in enumerate((big, small, big)):
            ref, got, _ = _scores_both_ways(B, Prefill, ctx, w, check_memory=n >= 1)
            _check(ref, got, w)
            oracle = np.concatenate([x.astype(np.float32).ravel() for x in O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 64)])
            _check(oracle, got, w)       # and directly against the CPU oracle
    finally:
        ctx.close()


def test_static_gate_refuses_what_does_not_fit():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests must run on a B200")
    from paper_2410_13276_b200 import binding as B
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    # 40 heads x 2048 blocks x 768 B = 63 MB of intermediates > 8 MiB built in
    too_big = B.make_shape([0, 131072], 32, 8)
    with pytest.raises(B.SeerError) as e:
        B.seer_gate_scores_static(too_big, buf, buf, buf, buf, buf)
    assert e.value.status == 3                                  # SEER_ERR_WORKSPACE
    many = B.make_shape(list(range(0, 64 * 300, 64)), 2, 1)      # 299 sequences > SEER_STATIC_MAX_BATCH
    with pytest.raises(B.SeerError) as e:
        B.seer_gate_scores_static(many, buf, buf, buf, buf, buf)
    assert e.value.status == 3
    with pytest.raises(B.SeerError) as e:
        B.seer_gate_scores_static(B.make_shape([0, 128], 2, 1), None, buf, buf, buf, buf)
    assert e.value.status == 1


def test_static_gate_accepts_exactly_what_fits():
    """10922 (head, block) pairs of 768 bytes are the most the 8 MiB array holds: 1 + 1 heads x 5461 blocks run (and
    agree with seer_gate_scores), 2 + 1 heads x 3641 blocks = 10923 pairs are refused."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests must run on a B200")
    from paper_2410_13276_b200 import binding as B
    from paper_2410_13276_b200.prefill import Prefill
    ctx = B.Context(0)
    try:
        w = W.make_small(303, [5461 * 64], 1, 1)
        ref, got, _ = _scores_both_ways(B, Prefill, ctx, w, check_memory=False)
        nb = 5461
        il = np.tril_indices(nb)
        r, g = ref.reshape(nb, nb)[il].astype(np.float64), got.reshape(nb, nb)[il].astype(np.float64)
        assert np.all(np.abs(g - r) <= 1e-3 * np.abs(r))
    finally:
        ctx.close()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SeerError) as e:
        B.seer_gate_scores_static(B.make_shape([0, 3641 * 64], 2, 1), buf, buf, buf, buf, buf)
    assert e.value.status == 3                                  # SEER_ERR_WORKSPACE
