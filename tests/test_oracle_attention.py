"""Pins for the attention oracle (dense attention of Sec. 2 restricted to the
listed blocks, Sec. 3.3) and for the max-pooled attention map (Sec. 3.2 and the
appendix identity a_ij = exp(r_ij - m_i) / l_i)."""
import math

import numpy as np
import pytest

from oracle import seer_oracle as O
from paper_2410_13276_b200 import workloads as W


def small(seed, seqlens, hq, hkv, **kw):
    return W.make_small(seed, seqlens, hq, hkv, **kw)


def attn(w, row_ptr, col, rows=None, q=None, k=None, v=None):
    return O.sparse_attention(w.q if q is None else q, w.k if k is None else k, w.v if v is None else v,
                              w.cu_seqlens, row_ptr, col, w.num_q_heads, w.num_kv_heads, w.block,
                              1.0 / math.sqrt(w.head_dim), rows=rows)


def brute_dense_causal(qf, kf, vf, scale):
    """Loop-level dense causal softmax attention for one head: [S, d] arrays."""
    S, d = qf.shape
    out = np.zeros((S, d))
    lse = np.zeros(S)
    for t in range(S):
        logits = [scale * sum(qf[t, c] * kf[s, c] for c in range(d)) for s in range(t + 1)]
        mx = max(logits)
        p = [math.exp(x - mx) for x in logits]
        den = sum(p)
        for s in range(t + 1):
            out[t] += p[s] / den * vf[s]
        lse[t] = mx + math.log(den)
    return out, lse


def test_full_lists_equal_brute_force_dense_causal():
    w = small(20, [11, 6], 4, 2, block=4, head_dim=8)
    rp, col = O.full_causal_lists(w.cu_seqlens, 4, 4)
    o, lse = attn(w, rp, col)
    qf, kf, vf = (O.bf16_bits_to_f64(x) for x in (w.q, w.k, w.v))
    for b in range(2):
        s0, s1 = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        for h in range(4):
            ref, rl = brute_dense_causal(qf[s0:s1, h], kf[s0:s1, h // 2], vf[s0:s1, h // 2], 1 / math.sqrt(8))
            np.testing.assert_allclose(o[s0:s1, h], ref, atol=1e-12)
            np.testing.assert_allclose(lse[h, s0:s1], rl, atol=1e-12)


def test_equals_dense_softmax_with_token_mask_expanded_from_lists():
    w = small(21, [23], 2, 1, block=4, head_dim=8)
    nb = 6
    rng = np.random.default_rng(0)
    scores = [rng.random((2, nb, nb)).astype(np.float32)]
    rp, col = O.block_mask(scores, O.MODE_TOPK_COUNT, k=3, flags=O.FORCE_DIAG)
    o, _ = attn(w, rp, col)
    qf, kf, vf = (O.bf16_bits_to_f64(x) for x in (w.q, w.k, w.v))
    for h in range(2):
        bias = np.full((23, 23), -np.inf)
        for i in range(nb):
            for j in col[rp[h * nb + i]:rp[h * nb + i + 1]]:
                for t in range(4 * i, min(4 * i + 4, 23)):
                    for s in range(4 * j, min(4 * j + 4, 23)):
                        if s <= t:
                            bias[t, s] = 0.0
        A = qf[:, h] @ kf[:, 0].T / math.sqrt(8) + bias
        A = np.exp(A - A.max(axis=1, keepdims=True))
        A /= A.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(o[:, h], A @ vf[:, 0], atol=1e-12)


def test_constant_v_gives_constant_output_for_any_mask():
    w = small(22, [37], 2, 2, block=8, head_dim=8)
    v = W.f32_to_bf16_bits(np.ones((37, 2, 8), np.float32))
    scores = [np.random.default_rng(1).random((2, 5, 5)).astype(np.float32)]
    rp, col = O.block_mask(scores, O.MODE_THRESHOLD, threshold=0.6, flags=O.FORCE_DIAG)
    o, _ = attn(w, rp, col, v=v)
    np.testing.assert_allclose(o, 1.0, atol=1e-14)


def test_single_key_returns_its_value_row():
    w = small(23, [6], 1, 1, block=1, head_dim=4)
    vf = O.bf16_bits_to_f64(w.v)
    # token 0 of any sequence sees only key 0
    rp, col = O.full_causal_lists(w.cu_seqlens, 1, 1)
    o, lse = attn(w, rp, col)
    np.testing.assert_array_equal(o[0, 0], vf[0, 0])
    # B = 1 and one listed block per row: the output is that block's V row
    pick = [0, 0, 2, 1, 4, 3]
    o, _ = attn(w, np.arange(7), np.asarray(pick, np.int32))
    for t, j in enumerate(pick):
        np.testing.assert_allclose(o[t, 0], vf[j, 0], atol=1e-15)
    # zero keys -> uniform softmax -> lse = log(number of visible keys)
    k0 = W.f32_to_bf16_bits(np.zeros((6, 1, 4), np.float32))
    _, lse = attn(w, rp, col, k=k0)
    np.testing.assert_allclose(lse[0], np.log(np.arange(1, 7)), atol=1e-14)


def test_diagonal_only_lists_equal_local_block_attention():
    w = small(24, [20], 2, 1, block=8, head_dim=8)
    nb = 3
    rp = np.arange(2 * nb + 1)
    col = np.asarray(list(range(nb)) * 2, np.int32)
    o, _ = attn(w, rp, col)
    qf, kf, vf = (O.bf16_bits_to_f64(x) for x in (w.q, w.k, w.v))
    for h in range(2):
        for i in range(nb):
            t0, t1 = 8 * i, min(8 * i + 8, 20)
            ref, _ = brute_dense_causal(qf[t0:t1, h], kf[t0:t1, 0], vf[t0:t1, 0], 1 / math.sqrt(8))
            np.testing.assert_allclose(o[t0:t1, h], ref, atol=1e-12)


def test_list_order_does_not_matter_and_lse_merge():
    w = small(25, [48], 1, 1, block=8, head_dim=16)
    # row 5 (last block) with lists A = {0, 3}, B = {1, 5}, and their union
    def run(lst):
        rp = np.zeros(7, np.int64)
        rp[6] = len(lst)
        return attn(w, rp, np.asarray(lst, np.int32), rows=[5])
    oa, la = run([0, 3])
    ob, lb = run([1, 5])
    ou, lu = run([0, 1, 3, 5])
    op, lp = run([5, 0, 3, 1])
    t = slice(40, 48)
    np.testing.assert_allclose(op[t], ou[t], atol=1e-12)
    # combine two partial softmaxes through their log-sum-exp (the identity behind the online rescale)
    la, lb, lu = la[0, t], lb[0, t], lu[0, t]
    np.testing.assert_allclose(np.logaddexp(la, lb), lu, atol=1e-12)
    wa, wb = np.exp(la - lu)[:, None], np.exp(lb - lu)[:, None]
    np.testing.assert_allclose(wa * oa[t, 0] + wb * ob[t, 0], ou[t, 0], atol=1e-12)
    assert np.isnan(ou[:40]).all()                                   # rows not asked for stay untouched


def test_gqa_heads_share_kv_and_sequences_do_not_leak():
    w = small(26, [12, 9], 4, 2, block=4, head_dim=8)
    q = w.q.copy()
    q[:, 1] = q[:, 0]                                                # heads 0,1 share KV head 0
    q[:, 3] = q[:, 0]                                                # head 3 uses KV head 1
    rp, col = O.full_causal_lists(w.cu_seqlens, 4, 4)
    o, _ = attn(w, rp, col, q=q)
    np.testing.assert_array_equal(o[:, 0], o[:, 1])
    assert np.abs(o[:, 0] - o[:, 3]).max() > 1e-3
    k2, v2 = w.k.copy(), w.v.copy()
    k2[:12] = k2[:12][::-1]
    v2[:12] = 0                                                      # perturb sequence 0 only
    o2, _ = attn(w, rp, col, q=q, k=k2, v=v2)
    np.testing.assert_array_equal(o2[12:], o[12:])


def test_empty_list_gives_zero_and_minus_inf():
    w = small(27, [8], 1, 1, block=4, head_dim=4)
    o, lse = attn(w, np.array([0, 1, 1]), np.array([0], np.int32))
    assert np.all(o[4:] == 0) and np.all(np.isneginf(lse[0, 4:])) and np.all(np.isfinite(o[:4]))


def test_maxpool_map_brute_force_and_appendix_identity():
    w = small(28, [22], 2, 1, block=4, head_dim=8)
    B, nb, S = 4, 6, 22
    gt = O.maxpool_attention_map(w.q, w.k, w.cu_seqlens, 2, 1, B, 1 / math.sqrt(8))[0]
    qf, kf = O.bf16_bits_to_f64(w.q), O.bf16_bits_to_f64(w.k)
    rp, col = O.full_causal_lists(w.cu_seqlens, B, 2)
    _, lse = attn(w, rp, col)
    for h in range(2):
        A = np.zeros((S, S))
        for t in range(S):
            lg = np.array([qf[t, h] @ kf[s, 0] / math.sqrt(8) for s in range(t + 1)])
            p = np.exp(lg - lg.max())
            A[t, : t + 1] = p / p.sum()
        for i in range(nb):
            for j in range(nb):
                blk = A[B * i:B * i + B, B * j:B * j + B]
                assert abs(gt[h, i, j] - (blk.max() if j <= i else 0.0)) <= 1e-14
                if j <= i:
                    # appendix: a = exp(r_ij - m_i) / l_i per query row, then the max over the block's rows
                    a = []
                    for t in range(B * i, min(B * i + B, S)):
                        keys = [s for s in range(B * j, min(B * j + B, S)) if s <= t]
                        if keys:
                            r = max(qf[t, h] @ kf[s, 0] / math.sqrt(8) for s in keys)
                            a.append(math.exp(r - lse[h, t]))
                    assert abs(gt[h, i, j] - max(a)) <= 1e-13
    np.testing.assert_allclose(gt[:, 0, 0], 1.0)                      # token 0 puts all its mass on key 0


# --------------------------------------------------------------------------- max-pooled map on listed blocks
def test_maxpool_listed_blocks_dense_lists_equal_eq2_map():
    """Full causal lists: every entry is the B x B max-pool of the dense causal softmax map (Eq. 2)."""
    w = W.make_small(seed=61, seqlens=[50, 23], hq=4, hkv=2, block=8, head_dim=16)
    rp, col = O.full_causal_lists(w.cu_seqlens, w.block, w.num_q_heads)
    got = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, w.num_q_heads, w.num_kv_heads, w.block, 0.25)
    gt = O.maxpool_attention_map(w.q, w.k, w.cu_seqlens, w.num_q_heads, w.num_kv_heads, w.block, 0.25)
    base = O.row_base(w.cu_seqlens, w.block, w.num_q_heads)
    for b, nb in enumerate(O.blocks_per_sequence(w.cu_seqlens, w.block)):
        for h in range(w.num_q_heads):
            for i in range(int(nb)):
                r = int(base[b]) + h * int(nb) + i
                for p_ in range(int(rp[r]), int(rp[r + 1])):
                    assert got[p_] == pytest.approx(gt[b][h, i, int(col[p_])], rel=1e-12, abs=0)


def test_maxpool_listed_blocks_block_one_is_the_softmax_itself():
    """B = 1: a tile is one (query, key) pair, so the values of a row are its softmax probabilities and sum to 1."""
    w = W.make_small(seed=62, seqlens=[12], hq=2, hkv=1, block=1, head_dim=8)
    rng = np.random.default_rng(5)
    rp, col = [0], []
    for h in range(2):
        for i in range(12):
            keep = sorted(set([i] + [int(j) for j in rng.choice(i + 1, size=min(3, i + 1), replace=False)]))
            col += keep
            rp.append(len(col))
    rp, col = np.array(rp), np.array(col)
    got = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, 2, 1, 1, 0.3)
    Q, K = O.bf16_bits_to_f64(w.q), O.bf16_bits_to_f64(w.k)
    for r in range(24):
        h, i = divmod(r, 12)
        js = col[rp[r]:rp[r + 1]]
        s = np.array([Q[i, h] @ K[j, 0] * 0.3 for j in js])
        want = np.exp(s - s.max()) / np.exp(s - s.max()).sum()
        np.testing.assert_allclose(got[rp[r]:rp[r + 1]], want, rtol=1e-12)
        assert got[rp[r]:rp[r + 1]].sum() == pytest.approx(1.0, abs=1e-12)


def test_maxpool_listed_blocks_invariants():
    w = W.make_small(seed=63, seqlens=[70], hq=2, hkv=1, block=16, head_dim=8)
    scores = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, w.block)
    rp, col = O.block_mask(scores, O.MODE_TOPK_RATIO, keep_num=1, keep_den=2, flags=O.FORCE_DIAG)
    got = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, 2, 1, 16, 0.35)
    assert np.all(got > 0) and np.all(got <= 1.0)
    # order of a row's list does not matter: reversed lists give the reversed values
    col_r = col.copy()
    for r in range(len(rp) - 1):
        col_r[rp[r]:rp[r + 1]] = col[rp[r]:rp[r + 1]][::-1]
    got_r = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col_r, 2, 1, 16, 0.35)
    for r in range(len(rp) - 1):
        np.testing.assert_allclose(got_r[rp[r]:rp[r + 1]], got[rp[r]:rp[r + 1]][::-1], rtol=1e-12)
    # rows not asked for stay NaN
    part = O.maxpool_listed_blocks(w.q, w.k, w.cu_seqlens, rp, col, 2, 1, 16, 0.35, rows=[1])
    assert np.isnan(part[rp[2]:]).all() and not np.isnan(part[rp[1]:rp[2]]).any()

