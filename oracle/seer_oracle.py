"""CPU oracle for the SeerAttention prefill hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the path computes, written from the
paper's definitions.  It shares no code with the CUDA library and must never
be imported by the product path: only the tests, the smoke check and the
benchmark's CPU-baseline leg use it.

What it follows
---------------
* AttnGate, Sec. 3.1 and Eq. 1:  score = softmax((Wq Pq(Q)) (Wk Pk(K))^T / sqrt(d)),
  with Pq, Pk non-overlapping pooling of kernel = stride = B along the sequence
  (`pool_avg`, `project`, `gate_logits`, `gate_scores`); its two refinements in the same
  section, composed avg/max/min pooling and block-level RoPE with theta/B
  (`pool_compose`, `block_rope`, `gate_scores_ex`).
* Binary block mask, Sec. 3.3 "Generating Binary Block Mask", Eq. 3 (TopK) and
  Eq. 4 (score > threshold) (`select_row`, `block_mask`).
* Block-sparse attention, Sec. 3.3 "Block Sparse Flash-Attn Kernel": the tiles
  of unselected blocks are skipped, i.e. dense attention A = softmax(QK^T/sqrt(d))
  (Sec. 2) with the unselected blocks removed from every softmax row
  (`sparse_attention`).
* Chunked prefill (the queries are the last S_q positions of a sequence of S_k keys): the same definitions with the
  query positions shifted (`chunk_offsets`, `gate_scores_chunk`, `block_mask_chunk`, `sparse_attention_chunk`); rows
  keep the numbering of the whole sequence, so a chunk's results are rows of the whole problem's.
* 2D-max-pooled attention map used as distillation target, Sec. 3.2 / Eq. 2 and
  the appendix's a_ij = exp(r_ij - m_i) / l_i (`maxpool_attention_map`).

Readings taken where the paper is silent (each is restated next to the code):
average pooling on both Q and K; per-query-head Wq and per-KV-head Wk applied
as row-vector x matrix, no bias; query head h uses KV head h // G; the sqrt(d)
of Eq. 1 is the gate's output width; the gate softmax is block-causal (j <= i);
scores are rounded once to fp32; TopK keeps k_i = ceil(rho * (i+1)) blocks in
row i with forced blocks counted inside k_i; ties go to the lower block index;
the threshold compare is strict and in fp32; NaN scores are never selected.

Parity pins (tests/test_oracle_*.py): every function here is pinned by closed
forms, invariants or brute force; none is "parity unpinned".

Conventions: bf16 tensors arrive as uint16 bit patterns; `cu_seqlens` are the
cumulative token offsets of the packed sequences; row id of (sequence b, query
head h, query block i) is Hq * off_b + h * nb_b + i with off_b the number of
blocks of the sequences before b.
"""
from __future__ import annotations

import math

import numpy as np

MODE_TOPK_RATIO = 0
MODE_TOPK_COUNT = 1
MODE_THRESHOLD = 2
FORCE_DIAG = 1
FORCE_SINK = 2


# --------------------------------------------------------------------------- helpers
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> fp64, exactly (bf16 is the top half of an fp32)."""
    return (np.asarray(bits).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def blocks_per_sequence(cu_seqlens, B: int) -> np.ndarray:
    lens = np.diff(np.asarray(cu_seqlens, dtype=np.int64))
    return (lens + B - 1) // B


def row_base(cu_seqlens, B: int, num_q_heads: int) -> np.ndarray:
    """First row id of each sequence (and the total as last entry)."""
    nb = blocks_per_sequence(cu_seqlens, B)
    return num_q_heads * np.concatenate([[0], np.cumsum(nb)])


# --------------------------------------------------------------------------- AttnGate (Sec. 3.1, Eq. 1)
def pool_avg(x_bits: np.ndarray, cu_seqlens, B: int) -> list:
    """P(X): average pooling along the sequence with kernel = stride = B
    (Sec. 3.1).  The last block of a sequence whose length is not a multiple
    of B averages the tokens it has.  Returns one [H, nb_b, d] array per sequence."""
    out = []
    for b in range(len(cu_seqlens) - 1):
        s0, s1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        nb = (s1 - s0 + B - 1) // B
        H, d = x_bits.shape[1], x_bits.shape[2]
        pooled = np.zeros((H, nb, d), dtype=np.float64)
        for i in range(nb):
            t0, t1 = s0 + i * B, min(s0 + (i + 1) * B, s1)
            blk = bf16_bits_to_f64(x_bits[t0:t1])            # [tokens, H, d]
            pooled[:, i, :] = blk.sum(axis=0) / float(t1 - t0)
        out.append(pooled)
    return out


def project(pooled: np.ndarray, W: np.ndarray) -> np.ndarray:
    """W P(X) of Eq. 1 for every head: out[h, i, :] = pooled[h, i, :] @ W[h]
    (row vector times the head's [d, dg] matrix, no bias)."""
    W = np.asarray(W, dtype=np.float64)
    return np.einsum("hic,hco->hio", pooled, W)


def gate_logits(gq: np.ndarray, gk: np.ndarray) -> np.ndarray:
    """(Wq Pq(Q)) (Wk Pk(K))^T / sqrt(d) of Eq. 1 for one sequence.
    gq [Hq, nb, dg], gk [Hkv, nb, dg]; query head h pairs with KV head h // G;
    d is the projected width dg.  Returns [Hq, nb, nb] (all j, causal or not)."""
    Hq, nb, dg = gq.shape
    G = Hq // gk.shape[0]
    L = np.empty((Hq, nb, nb), dtype=np.float64)
    for h in range(Hq):
        L[h] = gq[h] @ gk[h // G].T / math.sqrt(dg)
    return L


def causal_softmax_rows(L: np.ndarray, first: int = 0) -> np.ndarray:
    """Row softmax of Eq. 1 restricted to the causal blocks j <= i of row i
    (a query block cannot attend to later key blocks, and the rows must sum
    to 1 as Sec. 3.2 states).  Entries j > i are returned as 0.  `first` is the
    block position of row 0 (rows are query blocks first, first + 1, ...)."""
    S = np.zeros_like(L)
    for r in range(L.shape[-2]):
        i = first + r
        row = L[..., r, : i + 1]
        e = np.exp(row - row.max(axis=-1, keepdims=True))
        S[..., r, : i + 1] = e / e.sum(axis=-1, keepdims=True)
    return S


def gate_scores(q_bits, k_bits, wq, wk, cu_seqlens, B: int) -> list:
    """AttnGate of Eq. 1.  Returns, per sequence, the fp32 array [Hq, nb, nb]
    of gating scores (fp64 result rounded once to fp32; zero above the diagonal)."""
    pq = pool_avg(q_bits, cu_seqlens, B)
    pk = pool_avg(k_bits, cu_seqlens, B)
    out = []
    for b in range(len(pq)):
        gq = project(pq[b], wq)
        gk = project(pk[b], wk)
        out.append(causal_softmax_rows(gate_logits(gq, gk)).astype(np.float32))
    return out


# --------------------------------------------------------------------------- AttnGate variants (Sec. 3.1)
POOL_AVG = 1
POOL_MAX = 2
POOL_MIN = 4


def pool_compose(x_bits: np.ndarray, cu_seqlens, B: int, methods: int) -> list:
    """Sec. 3.1, "Pooling Method Selection": several pooling methods (average, max, min; kernel = stride = B)
    applied to the same tensor, their results concatenated in the hidden dimension before the linear layer.
    `methods` is a non-empty subset of POOL_AVG | POOL_MAX | POOL_MIN; the concatenation order is avg, max, min
    (a reading: the paper fixes no order, and a learned layer absorbs any).  A ragged last block pools the tokens
    it has.  Returns one [H, nb_b, n * d] array per sequence (n = number of methods)."""
    if methods <= 0 or methods & ~(POOL_AVG | POOL_MAX | POOL_MIN):
        raise ValueError("methods must be a non-empty subset of avg | max | min")
    out = []
    for b in range(len(cu_seqlens) - 1):
        s0, s1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        nb = (s1 - s0 + B - 1) // B
        H, d = x_bits.shape[1], x_bits.shape[2]
        parts = []
        for bit in (POOL_AVG, POOL_MAX, POOL_MIN):
            if not methods & bit:
                continue
            pooled = np.zeros((H, nb, d), dtype=np.float64)
            for i in range(nb):
                t0, t1 = s0 + i * B, min(s0 + (i + 1) * B, s1)
                blk = bf16_bits_to_f64(x_bits[t0:t1])        # [tokens, H, d]
                if bit == POOL_AVG:
                    pooled[:, i, :] = blk.sum(axis=0) / float(t1 - t0)
                elif bit == POOL_MAX:
                    pooled[:, i, :] = blk.max(axis=0)
                else:
                    pooled[:, i, :] = blk.min(axis=0)
            parts.append(pooled)
        out.append(np.concatenate(parts, axis=-1))
    return out


def block_rope(g: np.ndarray, theta: float, B: int, first: int = 0) -> np.ndarray:
    """Sec. 3.1, "Block-level RoPE in AttnGate": rotary position encoding applied after the gate's linear layer,
    at block granularity, with the reduced base theta' = theta / B.  g is [H, nb, dg] for one sequence; block i
    is position first + i.  Standard rotary form (a reading, the paper gives none): pair (c, c + dg/2), frequency
    theta'^(-2c/dg), (x_c, x_{c+dg/2}) -> (x_c cos a - x_{c+dg/2} sin a, x_{c+dg/2} cos a + x_c sin a), a = i * frequency."""
    H, nb, dg = g.shape
    half = dg // 2
    base = float(theta) / float(B)
    freq = base ** (-2.0 * np.arange(half, dtype=np.float64) / dg)          # [half]
    ang = (first + np.arange(nb, dtype=np.float64))[:, None] * freq[None, :]  # [nb, half]
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = g[..., :half], g[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def gate_scores_ex(q_bits, k_bits, wq, wk, cu_seqlens, B: int, pool_q: int = POOL_AVG, pool_k: int = POOL_AVG,
                   rope_theta: float = 0.0) -> list:
    """AttnGate of Eq. 1 with the paper's two refinements: composed pooling on Q and on K (wq is [Hq, nq*d, dg], wk
    [Hkv, nk*d, dg]) and, when rope_theta > 0, block-level RoPE on the projected tensors.  Defaults reduce to
    `gate_scores`.  Returns, per sequence, the fp32 array [Hq, nb, nb]."""
    pq = pool_compose(q_bits, cu_seqlens, B, pool_q)
    pk = pool_compose(k_bits, cu_seqlens, B, pool_k)
    out = []
    for b in range(len(pq)):
        gq = project(pq[b], wq)
        gk = project(pk[b], wk)
        if rope_theta > 0.0:
            gq, gk = block_rope(gq, rope_theta, B), block_rope(gk, rope_theta, B)
        out.append(causal_softmax_rows(gate_logits(gq, gk)).astype(np.float32))
    return out


def flatten_scores(scores: list) -> np.ndarray:
    """Per-sequence [Hq, nb, nb] arrays -> one flat array, sequence after sequence."""
    return np.concatenate([s.reshape(-1) for s in scores]) if scores else np.zeros(0, np.float32)


def unflatten_scores(flat: np.ndarray, cu_seqlens, B: int, num_q_heads: int) -> list:
    out, p = [], 0
    for nb in blocks_per_sequence(cu_seqlens, B):
        n = num_q_heads * int(nb) * int(nb)
        out.append(np.asarray(flat[p:p + n]).reshape(num_q_heads, int(nb), int(nb)))
        p += n
    return out


# --------------------------------------------------------------------------- block mask (Sec. 3.3, Eq. 3 / Eq. 4)
def keep_count(n: int, mode: int, keep_num: int = 1, keep_den: int = 1, k: int = 0) -> int:
    """Number of blocks TopK keeps in a row with n causal blocks: the "TopK
    ratio" of Sec. 3.3 as an exact rational, k_i = ceil(num * n / den) clamped
    to [1, n]; or a fixed count min(k, n)."""
    if mode == MODE_TOPK_RATIO:
        return min(max(-((-keep_num * n) // keep_den), 1), n)
    if mode == MODE_TOPK_COUNT:
        return min(max(k, 0), n)
    raise ValueError(mode)


def select_row(score_row: np.ndarray, i: int, mode: int, *, keep_num=1, keep_den=1, k=0,
               threshold=0.0, flags=FORCE_DIAG) -> list:
    """Kept key blocks of query-block row i (ascending), from its fp32 scores
    score_row[0..i].

    Forced blocks: the diagonal block i (FORCE_DIAG) and block 0 (FORCE_SINK).
    TopK (Eq. 3): forced blocks count toward k_i; the remaining k_i - |forced|
    places go to the best other blocks, ordered by score descending, then block
    index ascending.  Threshold (Eq. 4): every block whose fp32 score is
    strictly greater than the fp32 threshold, plus the forced blocks.
    NaN scores are never selected (they compare false)."""
    n = i + 1
    s = np.asarray(score_row[:n], dtype=np.float32)
    forced = set()
    if flags & FORCE_DIAG:
        forced.add(i)
    if flags & FORCE_SINK:
        forced.add(0)
    if mode == MODE_THRESHOLD:
        kept = set(np.flatnonzero(s > np.float32(threshold)).tolist())
        return sorted(kept | forced)
    ki = keep_count(n, mode, keep_num, keep_den, k)
    is_cand = ~np.isnan(s)
    is_cand[list(forced)] = False
    cands = np.flatnonzero(is_cand)
    # sort candidates by (score descending, index ascending): lexsort's last key is the primary one
    order = cands[np.lexsort((cands, -s[cands].astype(np.float64)))]
    take = max(ki - len(forced), 0)
    return sorted(forced | set(order[:take].tolist()))


def block_mask(scores: list, mode: int, *, keep_num=1, keep_den=1, k=0, threshold=0.0, flags=FORCE_DIAG, dense_tail=0):
    """All rows of all sequences -> CSR index lists (row_ptr int64 [R+1], col_idx int32 [nnz]).
    `scores` is the per-sequence list of [Hq, nb, nb] fp32 arrays.  dense_tail: the last `dense_tail` query blocks
    of every sequence keep all their causal blocks (Sec. 4: sparsity is applied to the context, not to the question
    that ends the prompt)."""
    row_ptr = [0]
    cols = []
    for S in scores:
        Hq, nb, _ = S.shape
        for h in range(Hq):
            for i in range(nb):
                if i >= nb - dense_tail:
                    lst = list(range(i + 1))
                else:
                    lst = select_row(S[h, i], i, mode, keep_num=keep_num, keep_den=keep_den, k=k,
                                     threshold=threshold, flags=flags)
                cols.extend(lst)
                row_ptr.append(len(cols))
    return np.asarray(row_ptr, dtype=np.int64), np.asarray(cols, dtype=np.int32)


def full_causal_lists(cu_seqlens, B: int, num_q_heads: int):
    """Lists that keep every causal block (the dense mask)."""
    row_ptr, cols = [0], []
    for nb in blocks_per_sequence(cu_seqlens, B):
        for _h in range(num_q_heads):
            for i in range(int(nb)):
                cols.extend(range(i + 1))
                row_ptr.append(len(cols))
    return np.asarray(row_ptr, dtype=np.int64), np.asarray(cols, dtype=np.int32)


# --------------------------------------------------------------------------- block-sparse attention (Sec. 2, Sec. 3.3)
def sparse_attention(q_bits, k_bits, v_bits, cu_seqlens, row_ptr, col_idx, num_q_heads: int,
                     num_kv_heads: int, B: int, scale: float, rows=None):
    """softmax(Q K^T * scale) V per query token, the softmax taken over the keys
    that (a) lie in a key block listed for the token's (sequence, head, query
    block) row, (b) are not later than the query (causal) and (c) exist
    (sequence length).  fp64 throughout; outputs are not rounded.

    rows: optional iterable of row ids to compute (others stay NaN).
    Returns o [T, Hq, d] and lse [Hq, T] (log of the softmax denominator,
    scaled logits, natural log).  A token with no key gets o = 0, lse = -inf."""
    T, Hq, d = q_bits.shape
    G = num_q_heads // num_kv_heads
    o = np.full((T, Hq, d), np.nan, dtype=np.float64)
    lse = np.full((Hq, T), np.nan, dtype=np.float64)
    nbs = blocks_per_sequence(cu_seqlens, B)
    base = row_base(cu_seqlens, B, num_q_heads)
    wanted = None if rows is None else set(int(r) for r in rows)
    for b, nb in enumerate(nbs):
        s0, s1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(num_q_heads):
            g = h // G
            for i in range(int(nb)):
                r = int(base[b]) + h * int(nb) + i
                if wanted is not None and r not in wanted:
                    continue
                tq = np.arange(s0 + i * B, min(s0 + (i + 1) * B, s1))
                blocks = col_idx[int(row_ptr[r]):int(row_ptr[r + 1])]
                tk = np.concatenate([np.arange(s0 + int(j) * B, min(s0 + (int(j) + 1) * B, s1)) for j in blocks]) \
                    if len(blocks) else np.zeros(0, dtype=np.int64)
                Q = bf16_bits_to_f64(q_bits[tq, h, :])
                if len(tk) == 0:
                    o[tq, h, :] = 0.0
                    lse[h, tq] = -np.inf
                    continue
                K = bf16_bits_to_f64(k_bits[tk, g, :])
                V = bf16_bits_to_f64(v_bits[tk, g, :])
                S = (Q @ K.T) * scale
                S[tk[None, :] > tq[:, None]] = -np.inf
                m = S.max(axis=1, keepdims=True)
                dead = ~np.isfinite(m[:, 0])
                m[dead] = 0.0
                P = np.exp(S - m)
                l = P.sum(axis=1, keepdims=True)
                with np.errstate(divide="ignore", invalid="ignore"):
                    out = (P @ V) / l
                    ls = m[:, 0] + np.log(l[:, 0])
                out[dead] = 0.0
                ls[dead] = -np.inf
                o[tq, h, :] = out
                lse[h, tq] = ls
    return o, lse


# --------------------------------------------------------------------------- chunked prefill
def chunk_offsets(cu_seqlens_q, cu_seqlens_k, B: int) -> np.ndarray:
    """Per sequence, the block position of the chunk's first query block: the S_q queries are the last S_q positions
    of the S_k keys and the chunk starts on a block boundary (a reading: the paper evaluates whole prompts; serving
    stacks split them into block-aligned chunks)."""
    sq = np.diff(np.asarray(cu_seqlens_q, dtype=np.int64))
    sk = np.diff(np.asarray(cu_seqlens_k, dtype=np.int64))
    if np.any(sq > sk) or np.any(((sk - sq) % B != 0) & (sq > 0)):
        raise ValueError("a chunk must end its sequence and start on a block boundary")
    return np.where(sq > 0, (sk - sq) // B, (sk + B - 1) // B)     # a sequence without queries: past its last block


def gate_scores_chunk(q_bits, k_bits, wq, wk, cu_seqlens_q, cu_seqlens_k, B: int, pool_q: int = POOL_AVG,
                      pool_k: int = POOL_AVG, rope_theta: float = 0.0) -> list:
    """Eq. 1 for a chunk: q_bits holds only the chunk's tokens.  Returns per sequence the fp32 array
    [Hq, nbq, nbk]; row r is query block off + r of the sequence and its softmax runs over key blocks j <= off + r."""
    off = chunk_offsets(cu_seqlens_q, cu_seqlens_k, B)
    pq = pool_compose(q_bits, cu_seqlens_q, B, pool_q)
    pk = pool_compose(k_bits, cu_seqlens_k, B, pool_k)
    out = []
    for b in range(len(pq)):
        gq, gk = project(pq[b], wq), project(pk[b], wk)
        if rope_theta > 0.0:
            gq, gk = block_rope(gq, rope_theta, B, first=int(off[b])), block_rope(gk, rope_theta, B)
        Hq, nbq, dg = gq.shape
        G = Hq // gk.shape[0]
        L = np.empty((Hq, nbq, gk.shape[1]), dtype=np.float64)
        for h in range(Hq):
            L[h] = gq[h] @ gk[h // G].T / math.sqrt(dg)
        out.append(causal_softmax_rows(L, first=int(off[b])).astype(np.float32))
    return out


def block_mask_chunk(scores: list, mode: int, *, keep_num=1, keep_den=1, k=0, threshold=0.0, flags=FORCE_DIAG,
                     dense_tail=0):
    """Lists for a chunk from its [Hq, nbq, nbk] score arrays, in the row numbering of the whole sequences: the CSR
    structure has Hq * nbk rows per sequence and the rows of the blocks before the chunk are empty."""
    row_ptr, cols = [0], []
    for S in scores:
        Hq, nbq, nbk = S.shape
        off = nbk - nbq
        for h in range(Hq):
            for i in range(nbk):
                if i >= off and i >= nbk - dense_tail:
                    cols.extend(range(i + 1))
                elif i >= off:
                    cols.extend(select_row(S[h, i - off], i, mode, keep_num=keep_num, keep_den=keep_den, k=k,
                                           threshold=threshold, flags=flags))
                row_ptr.append(len(cols))
    return np.asarray(row_ptr, dtype=np.int64), np.asarray(cols, dtype=np.int32)


def sparse_attention_chunk(q_bits, k_bits, v_bits, cu_seqlens_q, cu_seqlens_k, row_ptr, col_idx, num_q_heads: int,
                           num_kv_heads: int, B: int, scale: float):
    """Block-sparse attention of a chunk: query token u of sequence b (0 <= u < S_q) sits at position S_k - S_q + u and
    sees the keys at positions <= its own inside the key blocks listed for row (b, head, its block), rows numbered
    over the whole sequence.  Returns o [Tq, Hq, d] and lse [Hq, Tq]; a token with no key gets o = 0, lse = -inf."""
    Tq, Hq, d = q_bits.shape
    G = num_q_heads // num_kv_heads
    o = np.zeros((Tq, Hq, d), dtype=np.float64)
    lse = np.full((Hq, Tq), -np.inf, dtype=np.float64)
    base = row_base(cu_seqlens_k, B, num_q_heads)
    for b in range(len(cu_seqlens_k) - 1):
        k0, k1 = int(cu_seqlens_k[b]), int(cu_seqlens_k[b + 1])
        q0, q1 = int(cu_seqlens_q[b]), int(cu_seqlens_q[b + 1])
        Sk, Sq = k1 - k0, q1 - q0
        nbk = (Sk + B - 1) // B
        for h in range(num_q_heads):
            Kh = bf16_bits_to_f64(k_bits[k0:k1, h // G, :])
            Vh = bf16_bits_to_f64(v_bits[k0:k1, h // G, :])
            for u in range(Sq):
                pos = Sk - Sq + u
                r = int(base[b]) + h * nbk + pos // B
                keys = [t for j in col_idx[int(row_ptr[r]):int(row_ptr[r + 1])]
                        for t in range(int(j) * B, min((int(j) + 1) * B, Sk)) if t <= pos]
                if not keys:
                    continue
                qv = bf16_bits_to_f64(q_bits[q0 + u, h, :])
                sc = (Kh[keys] @ qv) * scale
                m = sc.max()
                p = np.exp(sc - m)
                o[q0 + u, h, :] = (p @ Vh[keys]) / p.sum()
                lse[h, q0 + u] = m + math.log(p.sum())
    return o, lse


# --------------------------------------------------------------------------- distillation target (Sec. 3.2, Eq. 2; appendix)
def maxpool_attention_map(q_bits, k_bits, cu_seqlens, num_q_heads: int, num_kv_heads: int, B: int, scale: float) -> list:
    """gt = MaxPool2D(softmax(Q K^T / sqrt(d))) of Eq. 2 with a BxB window and
    stride B on the dense causal attention map of every head.  Per sequence
    [Hq, nb, nb] fp64, zero above the diagonal."""
    G = num_q_heads // num_kv_heads
    out = []
    for b in range(len(cu_seqlens) - 1):
        s0, s1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        S_len = s1 - s0
        nb = (S_len + B - 1) // B
        gt = np.zeros((num_q_heads, nb, nb), dtype=np.float64)
        pos = np.arange(S_len)
        for h in range(num_q_heads):
            Q = bf16_bits_to_f64(q_bits[s0:s1, h, :])
            K = bf16_bits_to_f64(k_bits[s0:s1, h // G, :])
            A = (Q @ K.T) * scale
            A[pos[None, :] > pos[:, None]] = -np.inf
            A = np.exp(A - A.max(axis=1, keepdims=True))
            A /= A.sum(axis=1, keepdims=True)
            for i in range(nb):
                for j in range(i + 1):
                    gt[h, i, j] = A[i * B:(i + 1) * B, j * B:(j + 1) * B].max()
        out.append(gt)
    return out


def maxpool_listed_blocks(q_bits, k_bits, cu_seqlens, row_ptr, col_idx, num_q_heads: int, num_kv_heads: int, B: int,
                          scale: float, rows=None) -> np.ndarray:
    """The 2D max-pooling of Eq. 2 taken on the attention the block lists define: for the row (sequence, head, query
    block i) and each listed key block j, the largest softmax probability a_ts = exp(r_ts - m_t) / l_t (appendix) over
    the B x B tile, the softmax of query t running over the keys of the row's listed blocks that are not later than t.
    With full causal lists this is entry [h, i, j] of `maxpool_attention_map`.  Returns one fp64 value per entry of
    col_idx (NaN for rows not in `rows`); a tile in which no (query, key) pair is causal gives 0."""
    G = num_q_heads // num_kv_heads
    out = np.full(len(col_idx), np.nan, dtype=np.float64)
    nbs = blocks_per_sequence(cu_seqlens, B)
    base = row_base(cu_seqlens, B, num_q_heads)
    wanted = None if rows is None else set(int(r) for r in rows)
    for b, nb in enumerate(nbs):
        s0, s1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(num_q_heads):
            g = h // G
            for i in range(int(nb)):
                r = int(base[b]) + h * int(nb) + i
                if wanted is not None and r not in wanted:
                    continue
                l0, l1 = int(row_ptr[r]), int(row_ptr[r + 1])
                if l1 == l0:
                    continue
                tq = np.arange(s0 + i * B, min(s0 + (i + 1) * B, s1))
                Q = bf16_bits_to_f64(q_bits[tq, h, :])
                tiles = []
                for j in col_idx[l0:l1]:
                    tk = np.arange(s0 + int(j) * B, min(s0 + (int(j) + 1) * B, s1))
                    S = (Q @ bf16_bits_to_f64(k_bits[tk, g, :]).T) * scale
                    S[tk[None, :] > tq[:, None]] = -np.inf
                    tiles.append(S)
                allS = np.concatenate(tiles, axis=1)
                m = allS.max(axis=1, keepdims=True)
                m[~np.isfinite(m)] = 0.0
                l = np.exp(allS - m).sum(axis=1, keepdims=True)
                for p_, S in enumerate(tiles):
                    with np.errstate(divide="ignore", invalid="ignore"):
                        A = np.exp(S - m) / l
                    A[~np.isfinite(A)] = 0.0
                    out[l0 + p_] = A.max() if A.size else 0.0
    return out

