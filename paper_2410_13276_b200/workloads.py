"""Seeded synthetic inputs for the SeerAttention prefill hot path.

This module only *draws data*: Q/K/V tensors (as bf16 bit patterns), gate
weights, sequence lengths and the mask parameters of each named workload.
It holds none of the method's arithmetic (no pooling, no softmax, no
selection, no attention), so both the CUDA path and the CPU oracle may be
fed from it without sharing any of the code under test.

The workloads stand in for the paper's kernel-latency experiment (Sec. 4.2.1:
Llama-3.1-8B-Instruct head shapes, 8k-128k tokens, sparsity statistics from
PG19).  Neither the model, the trained gate nor the dataset is available, so
the tensors are random with the same shapes, and the structured workload
plants the mask patterns the paper shows in its visualisation of learned
gates (sink column, vertical stripes, local band, diffuse heads).

Layout: q [T, Hq, d], k/v [T, Hkv, d], row-major, T = total packed tokens of
all sequences, `cu_seqlens` the cumulative offsets.  bf16 values are carried
as uint16 bit patterns (numpy has no bf16).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

BLOCK = 64          # gate block = attention tile (Sec. 4: fixed at 64)
HEAD_DIM = 128
GATE_DIM = 128

MODE_TOPK_RATIO = 0
MODE_TOPK_COUNT = 1
MODE_THRESHOLD = 2
FORCE_DIAG = 1
FORCE_SINK = 2


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rnd = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bits to fp32 (data plumbing only)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class MaskSpec:
    mode: int
    keep_num: int = 1
    keep_den: int = 1
    k: int = 0
    threshold: Optional[float] = None     # None: tuned from oracle scores to `target_sparsity`
    flags: int = FORCE_DIAG
    target_sparsity: Optional[float] = None


@dataclass
class Workload:
    name: str
    cu_seqlens: np.ndarray                # int32 [batch+1]
    num_q_heads: int
    num_kv_heads: int
    q: np.ndarray                         # uint16 [T, Hq, d]
    k: np.ndarray                         # uint16 [T, Hkv, d]
    v: np.ndarray                         # uint16 [T, Hkv, d]
    wq: np.ndarray                        # float32 [Hq, d, dg]
    wk: np.ndarray                        # float32 [Hkv, d, dg]
    masks: list = field(default_factory=list)   # list[MaskSpec]
    block: int = BLOCK
    head_dim: int = HEAD_DIM
    gate_dim: int = GATE_DIM

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def seqlens(self):
        return np.diff(self.cu_seqlens).astype(np.int64)

    @property
    def num_blocks(self):
        return (self.seqlens + self.block - 1) // self.block

    @property
    def softmax_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))


def _seed(config: int, stream: int, twin: bool) -> int:
    # streams: 0 Q, 1 K, 2 V, 3 Wq, 4 Wk, 5 structure.  Config 1 draws Q from the literal seed 0.
    if config == 1 and stream == 0 and not twin:
        return 0
    return 1000 * config + (100 if twin else 0) + stream


def _normal(seed: int, shape) -> np.ndarray:
    return np.random.default_rng(seed).standard_normal(shape, dtype=np.float32)


def _rope_inplace(x: np.ndarray, cu_seqlens: np.ndarray, base: float) -> None:
    """Standard rotary embedding on x [T, H, d] (fp32, in place), half-split
    pairing (c, c + d/2), positions local to each sequence."""
    T, H, d = x.shape
    half = d // 2
    inv = base ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    for b in range(len(cu_seqlens) - 1):
        s0, s1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        step = 8192
        for t0 in range(s0, s1, step):
            t1 = min(t0 + step, s1)
            ang = np.arange(t0 - s0, t1 - s0, dtype=np.float64)[:, None] * inv[None, :]
            c = np.cos(ang).astype(np.float32)[:, None, :]
            s = np.sin(ang).astype(np.float32)[:, None, :]
            lo = x[t0:t1, :, :half].copy()
            hi = x[t0:t1, :, half:]
            x[t0:t1, :, :half] = lo * c - hi * s
            x[t0:t1, :, half:] = hi * c + lo * s


def _gate_weights(seed: int, heads: int, d: int, dg: int) -> np.ndarray:
    return (_normal(seed, (heads, d, dg)) * np.float32(1.0 / np.sqrt(128.0))).astype(np.float32)


def make_gate_weights(seed: int, heads: int, in_dim: int, dg: int = 128) -> np.ndarray:
    """Seeded gate matrices [heads, in_dim, dg] (fp32, N(0, std 1/sqrt(128))) for the gate variants whose input is a
    concatenation of several pooled tensors (in_dim = number of pooling methods x head_dim)."""
    return _gate_weights(seed, heads, in_dim, dg)


def _random_layer(config, twin, seqlens, hq, hkv, rope_base=None):
    cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int32)
    T = int(cu[-1])
    q = _normal(_seed(config, 0, twin), (T, hq, HEAD_DIM))
    k = _normal(_seed(config, 1, twin), (T, hkv, HEAD_DIM))
    v = _normal(_seed(config, 2, twin), (T, hkv, HEAD_DIM))
    if rope_base is not None:
        _rope_inplace(q, cu, rope_base)
        _rope_inplace(k, cu, rope_base)
    wq = _gate_weights(_seed(config, 3, twin), hq, HEAD_DIM, GATE_DIM)
    wk = _gate_weights(_seed(config, 4, twin), hkv, HEAD_DIM, GATE_DIM)
    return cu, f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v), wq, wk


def _structured_layer(config, twin, S, hq, hkv):
    """Planted structure: per KV head a sink key at token 0 (norm x8), 16
    vertical-stripe key blocks sharing a direction c_g with the queries, and a
    slowly varying latent z_g(t) (correlation length 3 blocks) that makes
    nearby tokens attend to each other (local band).  Gate weights are tied
    (Wq[h] = Wk[h // G]) so that W^T W ~ I and the planted directions survive
    the projection."""
    from scipy.signal import lfilter

    G = hq // hkv
    d = HEAD_DIM
    cu = np.array([0, S], dtype=np.int32)
    nb = (S + BLOCK - 1) // BLOCK
    rs = np.random.default_rng(_seed(config, 5, twin))
    q = _normal(_seed(config, 0, twin), (S, hq, d))
    k = _normal(_seed(config, 1, twin), (S, hkv, d))
    v = _normal(_seed(config, 2, twin), (S, hkv, d))
    rho = float(np.exp(-1.0 / (3.0 * BLOCK)))
    pairs = [(8, 0), (6, .25), (5, .5), (4, .25), (3, .5), (3, .25), (2, .5), (4, 0)]
    n_stripes = min(16, max(nb - 1, 0))
    for g in range(hkv):
        c = rs.standard_normal(d)
        c /= np.linalg.norm(c)
        u = rs.standard_normal(d)
        u -= c * (u @ c)
        u /= np.linalg.norm(u)
        eps = rs.standard_normal((S, d))
        eps[0] /= np.sqrt(1.0 - rho * rho)           # stationary start
        z = lfilter([np.sqrt(1.0 - rho * rho)], [1.0, -rho], eps, axis=0).astype(np.float32)
        stripes = rs.choice(np.arange(1, nb), size=n_stripes, replace=False) if n_stripes else np.zeros(0, int)
        in_stripe = np.zeros(nb, dtype=bool)
        in_stripe[stripes] = True
        tok_stripe = np.repeat(in_stripe, BLOCK)[:S]
        k[:, g, :] += z
        k[tok_stripe, g, :] += (8.0 * c).astype(np.float32)
        k[0, g, :] = (8.0 * np.sqrt(128.0) * (0.08 * c + np.sqrt(1 - 0.08 ** 2) * u)).astype(np.float32)
        for hh in range(G):
            h = g * G + hh
            alpha, gamma = pairs[h % 8]
            if h % 16 == 7:
                alpha, gamma = 0.0, 0.0                # diffuse head
            q[:, h, :] += (alpha * c).astype(np.float32)[None, :] + np.float32(gamma) * z
    wk = _gate_weights(_seed(config, 4, twin), hkv, d, GATE_DIM)
    wq = np.repeat(wk, G, axis=0).copy()
    return cu, f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v), wq, wk


# name -> (config id, twin?)   "cN" = full size of benchmark configuration N, "cNs" = its reduced twin (~4096 tokens)
WORKLOADS = ("c1", "c2", "c3", "c4", "c5", "c2s", "c3s", "c4s", "c5s")

C3_RATIOS = ((1, 2), (1, 4), (1, 10), (1, 20))


def make_workload(name: str, seq: Optional[int] = None) -> Workload:
    """`seq` overrides the sequence length of the single-sequence workloads (c2, c3, c5) for profiling runs."""
    twin = name.endswith("s")
    config = int(name[1])
    if config == 1:
        cu, q, k, v, wq, wk = _random_layer(1, False, [2048], 4, 1)
        masks = [MaskSpec(MODE_TOPK_RATIO, 1, 2, flags=FORCE_DIAG)]
        hq, hkv = 4, 1
    elif config == 2:
        S = seq or (4096 if twin else 32768)
        hq, hkv = 32, 8
        cu, q, k, v, wq, wk = _random_layer(2, twin, [S], hq, hkv, rope_base=500000.0)
        masks = [MaskSpec(MODE_THRESHOLD, flags=FORCE_DIAG, target_sparsity=0.90)]
    elif config == 3:
        S = seq or (4096 if twin else 131072)
        hq, hkv = 32, 8
        cu, q, k, v, wq, wk = _random_layer(3, twin, [S], hq, hkv, rope_base=500000.0)
        masks = [MaskSpec(MODE_TOPK_RATIO, n, dn, flags=FORCE_DIAG | FORCE_SINK) for n, dn in C3_RATIOS]
    elif config == 4:
        lens = [512, 1024, 2048, 4096] if twin else [8192, 16384, 32768, 65536]
        hq, hkv = 40, 8
        cu, q, k, v, wq, wk = _random_layer(4, twin, lens, hq, hkv)
        masks = [MaskSpec(MODE_THRESHOLD, flags=FORCE_DIAG, target_sparsity=0.85)]
    elif config == 5:
        S = seq or (4096 if twin else 65536)
        hq, hkv = 32, 8
        cu, q, k, v, wq, wk = _structured_layer(5, twin, S, hq, hkv)
        masks = [MaskSpec(MODE_THRESHOLD, flags=FORCE_DIAG, target_sparsity=0.92)]
    else:
        raise ValueError(name)
    return Workload(name, cu, hq, hkv, q, k, v, wq, wk, masks)


def make_small(seed: int, seqlens, hq: int, hkv: int, *, block: int = BLOCK, head_dim: int = HEAD_DIM,
               gate_dim: int = GATE_DIM, w_std: float = 1.0 / np.sqrt(128.0), q_gain: float = 1.0) -> Workload:
    """Small random layer of arbitrary shape (ragged lengths, odd head counts)
    for parity and edge-case tests."""
    cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int32)
    T = int(cu[-1])
    r = np.random.default_rng(seed)
    q = (r.standard_normal((T, hq, head_dim), dtype=np.float32) * np.float32(q_gain))
    k = r.standard_normal((T, hkv, head_dim), dtype=np.float32)
    v = r.standard_normal((T, hkv, head_dim), dtype=np.float32)
    wq = (r.standard_normal((hq, head_dim, gate_dim), dtype=np.float32) * np.float32(w_std))
    wk = (r.standard_normal((hkv, head_dim, gate_dim), dtype=np.float32) * np.float32(w_std))
    return Workload(f"small{seed}", cu, hq, hkv, f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v),
                    wq, wk, [], block=block, head_dim=head_dim, gate_dim=gate_dim)


def sample_rows(cu_seqlens, num_q_heads: int, row_ptr: np.ndarray, seed: int, per_head_random: int = 8,
                heads=None, block: int = BLOCK) -> np.ndarray:
    """Stratified sample of mask rows for full-size checks: for every (sequence, head) the first two query
    blocks, the last, the row with the longest list, the row with the shortest, and a few seeded-random ones.
    Pure index selection; returns sorted unique row ids."""
    lens = np.diff(np.asarray(cu_seqlens, dtype=np.int64))
    nbs = (lens + block - 1) // block
    counts = np.diff(np.asarray(row_ptr, dtype=np.int64))
    rng = np.random.default_rng(seed)
    out = []
    base = 0
    for nb in nbs:
        nb = int(nb)
        for h in (range(num_q_heads) if heads is None else heads):
            if nb == 0:
                continue
            r0 = base + h * nb
            c = counts[r0:r0 + nb]
            picks = {0, min(1, nb - 1), nb - 1, int(np.argmax(c)), int(np.argmin(c))}
            picks |= set(rng.integers(0, nb, size=per_head_random).tolist())
            out.extend(r0 + i for i in picks)
        base += num_q_heads * nb
    return np.unique(np.asarray(out, dtype=np.int64))
