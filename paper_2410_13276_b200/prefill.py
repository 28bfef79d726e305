"""Device-buffer bookkeeping around the three C-ABI calls.

`Prefill` owns the torch tensors that hold one layer's inputs, intermediates
and outputs on a GPU and issues seer_gate_scores -> seer_block_mask ->
seer_sparse_attn on them.  It computes nothing itself.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B


def _bf16_from_bits(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


class Prefill:
    def __init__(self, cu_seqlens, num_q_heads: int, num_kv_heads: int, *, device: int = 0,
                 ctx: Optional[B.Context] = None, softmax_scale: float = 0.0, col_capacity: Optional[int] = None,
                 want_lse: bool = True, block: int = 64, cu_seqlens_q=None):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU path)")
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.ctx = ctx or B.Context(device)
        self.cu = np.asarray(cu_seqlens, dtype=np.int32)
        self.hq, self.hkv = num_q_heads, num_kv_heads
        self.block = block
        # chunked prefill: q / o / lse hold the last cu_q[b+1] - cu_q[b] positions of each sequence only
        self.cu_q = None if cu_seqlens_q is None else np.asarray(cu_seqlens_q, dtype=np.int32)
        self.shape = B.make_shape(self.cu, num_q_heads, num_kv_heads, softmax_scale=softmax_scale, block=block,
                                  cu_seqlens_q=self.cu_q)
        # the attention kernels tile by 64 tokens: 128-token lists are expanded for them (seer_expand_block_lists)
        self.attn_shape = self.shape if block == 64 else B.make_shape(self.cu, num_q_heads, num_kv_heads,
                                                                      softmax_scale=softmax_scale, block=64,
                                                                      cu_seqlens_q=self.cu_q)
        self.T = int(self.cu[-1])
        self.Tq = self.T if self.cu_q is None else int(self.cu_q[-1])
        self.rows = B.seer_mask_rows(self.shape)
        self.causal_blocks = B.seer_causal_blocks(self.shape)
        if self.rows < 0:
            raise B.SeerError(2, "shape")
        d = self.device
        self.ws = torch.empty(max(B.seer_workspace_bytes(self.shape), 256), dtype=torch.uint8, device=d)
        self.scores = torch.empty(max(B.seer_scores_elems(self.shape), 1), dtype=torch.float32, device=d)
        self.row_ptr = torch.zeros(self.rows + 1, dtype=torch.int32, device=d)
        cap = self.causal_blocks if col_capacity is None else col_capacity
        self.col_idx = torch.empty(max(cap, 1), dtype=torch.int32, device=d)
        self.col_capacity = cap
        self.nnz = torch.zeros(1, dtype=torch.int64, device=d)
        if block != 64:
            self.row_ptr64 = torch.zeros(B.seer_mask_rows(self.attn_shape) + 1, dtype=torch.int32, device=d)
            self.col_idx64 = torch.empty(max(4 * cap, 1), dtype=torch.int32, device=d)
            self.nnz64 = torch.zeros(1, dtype=torch.int64, device=d)
        self.q = self.k = self.v = self.wq = self.wk = None
        self.o = torch.empty((self.Tq, num_q_heads, 128), dtype=torch.bfloat16, device=d)
        self.lse = torch.empty((num_q_heads, self.Tq), dtype=torch.float32, device=d) if want_lse else None

    # ---- uploads (plain copies)
    def set_inputs(self, q_bits, k_bits, v_bits, wq=None, wk=None):
        self.q = _bf16_from_bits(q_bits, self.device)
        self.k = _bf16_from_bits(k_bits, self.device)
        self.v = _bf16_from_bits(v_bits, self.device)
        if wq is not None:
            self.wq = torch.from_numpy(np.ascontiguousarray(wq, dtype=np.float32)).to(self.device)
            self.wk = torch.from_numpy(np.ascontiguousarray(wk, dtype=np.float32)).to(self.device)

    def set_scores(self, flat: np.ndarray):
        self.scores[: flat.size].copy_(torch.from_numpy(np.ascontiguousarray(flat, dtype=np.float32)))

    def set_lists(self, row_ptr: np.ndarray, col_idx: np.ndarray):
        self.row_ptr.copy_(torch.from_numpy(row_ptr.astype(np.int32)))
        if col_idx.size > self.col_idx.numel():
            self.col_idx = torch.empty(col_idx.size, dtype=torch.int32, device=self.device)
        self.col_idx[: col_idx.size].copy_(torch.from_numpy(col_idx.astype(np.int32)))

    # ---- the three calls
    def gate(self, stream=None):
        B.seer_gate_scores(self.ctx, self.shape, self.q, self.k, self.wq, self.wk, self.scores, self.ws, stream)

    def gate_project(self, stream=None):
        """Pooling and projection only (the first kernel of the gate)."""
        B.seer_gate_project(self.ctx, self.shape, self.q, self.k, self.wq, self.wk, self.ws, stream)

    def gate_ex(self, options: B.seer_gate_options, wq, wk, stream=None):
        """Gate with composed pooling and / or block-level RoPE (Sec. 3.1); wq, wk are device tensors
        [heads, n * 128, 128] matching the pooling subsets in `options`."""
        B.seer_gate_scores_ex(self.ctx, self.shape, options, self.q, self.k, wq, wk, self.scores, self.ws, stream)

    def gate_mask(self, params: B.seer_mask_params, *, band_bytes: int = 128 << 20, options=None, wq=None, wk=None,
                  stream=None):
        """Gate and mask in one call, the scores held one band at a time in a scratch of `band_bytes` (never the whole
        score matrix); fills row_ptr / col_idx / nnz exactly as gate() + mask() do."""
        need = B.seer_gate_mask_workspace_bytes(self.shape, band_bytes)
        if getattr(self, "ws_fused", None) is None or self.ws_fused.numel() != need:
            self.ws_fused = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
        B.seer_gate_block_mask(self.ctx, self.shape, options, self.q, self.k, self.wq if wq is None else wq,
                               self.wk if wk is None else wk, params, self.row_ptr, self.col_idx, self.col_capacity,
                               self.nnz, self.ws_fused, stream)
        if self.block != 64:
            self.expand(stream)

    def block_max(self, stream=None):
        """Max-pooled attention map on the listed blocks (Eq. 2) from the lse of the last `attn` call; returns the
        device tensor [col_capacity] fp32 aligned with col_idx."""
        if self.lse is None:
            raise ValueError("block_max needs the lse output: construct with want_lse=True")
        if getattr(self, "bmax", None) is None or self.bmax.numel() < self.col_idx.numel():
            self.bmax = torch.empty(max(self.col_idx.numel(), 1), dtype=torch.float32, device=self.device)
        B.seer_attn_block_max(self.ctx, self.shape, self.q, self.k, self.row_ptr, self.col_idx, self.lse, self.bmax,
                              stream)
        return self.bmax

    def mask(self, params: B.seer_mask_params, stream=None):
        B.seer_block_mask(self.ctx, self.shape, self.scores, params, self.row_ptr, self.col_idx, self.col_capacity,
                          self.nnz, None, stream)
        if self.block != 64:
            self.expand(stream)

    def expand(self, stream=None):
        """128-token lists -> the 64-token lists the attention takes."""
        B.seer_expand_block_lists(self.ctx, self.shape, self.row_ptr, self.col_idx, self.row_ptr64, self.col_idx64, None,
                                  self.nnz64, stream)

    def attn(self, stream=None, dynamic=True):
        """Block-sparse attention over the lists.  With `dynamic` the call gets the workspace, whose first word the
        tcgen05 kernel uses as the counter its streams draw their work items from; without, the items are dealt
        statically (the results are the same bit for bit)."""
        rp, col = (self.row_ptr, self.col_idx) if self.block == 64 else (self.row_ptr64, self.col_idx64)
        B.seer_sparse_attn(self.ctx, self.attn_shape, self.q, self.k, self.v, rp, col, self.o, self.lse,
                           self.ws if dynamic else None, stream)

    def run(self, params: B.seer_mask_params, stream=None):
        self.gate(stream)
        self.mask(params, stream)
        self.attn(stream)

    # ---- downloads
    def scores_host(self) -> np.ndarray:
        return self.scores[: B.seer_scores_elems(self.shape)].cpu().numpy()

    def lists64_host(self):
        """The expanded 64-token lists of a 128-token problem."""
        rp = self.row_ptr64.cpu().numpy().astype(np.int64)
        n = min(int(rp[-1]), self.col_idx64.numel())
        return rp, self.col_idx64[:n].cpu().numpy()

    def lists_host(self):
        rp = self.row_ptr.cpu().numpy().astype(np.int64)
        n = min(int(rp[-1]), self.col_idx.numel())
        return rp, self.col_idx[:n].cpu().numpy()

    def o_host(self) -> np.ndarray:
        """bf16 output widened exactly to fp32 on the host."""
        bits = self.o.view(torch.int16).cpu().numpy().view(np.uint16)
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)

    def lse_host(self) -> np.ndarray:
        return self.lse.cpu().numpy()

    def status(self) -> int:
        return B.seer_poll_device_status(self.ctx)
