"""World-size-2 check of the multi-GPU partition (host logic) on CPU with the gloo backend: each rank runs the path
on its KV-head shard (here with the oracle standing in for the GPU library), the outputs are gathered, and the result
must equal the unsharded run exactly.  Rendezvous on 127.0.0.1."""
import math
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import seer_oracle as O
from paper_2410_13276_b200 import sharding, workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_path(q, k, v, wq, wk, cu, hq, hkv):
    scores = O.gate_scores(q, k, wq, wk, cu, 64)
    rp, col = O.block_mask(scores, O.MODE_TOPK_RATIO, keep_num=1, keep_den=2, flags=O.FORCE_DIAG)
    o, lse = O.sparse_attention(q, k, v, cu, rp, col, hq, hkv, 64, 1 / math.sqrt(128))
    return o, lse, int(rp[-1])


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.make_small(77, [200, 130], 6, 3)
        sh = sharding.kv_head_shard(6, 3, world, rank)
        q, k, v, wq, wk = sharding.slice_inputs(sh, w.q, w.k, w.v, w.wq, w.wk)
        o, lse, nnz = _run_path(np.ascontiguousarray(q), np.ascontiguousarray(k), np.ascontiguousarray(v), wq, wk,
                                w.cu_seqlens, sh.num_q_heads, sh.num_kv_heads)
        gathered = [None] * world
        dist.all_gather_object(gathered, (sh.q_lo, o, lse, nnz))
        if rank == 0:
            gathered.sort(key=lambda t: t[0])
            o_all = sharding.concat_heads([g[1] for g in gathered], axis=1)
            lse_all = sharding.concat_heads([g[2] for g in gathered], axis=0)
            o_ref, lse_ref, nnz_ref = _run_path(w.q, w.k, w.v, w.wq, w.wk, w.cu_seqlens, 6, 3)
            out.put((bool(np.array_equal(o_all, o_ref)), bool(np.array_equal(lse_all, lse_ref)),
                     sum(g[3] for g in gathered) == nnz_ref))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_kv_head_shards_reproduce_the_unsharded_layer_gloo_world2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert out.get(timeout=5) == (True, True, True)


def test_shard_ranges_partition_the_heads():
    for hq, hkv in ((32, 8), (40, 8), (4, 1), (6, 3)):
        for world in (1, 2, 3, 4, 8, 16):
            shards = [sharding.kv_head_shard(hq, hkv, world, r) for r in range(world)]
            assert shards[0].kv_lo == 0 and shards[-1].kv_hi == hkv
            assert all(a.kv_hi == b.kv_lo for a, b in zip(shards, shards[1:]))
            assert sum(s.num_q_heads for s in shards) == hq
            sizes = [s.num_kv_heads for s in shards]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.kv_head_shard(6, 4, 2, 0)
