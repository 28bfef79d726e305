#!/usr/bin/env python
"""Benchmark of the SeerAttention prefill hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c3] [--keep 1/10]

One step = one pass of the whole hot path (seer_gate_scores -> seer_block_mask -> seer_sparse_attn) over one
synthetic layer.  Default workload: Llama-3-8B-shaped layer at 131072 tokens, TopK keeping 1/10 of the causal
blocks (90 % block sparsity), diagonal and sink forced.  Prints ONE JSON line on rank 0.

value  = kept-block attention FLOPs (4 * 64 * 64 * 128 per kept block) of all ranks / step time, inputs resident in HBM.
e2e    = same, through seer_prefill_host: pinned host buffers in, pinned host buffer out, copies inside the timed region.
roofline = the attention kernel alone (CUDA events around its launch) against the measured bf16 dense peak.
cpu_baseline = the fp64 CPU oracle on this machine's host cores: gate and mask in full, attention on a sample of rows of
               the same workload (measured, and extrapolated to all kept blocks).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FLOP_PER_BLOCK = 4 * 64 * 64 * 128
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch of the default command, and the capture it is from
TRAFFIC_C3_KEEP10 = (4.64e9, "ncu dram__bytes_read.sum + dram__bytes_write.sum, one launch of this command "
                                 "(summary: profiles/attn_tc_kernel_c3_seq131072_keep10_dram.md)")
METRIC = "sparse_prefill_attention_effective_tflops_128k_90pct_block_sparsity"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--keep", default="1/10", help="TopK ratio for the c3 workload")
    ap.add_argument("--seq", type=int, default=None, help="override the sequence length (profiling on a smaller case)")
    ap.add_argument("--attn-impl", type=int, default=0, choices=[0, 1, 2], help="0 tcgen05 kernel, 1 mma.sync kernel, 2 chosen per call from the shape")
    ap.add_argument("--all-workloads", action="store_true",
                    help="also time the other four workloads (and the other TopK ratios of c3) and add the table as `all_workloads`")
    ap.add_argument("--timeline", action="store_true",
                    help="one extra attention launch of the instrumented kernel; adds `timeline` (per role: clocks per tile in each step of its loop, CTA 0) to the line")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense-list run of the attention kernel")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the side measurements outside the timed region (gate variant, one-call gate + mask, "
                         "128-token blocks, chunked prefill, max-pooled map)")
    return ap.parse_args()


def pick_mask(w, args, need_threshold=True):
    from paper_2410_13276_b200 import workloads as W
    if w.name.startswith("c3"):
        num, den = (int(x) for x in args.keep.split("/"))
        return W.MaskSpec(W.MODE_TOPK_RATIO, num, den, flags=W.FORCE_DIAG | W.FORCE_SINK)
    spec = w.masks[0]
    if spec.mode == W.MODE_THRESHOLD and spec.threshold is None and need_threshold:
        with open(os.path.join(ROOT, "tests", "golden", "thresholds.json")) as f:
            spec.threshold = float.fromhex(json.load(f)[w.name]["threshold_hex"])
    return spec


L2_BYTES = 126 << 20


def input_bytes(w) -> int:
    return int(w.total_tokens) * (w.num_q_heads + 2 * w.num_kv_heads) * 256


def workload_desc(w, spec):
    flush = input_bytes(w) <= 2 * L2_BYTES
    return {"workload": f"{w.name}: 1 attention layer, batch {len(w.cu_seqlens) - 1}, tokens {w.total_tokens}, "
                        f"{w.num_q_heads} q heads / {w.num_kv_heads} kv heads, head_dim 128, block 64, causal",
            "mask": ({0: "topk_ratio", 1: "topk_count", 2: "threshold"}[spec.mode]
                     + (f" {spec.keep_num}/{spec.keep_den}" if spec.mode == 0 else
                        f" {spec.threshold!r} (target sparsity {spec.target_sparsity})" if spec.mode == 2 else f" {spec.k}")
                     + f", flags {spec.flags}"),
            "l2": ("L2 flushed before every timed step (a 256 MB buffer is overwritten; the step time is the sum of the "
                   "per-step event spans)" if flush else "inputs larger than L2 (no flush)")}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d["bf16_tflops"], d.get("bf16_tflops_sustained"), d["hbm_gbs"], "measured"
    return 1590.0, 1400.0, 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi polled every 100 ms from before the warm-up (its start-up alone takes a few hundred ms); stop()
    keeps the samples taken between mark_start() and mark_end().  When the timed region was too short for three
    samples, the caller keeps the same load running a little longer before mark_end() and the result says so."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.t0 = self.t1 = None
        self.extended = False
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                       "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def _rows(self):
        import datetime
        out = []
        try:
            lines = [l.strip() for l in open(self.f.name) if l.strip()]
        except OSError:
            return out
        for l in lines:
            r = l.split(", ")
            try:
                ts = datetime.datetime.strptime(r[0].strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
                out.append((ts, float(r[1]), float(r[2]), float(r[3]), [v.strip().lower() == "active" for v in r[4:8]]))
            except (ValueError, IndexError):
                continue
        return out

    def count_since_start(self) -> int:
        return sum(1 for r in self._rows() if self.t0 is not None and r[0] >= self.t0)

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = self._rows()
        os.unlink(self.f.name)
        t0 = self.t0 if self.t0 is not None else 0.0
        t1 = self.t1 if self.t1 is not None else time.time()
        rows = [r for r in rows if t0 <= r[0] <= t1 + 0.05]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in rows for n, v in zip(names, r[4]) if v})
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": float(max(r[2] for r in rows)),
                "reasons": reasons, "power_w_max": max(r[3] for r in rows), "samples": len(rows),
                "load_extended_for_sampling": self.extended}


def cpu_oracle_sample(w, spec, rp, col, budget_rows=None):
    """Times the oracle as it stands: gate and mask in full, attention on a sample of (head, query-block) rows.
    Returns the `cpu_baseline` object."""
    from oracle import seer_oracle as O
    from paper_2410_13276_b200 import workloads as W
    rows = W.sample_rows(w.cu_seqlens, w.num_q_heads, rp, seed=1234, per_head_random=56)   # ~1900 rows, about 10 s of CPU work
    if budget_rows:
        rows = rows[:: max(1, len(rows) // budget_rows)]
    blocks = int(sum(int(rp[r + 1] - rp[r]) for r in rows))
    t0 = time.perf_counter()
    O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp, col, w.num_q_heads, w.num_kv_heads, 64, w.softmax_scale, rows=rows)
    dt = time.perf_counter() - t0
    total = int(rp[-1])
    t0 = time.perf_counter()
    sc = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, 64)
    gate_s = time.perf_counter() - t0
    t0 = time.perf_counter()
    O.block_mask(sc, spec.mode, keep_num=spec.keep_num, keep_den=spec.keep_den, k=spec.k,
                 threshold=spec.threshold or 0.0, flags=spec.flags)
    mask_s = time.perf_counter() - t0
    del sc
    cores = len(os.sched_getaffinity(0))
    return {"value": blocks * FLOP_PER_BLOCK / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
            "sample": f"oracle attention on {len(rows)} sampled (head, query-block) rows = {blocks} of {total} kept blocks; "
                      "gate and mask oracle in full",
            "seconds": dt, "attn_ms_extrapolated": 1e3 * dt * total / max(blocks, 1), "gate_ms": 1e3 * gate_s,
            "mask_ms": 1e3 * mask_s}


TIMELINE_TAGS = {1: "loop", 2: "wait for an empty K / V buffer", 10: "before S^T", 11: "wait K_FULL", 12: "S^T MMAs + commits",
                 13: "before P V", 14: "wait V_FULL", 15: "wait P_FULL", 16: "P V MMAs + commits",
                 29: "item start (decode, first list entries)", 30: "tile loop of an item (all tiles)", 31: "epilogue",
                 32: "wait S_FULL", 33: "softmax pass (incl. first-tile references)", 34: "next list entries",
                 35: "wait PV_DONE", 36: "vote (the group's barrier)", 37: "(branch)", 38: "P^T stores", 39: "proxy fence, arrive P_FULL",
                 40: "rebase: wait next S^T + vote", 41: "rebase: TMEM reads", 42: "rebase: column maxima (shuffles)",
                 43: "rebase: new references", 44: "rebase: fix MMAs, rescale", 45: "rebase: wait FIXED", 46: "rebase: pass + stores", 47: "next S_FULL test (waits behind the P^T stores)"}
TIMELINE_ROLES = ["producer K+Q, stream 0", "issuer, stream 0", "producer V, stream 0", "issuer, stream 1",
                  "softmax group, stream 0", "softmax group, stream 1"]


def attention_timeline(p, B, torch):
    """One attention launch with the trace buffer set: the instrumented instantiation accumulates, for CTA 0, the
    clocks each role spends in each step of its loop (softmax groups: every tile; helpers: every eighth tile)."""
    buf = torch.zeros(7 * 8192, dtype=torch.int64, device="cuda")
    B.seer_set_trace_buffer(p.ctx, buf)
    try:
        p.attn(); torch.cuda.synchronize()
    finally:
        B.seer_set_trace_buffer(p.ctx, None)
    t = buf.cpu().numpy().astype(np.uint64)
    roles = {}
    for r, name in enumerate(TIMELINE_ROLES):
        a = t[r * 8192: r * 8192 + 96].reshape(48, 2).astype(np.int64)
        roles[name] = {TIMELINE_TAGS.get(tag, str(tag)): {"events": int(a[tag, 1]), "clocks_per_event": float(a[tag, 0]) / float(a[tag, 1])}
                       for tag in range(48) if a[tag, 1]}
    n = int((t[6 * 8192 + 256: 6 * 8192 + 512] != 0).sum())
    clk = t[6 * 8192 + 256: 6 * 8192 + 256 + n].astype(np.int64)
    return {"cta0_roles": roles, "cta_wall_clocks": {"ctas": n, "min": int(clk.min()), "median": int(np.median(clk)), "max": int(clk.max())}}


def time_workload(name, keep, args, local, B, W, Prefill, torch, burst):
    """gate / mask / attention / dense-list attention of one workload (3 warm-ups, 8 timed steps, medians)."""
    w = W.make_workload(name)
    a2 = argparse.Namespace(**vars(args)); a2.keep = keep or "1/10"
    spec = pick_mask(w, a2)
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, device=local, want_lse=False)
    B.seer_set_attn_impl(p.ctx, args.attn_impl)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(spec.mode, keep_num=spec.keep_num, keep_den=spec.keep_den, k=spec.k,
                                threshold=spec.threshold or 0.0, flags=spec.flags)
    stream = torch.cuda.current_stream()
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if input_bytes(w) <= 2 * L2_BYTES else None
    for _ in range(3):
        p.run(params)
    torch.cuda.synchronize()
    nnz = int(p.nnz.item())
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(8)]
    for s in range(8):
        if flush is not None:
            flush.fill_(s)
        ev[s][0].record(stream); p.gate(); ev[s][1].record(stream); p.mask(params); ev[s][2].record(stream); p.attn(); ev[s][3].record(stream)
    torch.cuda.synchronize()
    g, mk, at = (float(np.median([e[i].elapsed_time(e[i + 1]) for e in ev])) for i in range(3))
    dparams = B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=1, flags=B.SEER_FORCE_DIAG)
    p.mask(dparams); p.attn(); torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if flush is not None:
        flush.fill_(1)
    a.record(stream); p.attn(); b.record(stream); torch.cuda.synchronize()
    dense_ms = a.elapsed_time(b)
    dense_blocks = B.seer_causal_blocks(p.shape)
    status = p.status()
    out = {"workload": name, "mask": workload_desc(w, spec)["mask"], "tokens": int(w.total_tokens), "kept_blocks": nnz,
           "gate_ms": g, "mask_ms": mk, "attn_ms": at, "attn_tflops": nnz * FLOP_PER_BLOCK / (at * 1e-3) / 1e12,
           "attn_frac_of_burst_peak": nnz * FLOP_PER_BLOCK / (at * 1e-3) / 1e12 / burst,
           "dense_attn_ms": dense_ms, "dense_tflops": dense_blocks * FLOP_PER_BLOCK / (dense_ms * 1e-3) / 1e12,
           "speedup_over_dense": dense_ms / at, "l2_flushed": flush is not None, "device_status": status}
    p.ctx.close()
    return out


def seeded_lists_for_rows(w, spec, rows, seed=99):
    """Lists for a handful of rows without running the gate: TopK of seeded random scores under the workload's mask
    parameters (for a TopK-ratio mask the list lengths equal those of the real mask).  Oracle selection code only."""
    from oracle import seer_oracle as O
    from paper_2410_13276_b200 import workloads as W
    nbs = [int(n) for n in w.num_blocks]
    rng = np.random.default_rng(seed)
    counts = np.zeros(sum(nbs) * w.num_q_heads, dtype=np.int64)
    lists = {}
    for r in rows:
        off = 0
        for nb in nbs:
            if r < off + nb * w.num_q_heads:
                break
            off += nb * w.num_q_heads
        i = (int(r) - off) % nb
        s = rng.random(i + 1).astype(np.float32)
        if spec.mode == W.MODE_THRESHOLD:      # no tuned scores here: keep the workload's target fraction by TopK instead
            keep = max(1, round((1.0 - spec.target_sparsity) * 1000))
            lists[int(r)] = O.select_row(s, i, O.MODE_TOPK_RATIO, keep_num=keep, keep_den=1000, flags=spec.flags)
        else:
            lists[int(r)] = O.select_row(s, i, spec.mode, keep_num=spec.keep_num, keep_den=spec.keep_den, k=spec.k,
                                         flags=spec.flags)
        counts[int(r)] = len(lists[int(r)])
    rp = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    col = np.concatenate([np.asarray(lists[int(r)], np.int32) for r in sorted(lists)]) if lists else np.zeros(0, np.int32)
    return rp, col


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, timed on this machine's host cores.  One step = the oracle's
    block-sparse attention on a fixed sample of (head, query-block) rows of the bench workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import seer_oracle as O
    from paper_2410_13276_b200 import workloads as W
    w = W.make_workload(args.workload, seq=args.seq)
    spec = pick_mask(w, args, need_threshold=False)
    nbs = [int(n) for n in w.num_blocks]
    rows, off = [], 0
    for nb in nbs:
        for h in range(0, w.num_q_heads, 8):
            rows += [off + h * nb + i for i in sorted({0, nb // 4, nb // 2, nb - 1})]
        off += nb * w.num_q_heads
    rp, col = seeded_lists_for_rows(w, spec, rows)
    blocks = int(rp[-1])
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        O.sparse_attention(w.q, w.k, w.v, w.cu_seqlens, rp, col, w.num_q_heads, w.num_kv_heads, 64, w.softmax_scale, rows=rows)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * float(np.mean(times))
    val = blocks * FLOP_PER_BLOCK / (ms * 1e-3) / 1e12
    cores = len(os.sched_getaffinity(0))
    sample = (f"oracle attention (fp64 numpy) on {len(rows)} sampled (head, query-block) rows = {blocks} kept blocks per step; "
              "gate and mask oracle not included")
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                      "config": workload_desc(w, spec),
                      "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
                      "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    from paper_2410_13276_b200 import binding as B, workloads as W
    from paper_2410_13276_b200.prefill import Prefill

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # every rank runs the same layer on its own GPU: shards are independent (no data-path collective) -> weak scaling
    w = W.make_workload(args.workload, seq=args.seq)
    spec = pick_mask(w, args)
    p = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, device=local, want_lse=False)
    B.seer_set_attn_impl(p.ctx, args.attn_impl)
    p.set_inputs(w.q, w.k, w.v, w.wq, w.wk)
    params = B.make_mask_params(spec.mode, keep_num=spec.keep_num, keep_den=spec.keep_den, k=spec.k,
                                threshold=spec.threshold or 0.0, flags=spec.flags)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local) if rank == 0 else None     # polls from here on; only the timed region's samples are kept

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        p.run(params)
    barrier()
    assert p.status() == 0, "device status raised during warm-up"
    nnz = int(p.nnz.item())

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    l0 = B.seer_launch_count(p.ctx)
    barrier()
    if sampler:
        sampler.mark_start()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    # small workloads fit the 126 MB L2: overwrite a buffer twice that size before every step, outside the event spans
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if input_bytes(w) <= 2 * L2_BYTES else None
    t_start.record(stream)
    for s in range(args.steps):
        if flush_buf is not None:
            flush_buf.fill_(s & 0xff)
        ev[s][0].record(stream); p.gate()
        ev[s][1].record(stream); p.mask(params)
        ev[s][2].record(stream); p.attn()
        ev[s][3].record(stream)
    t_end.record(stream)
    barrier()
    total_ms = t_start.elapsed_time(t_end)
    if flush_buf is not None:                                # leave the flushes out: sum of the per-step spans
        total_ms = float(sum(e[0].elapsed_time(e[3]) for e in ev))
        del flush_buf
    launches = B.seer_launch_count(p.ctx) - l0
    clocks = None
    if sampler:
        # a short timed region may have seen fewer than three samples: keep the same load running (untimed) until it has
        t_lim = time.time() + 3.0
        while sampler.count_since_start() < 3 and time.time() < t_lim:
            sampler.extended = True
            p.gate(); p.mask(params); p.attn()
            torch.cuda.synchronize()
        sampler.mark_end()
        clocks = sampler.stop()
    assert p.status() == 0
    if world > 1:
        t = torch.tensor([total_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_step = total_ms / args.steps
    # the gate's bandwidth-bound first kernel (pooling + projection) on its own, outside the timed region
    gate_pool_ms = None
    if rank == 0:
        for _ in range(3):
            p.gate_project()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(10):
            p.gate_project()
        b.record(stream); torch.cuda.synchronize()
        gate_pool_ms = a.elapsed_time(b) / 10
        p.gate(); p.mask(params)
    gate_ms = float(np.median([e[0].elapsed_time(e[1]) for e in ev]))
    mask_ms = float(np.median([e[1].elapsed_time(e[2]) for e in ev]))
    attn_all = [e[2].elapsed_time(e[3]) for e in ev]
    attn_ms = float(np.mean(attn_all))
    flops = nnz * FLOP_PER_BLOCK
    value = world * flops / (ms_step * 1e-3) / 1e12

    # dense-list run of the same attention kernel (speedup column), outside the timed region
    dense_ms = None
    if not args.no_dense and rank == 0:
        dparams = B.make_mask_params(B.SEER_TOPK_RATIO, keep_num=1, keep_den=1, flags=B.SEER_FORCE_DIAG)
        p.mask(dparams)
        p.attn(); torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); p.attn(); p.attn(); b.record(stream); torch.cuda.synchronize()
        dense_ms = a.elapsed_time(b) / 2
        p.mask(params)

    # the gate with the paper's best pooling (avg on Q; avg, max, min on K) and block-level RoPE, outside the timed
    # region: same single pass over Q and K, wider projection, a rotation in the epilogue
    gate_var = None
    if rank == 0 and not args.no_extras:
        theta = 500000.0
        wq_v = torch.from_numpy(W.make_gate_weights(9001, w.num_q_heads, 128)).cuda()
        wk_v = torch.from_numpy(W.make_gate_weights(9002, w.num_kv_heads, 3 * 128)).cuda()
        opt = B.seer_gate_options(B.SEER_POOL_AVG, B.SEER_POOL_AVG | B.SEER_POOL_MAX | B.SEER_POOL_MIN, theta)
        for _ in range(3):
            p.gate_ex(opt, wq_v, wk_v)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(5):
            p.gate_ex(opt, wq_v, wk_v)
        b.record(stream); torch.cuda.synchronize()
        gate_var = {"pool_q": "avg", "pool_k": "avg+max+min", "rope_theta": theta, "gate_ms": a.elapsed_time(b) / 5}
        p.gate()                                             # restore the scores of the bench mask
        del wq_v, wk_v

    # gate and mask in one call with the scores held one band at a time (no quadratic buffer), outside the timed
    # region; the lists must equal those of the two separate calls bit for bit
    fused = None
    if rank == 0 and not args.no_extras:
        band_mb = 128
        rp_ref, col_ref = p.row_ptr.clone(), p.col_idx[:nnz].clone()
        for _ in range(3):
            p.gate_mask(params, band_bytes=band_mb << 20)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(5):
            p.gate_mask(params, band_bytes=band_mb << 20)
        b.record(stream); torch.cuda.synchronize()
        fused = {"band_mb": band_mb, "ms": a.elapsed_time(b) / 5, "separate_ms": gate_ms + mask_ms,
                 "scratch_bytes": int(p.ws_fused.numel()), "separate_bytes": int(p.ws.numel() + p.scores.numel() * 4),
                 "lists_equal": bool(torch.equal(p.row_ptr, rp_ref) and torch.equal(p.col_idx[:nnz], col_ref))}
        p.ws_fused = None
        del rp_ref, col_ref

    # the same layer with 128-token gate blocks (gate and mask at B = 128, lists expanded for the 64-token attention
    # tiles), outside the timed region
    block128 = None
    if rank == 0 and not args.no_extras:
        p.scores = None                                      # one score matrix at a time
        p2 = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, device=local, ctx=p.ctx, want_lse=False, block=128)
        p2.q, p2.k, p2.v, p2.wq, p2.wk, p2.o = p.q, p.k, p.v, p.wq, p.wk, p.o
        for _ in range(2):
            p2.gate(); p2.mask(params); p2.attn()
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        e[0].record(stream); p2.gate(); e[1].record(stream)
        B.seer_block_mask(p2.ctx, p2.shape, p2.scores, params, p2.row_ptr, p2.col_idx, p2.col_capacity, p2.nnz, None)
        e[2].record(stream); p2.expand(); e[3].record(stream); p2.attn(); e[4].record(stream)
        torch.cuda.synchronize()
        n64 = int(p2.nnz64.item())
        t = [e[i].elapsed_time(e[i + 1]) for i in range(4)]
        block128 = {"gate_ms": t[0], "mask_ms": t[1], "expand_ms": t[2], "attn_ms": t[3], "kept_blocks_128": int(p2.nnz.item()),
                    "kept_blocks_64": n64, "attn_tflops": n64 * FLOP_PER_BLOCK / (t[3] * 1e-3) / 1e12}
        del p2
        p.scores = torch.empty(max(B.seer_scores_elems(p.shape), 1), dtype=torch.float32, device="cuda")
        p.gate(); p.mask(params)                             # back to the bench lists

    # chunked prefill: the last 8192 tokens of the same layer as queries against all its keys (block-aligned chunk;
    # rows and lists keep the numbering of the whole sequence), outside the timed region
    chunked = None
    if rank == 0 and not args.no_extras and w.total_tokens >= 16384 and len(w.cu_seqlens) == 2:
        ct = 8192
        p.scores = None
        p3 = Prefill(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, device=local, ctx=p.ctx, want_lse=False,
                     cu_seqlens_q=[0, ct])
        p3.q = p.q[w.total_tokens - ct:].contiguous()
        p3.k, p3.v, p3.wq, p3.wk = p.k, p.v, p.wq, p.wk
        for _ in range(2):
            p3.run(params)
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record(stream); p3.gate(); e[1].record(stream); p3.mask(params); e[2].record(stream); p3.attn(); e[3].record(stream)
        torch.cuda.synchronize()
        n3 = int(p3.nnz.item())
        t = [e[i].elapsed_time(e[i + 1]) for i in range(3)]
        o3 = p3.o
        del p3
        p.scores = torch.empty(max(B.seer_scores_elems(p.shape), 1), dtype=torch.float32, device="cuda")
        p.gate(); p.mask(params); p.attn()                   # the whole layer again: the chunk must equal its last rows
        torch.cuda.synchronize()
        same = bool(torch.equal(o3, p.o[w.total_tokens - ct:]))
        chunked = {"chunk_tokens": ct, "gate_ms": t[0], "mask_ms": t[1], "attn_ms": t[2], "kept_blocks": n3,
                   "attn_tflops": n3 * FLOP_PER_BLOCK / (t[2] * 1e-3) / 1e12, "o_equals_rows_of_whole_run": same}
        del o3

    # list statistics of the bench mask: K/V sharing factor of the lists inside a GQA group (entries / distinct
    # (KV head, query block, key block) triples) and issued over useful MMA work of the tcgen05 kernel (S^T is computed on
    # whole 128-key tiles, so the last tile of an odd list is half padding; P V skips that half)
    list_stats = None
    if rank == 0 and not args.no_extras and len(w.cu_seqlens) == 2:
        rp_h = p.row_ptr.cpu().numpy().astype(np.int64)
        col_h = p.col_idx[:nnz].cpu().numpy().astype(np.int64)
        nb_h = int(w.num_blocks[0]); G_h = w.num_q_heads // w.num_kv_heads
        counts = np.diff(rp_h)
        row_of = np.repeat(np.arange(len(counts), dtype=np.int64), counts)
        head_of, i_of = row_of // nb_h, row_of % nb_h
        triple = ((head_of // G_h) * nb_h + i_of) * nb_h + col_h
        useful = float(counts.sum())
        issued = float((2 * ((counts + 1) // 2)).sum())
        list_stats = {"kv_sharing_factor": useful / float(np.unique(triple).size),
                      "mma_issued_over_useful": (issued + useful) / (2.0 * useful)}
        del rp_h, col_h, row_of, head_of, i_of, triple

    # the max-pooled attention map on the kept blocks (Eq. 2; a side output for distillation / diagnostics), outside the
    # timed region: one attention launch that also writes lse, then the block-max pass
    block_max_ms = None
    if rank == 0 and not args.no_extras:
        p.lse = torch.empty((w.num_q_heads, w.total_tokens), dtype=torch.float32, device="cuda")
        p.attn(); p.block_max(); torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); p.block_max(); b.record(stream); torch.cuda.synchronize()
        block_max_ms = a.elapsed_time(b)
        p.lse = None; p.bmax = None

    # the kernel's own timeline: one launch of the instrumented instantiation (CTA 0; clocks per tile by role and step)
    timeline = None
    if rank == 0 and args.timeline:
        timeline = attention_timeline(p, B, torch)

    # the other workloads (and the other TopK ratios of c3), outside the timed region: gate, mask, attention, dense lists
    all_wl = None
    if rank == 0 and args.all_workloads:
        all_wl = []
        burst = peaks()[0]
        for name, keep in (("c1", None), ("c2", None), ("c3", "1/2"), ("c3", "1/4"), ("c3", "1/10"), ("c3", "1/20"),
                           ("c4", None), ("c5", None)):
            all_wl.append(time_workload(name, keep, args, local, B, W, Prefill, torch, burst))

    # end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        shape = p.shape
        hq = torch.from_numpy(w.q.view(np.int16)).pin_memory()
        hk = torch.from_numpy(w.k.view(np.int16)).pin_memory()
        hv = torch.from_numpy(w.v.view(np.int16)).pin_memory()
        hwq = torch.from_numpy(w.wq).pin_memory(); hwk = torch.from_numpy(w.wk).pin_memory()
        ho = torch.empty((w.total_tokens, w.num_q_heads, 128), dtype=torch.int16).pin_memory()
        arena = torch.empty(B.seer_prefill_host_arena_bytes(shape), dtype=torch.uint8, device="cuda")
        n_e2e = max(2, min(args.steps, 5))
        for _ in range(2):
            B.seer_prefill_host(p.ctx, shape, hq, hk, hv, hwq, hwk, params, ho, None, arena)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            B.seer_prefill_host(p.ctx, shape, hq, hk, hv, hwq, hwk, params, ho, None, arena)
        b.record(stream)
        barrier()
        e_ms = a.elapsed_time(b) / n_e2e
        if world > 1:
            t = torch.tensor([e_ms], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t.item())
        h2d = hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2 + hwq.numel() * 4 + hwk.numel() * 4
        e2e = {"value": world * flops / (e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(ho.numel() * 2), "steps": n_e2e}
        del arena

    if rank == 0:
        burst, sustained, hbm, src = peaks()
        achieved = flops / (attn_ms * 1e-3) / 1e12
        gate_pool_bytes = (w.num_q_heads + w.num_kv_heads) * (w.total_tokens * 256 + int(sum(w.num_blocks)) * 768)
        mask_bytes = (B.seer_causal_blocks(p.shape) + nnz + B.seer_mask_rows(p.shape)) * 4
        # DRAM bytes of one attention launch from an ncu capture of this very command; other workloads have no capture
        traffic, traffic_source = None, "no ncu capture for this command"
        if w.name == "c3" and args.seq is None and (spec.keep_num, spec.keep_den) == (1, 10) and args.attn_impl == 0:
            traffic, traffic_source = TRAFFIC_C3_KEEP10
        out = {"metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
               "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_desc(w, spec),
               "kept_blocks": nnz, "stage_ms": {"gate": gate_ms, "mask": mask_ms, "attn": attn_ms,
                                                "attn_min": float(min(attn_all)), "attn_median": float(np.median(attn_all))},
               "attn_kernel": {0: "tcgen05", 1: "mma.sync", 2: "chosen by shape"}[args.attn_impl],
               # the same attention time with a row's diagonal block counted as (B + 1) / 2B of a block (what a causal
               # kernel needs of it): the figure FlashAttention-style FLOP counts give
               "attn_tflops_diag_counted_half": (nnz - B.seer_mask_rows(p.shape) * (1.0 - 65.0 / 128.0)) * FLOP_PER_BLOCK
                                                / (attn_ms * 1e-3) / 1e12,
               "roofline": {"bound": "tensor", "achieved": achieved, "peak": burst, "unit": "TFLOP/s",
                            "frac": achieved / burst, "peak_source": f"bf16 dense burst, of {src}",
                            "frac_of_sustained": (achieved / sustained) if sustained else None, "traffic": traffic,
                            "traffic_source": traffic_source, "kernel": "seer_sparse_attn"},
               "gate_gbs": ((w.num_q_heads + w.num_kv_heads) * w.total_tokens * 256) / (gate_ms * 1e-3) / 1e9,
               # pooling + projection alone: Q and K read once, 768 bytes written per (head, block); against the measured copy bandwidth
               "gate_pool_ms": gate_pool_ms,
               "gate_pool_gbs": gate_pool_bytes / (gate_pool_ms * 1e-3) / 1e9,
               "gate_pool_frac": gate_pool_bytes / (gate_pool_ms * 1e-3) / 1e9 / hbm,
               # mask builder: every causal score read once, every kept block and row offset written once (algorithmic bytes)
               "mask_gbs": mask_bytes / (mask_ms * 1e-3) / 1e9, "mask_frac": mask_bytes / (mask_ms * 1e-3) / 1e9 / hbm,
               "all_workloads": all_wl, "timeline": timeline, "gate_variant": gate_var, "block_max_ms": block_max_ms, "fused_gate_mask": fused, "block128": block128, "chunked_prefill": chunked, "list_stats": list_stats,
               "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e}
        if dense_ms:
            dense_blocks = B.seer_causal_blocks(p.shape)
            out["dense"] = {"attn_ms": dense_ms, "tflops": dense_blocks * FLOP_PER_BLOCK / (dense_ms * 1e-3) / 1e12,
                            "speedup_sparse_over_dense": dense_ms / attn_ms}
        if not args.no_cpu:
            rp, col = p.lists_host()
            out["cpu_baseline"] = cpu_oracle_sample(w, spec, rp, col)
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
