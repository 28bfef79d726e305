"""Writes tests/golden/thresholds.json: the fp32 gate-score threshold of every threshold-mask workload, tuned by
bisection on the ORACLE's scores until the kept fraction of causal blocks (forced blocks included) is within 0.5 %
(absolute) of the workload's target sparsity.  Calls only oracle/ and the input generators.

    python tests/golden/make_thresholds.py [names...]
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import seer_oracle as O                      # noqa: E402
from paper_2410_13276_b200 import workloads as W         # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "thresholds.json")


def kept_fraction(scores, thr, flags):
    kept = causal = 0
    thr = np.float32(thr)
    for S in scores:
        nb = S.shape[-1]
        il = np.tril_indices(nb)
        m = S > thr
        if flags & O.FORCE_DIAG:
            m[:, np.arange(nb), np.arange(nb)] = True
        if flags & O.FORCE_SINK:
            m[:, :, 0] = True
        kept += int(m[:, il[0], il[1]].sum())
        causal += S.shape[0] * len(il[0])
    return kept / causal


def tune(name):
    w = W.make_workload(name)
    spec = w.masks[0]
    assert spec.mode == W.MODE_THRESHOLD
    scores = O.gate_scores(w.q, w.k, w.wq, w.wk, w.cu_seqlens, w.block)
    target_keep = 1.0 - spec.target_sparsity
    lo, hi = 0.0, 1.0                                     # keep fraction is non-increasing in the threshold
    for _ in range(60):
        mid = np.float32(0.5 * (lo + hi))
        if kept_fraction(scores, mid, spec.flags) > target_keep:
            lo = float(mid)
        else:
            hi = float(mid)
    thr = np.float32(hi)
    frac = kept_fraction(scores, thr, spec.flags)
    rp, _ = O.block_mask(scores, O.MODE_THRESHOLD, threshold=float(thr), flags=spec.flags)
    dens = []
    base = 0
    for S in scores:
        hq, nb, _ = S.shape
        cnt = np.diff(rp[base:base + hq * nb + 1]).reshape(hq, nb)
        dens.append((cnt / np.arange(1, nb + 1)[None, :])[:, 64:].ravel() if nb > 64 else (cnt / np.arange(1, nb + 1)).ravel())
        base += hq * nb
    dens = np.concatenate(dens)
    return {"threshold_hex": float(thr).hex(), "threshold": float(thr), "kept_fraction": frac,
            "target_sparsity": spec.target_sparsity, "kept_blocks": int(rp[-1]),
            "row_density_p5_p50_p95": [float(np.percentile(dens, p)) for p in (5, 50, 95)]}


if __name__ == "__main__":
    names = sys.argv[1:] or ["c2s", "c4s", "c5s", "c2", "c4", "c5"]
    data = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for n in names:
        data[n] = tune(n)
        print(n, data[n], flush=True)
        with open(OUT, "w") as f:
            json.dump(data, f, indent=1, sort_keys=True)
