"""Times sb_tree_attention on the five benchmark configurations and prints one JSON line each.

    python -m paper_2605_07243_b200.time_configs [--configs 1,2,3,4,5] [--iters 30] [--num-splits S]

For every configuration: CUDA-event time per call (a CUDA graph walks buffer sets whose total
exceeds L2, so K/V come from HBM; median over `iters` replays), algorithmic bytes and flops,
achieved GB/s and TFLOP/s, and the fraction of the binding roof (HBM copy bandwidth or dense bf16
throughput, from MEASURED_PEAKS.json when present).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

import numpy as np
import torch

from . import binding as sb
from . import device_inputs as dev
from . import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peaks():
    try:
        d = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 6650.0, 1400.0, "fallback"


def _cases(which):
    if which == 1:
        return W.config1_tiny()[0], 0
    if which == 2:
        return W.config2_verify_layer(), 0
    if which == 3:
        return W.config3_drafter()[0], 0
    if which == 4:
        return W.config4_batched(with_logits=False)[0], 0
    if which == 5:
        return W.config5_long(with_logits=False)[0], 16
    raise ValueError(which)


def time_config(which, iters, num_splits=None):
    case, splits = _cases(which)
    if num_splits is not None:
        splits = num_splits
    kv_bytes = case.k.nbytes + case.v.nbytes
    # enough distinct KV copies to exceed L2 (126 MB) between two uses of the same copy
    n_sets = max(2, min(32, int(np.ceil(2 * 134e6 / kv_bytes))))
    tb, q, kw = dev.attention_args(case)
    sets = [(tb.k_cache, tb.v_cache)] + [(tb.k_cache.clone(), tb.v_cache.clone()) for _ in range(n_sets - 1)]
    out = torch.empty_like(q)
    lse = torch.empty((q.shape[0], case.n_q_heads), dtype=torch.float32, device="cuda")
    status = torch.empty(case.batch, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(256, sb.sb_tree_attention_workspace_bytes(tb, q.shape[0], splits)), dtype=torch.uint8, device="cuda")

    def call(i):
        k, v = sets[i % n_sets]
        sb.sb_tree_attention(tb, q, out, lse, num_splits=splits, workspace=ws, status=status, k_cache=k, v_cache=v, **kw)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(n_sets):
            call(i)
        stream.synchronize()
        assert int(status.max()) == 0
        # one CUDA graph that walks all buffer sets once: host launch cost is out of the picture
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(n_sets):
                call(i)
        graph.replay()
        stream.synchronize()
        times = []
        for _ in range(iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3 / n_sets)
    us = statistics.median(times)
    hbm, tflops, kind = _peaks()
    nbytes, flops = case.algorithmic_bytes(), case.flops()
    t_hbm, t_tc = nbytes / (hbm * 1e9) * 1e6, flops / (tflops * 1e12) * 1e6
    bound = "hbm" if t_hbm >= t_tc else "tensor"
    return {"config": which, "us_per_call": us, "p10_us": float(np.percentile(times, 10)),
            "p90_us": float(np.percentile(times, 90)), "algorithmic_bytes": nbytes, "flops": flops,
            "GBps": nbytes / us / 1e3, "TFLOPps": flops / us / 1e6, "bound": bound,
            "roof_us": max(t_hbm, t_tc), "frac_of_roof": max(t_hbm, t_tc) / us, "peaks": kind,
            "kv_sets_rotated": n_sets, "num_splits": splits}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--num-splits", type=int, default=None,
                    help="override the number of KV chunks (0 = the library's choice)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device")
    sb.load()
    for c in [int(x) for x in args.configs.split(",")]:
        print(json.dumps(time_config(c, args.iters, args.num_splits)), flush=True)


if __name__ == "__main__":
    main()
