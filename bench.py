#!/usr/bin/env python
"""Benchmark of the SpecBlock verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one draft-and-verify iteration's device work on the 8B-shaped configuration: ancestor
masks, the drafter's top-k expansion (32 rows x vocab 128256), tree attention for 32 layers
(32/8 heads, D=128, prefix 2048, 60-node K=4 block tree, 32 distinct KV buffers = 276 MB, larger
than L2), greedy acceptance over bf16 logits [60, 128256], and KV compaction of all 32 layers.
The step is captured once in a CUDA graph and replayed; time is taken with CUDA events on the
launching stream, max over ranks.  Prints ONE JSON line (rank 0).

Beside the contract's figure (exactly --steps replays between two events), the line carries
distributions that do not depend on --steps: the step and every breakdown entry as median / p10 / p90
over at least 200 samples, and under "configs" the tree attention of all five benchmark
configurations (at least 200 samples for 1-3, 30 for 4-5; configuration 5 with the 16 chunks it
prescribes and with the library's own choice), each a CUDA-graph replay that walks buffer sets larger
than L2, with algorithmic bytes and flops and the fraction of its binding roof.

With N > 1 (launched by torch.distributed.run) every rank runs its own sequence (weak scaling,
no data-path collective); NCCL is used only for the barrier and the max over ranks.

--impl reference times the CPU fp64 oracle, as it stands, on the host cores on a bounded sample
of the same workload.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree-verify attention GB/s (% of B200 HBM peak) and us per verify step"
N_LAYERS = 32
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch of this workload, from an ncu
# capture of the library as committed (the summary of that capture is committed with the profiles)
ATTN_DRAM_TRAFFIC_BYTES = 9183232
FALLBACK_HBM_GBS = 6650.0
FALLBACK_TFLOPS = 1400.0   # sustained dense bf16


def measured_peaks():
    """(HBM GB/s, sustained dense bf16 TFLOP/s, "measured" | "fallback")."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, FALLBACK_TFLOPS, "fallback"


def build_workload(rank, n_layers):
    from paper_2605_07243_b200 import workloads as W
    seed = W.SEEDS[2] + 100 * rank
    par = W.config2_tree(seed)
    layers = [W.config2_verify_layer(seed, layer=l, par=par) for l in range(n_layers)]
    ver = W.config2_logits(seed, accept_len=3, par=par)
    _attn3, exp = W.config3_drafter(W.SEEDS[3] + 100 * rank)
    return par, layers, ver, exp


class ClockSampler:
    """nvidia-smi in the background during the timed region (reads settings only)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            t = [x.strip() for x in line.split(",")]
            if len(t) < 9:
                continue
            try:
                sm.append(float(t[1]))
                mx.append(float(t[2]))
            except ValueError:
                continue
            for name, val in zip(names, t[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # "under load": the upper half of the samples (the sampler also sees idle gaps)
        sm_sorted = sorted(sm)
        load = sm_sorted[len(sm_sorted) // 2:]
        return {"sm_mhz": statistics.median(load), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample_step(layers, ver, exp, n_attn_layers):
    """One bounded sample of the step on the CPU oracle; returns the algorithmic bytes it covered."""
    import numpy as np
    import oracle
    nbytes = 0
    for c in layers[:n_attn_layers]:
        oracle.tree_attention(**c.oracle_kwargs())
        nbytes += c.algorithmic_bytes()
    r = oracle.verify_accept(ver.logits, ver.node_offsets, ver.parent, ver.tok, ver.max_depth)
    nbytes += ver.logits.size * ver.logits.itemsize
    oracle.tree_expand(exp.scores, exp.block_k, exp.bucket, exp.bmap, exp.start_parent, exp.node_budget,
                       tree=exp.tree)
    nbytes += exp.scores.size * 4
    c0 = layers[0]
    k = np.concatenate([c.k.reshape(-1) for c in layers[:n_attn_layers]])
    oracle.kv_compact(n_kv_heads=c0.n_kv_heads, head_dim=c0.head_dim, cache=k, n_layers=n_attn_layers,
                      layer_stride_elems=c0.k.size, kv_capacity=c0.kv_capacity, prefix_len=c0.prefix_len,
                      node_offsets=c0.node_offsets, path_nodes=r["path_nodes"], accept_len=r["accept_len"],
                      max_depth=ver.max_depth)
    return nbytes


def run_reference(args):
    """The oracle on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    n_attn = 1
    _par, layers, ver, exp = build_workload(0, n_attn)
    for _ in range(args.warmup):
        oracle_sample_step(layers, ver, exp, n_attn)
    t0 = time.perf_counter()
    nbytes = 0
    for _ in range(args.steps):
        nbytes += oracle_sample_step(layers, ver, exp, n_attn)
    dt = time.perf_counter() - t0
    value = nbytes / dt / 1e9
    sample = (f"per step: oracle tree attention on {n_attn} of {N_LAYERS} layers + full acceptance "
              f"(60 x 128256 bf16 logits) + full top-k expansion (32 x 128256) + compaction of {n_attn} layers")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": "8B-shaped verify step (configs[1]): 32/8 heads, D=128, prefix 2048, "
                               "60-node K=4 tree, vocab 128256; bounded sample", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


def max_over_ranks(torch, values, device):
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def time_graph(torch, graph, iters, dist_on):
    """Replay `graph` `iters` times between two events on the current stream; returns ms total."""
    if dist_on:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    return e0.elapsed_time(e1)


def capture(torch, fn):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def sample_graph(torch, graph, samples, replays_per_sample=1, calls_per_replay=1):
    """`samples` event pairs on the current stream, each around `replays_per_sample` replays of `graph`
    (which holds `calls_per_replay` calls): -> microseconds per call as median / p10 / p90."""
    import numpy as np
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(samples)]
    for e0, e1 in pairs:
        e0.record()
        for _ in range(replays_per_sample):
            graph.replay()
        e1.record()
    torch.cuda.synchronize()
    us = np.asarray([e0.elapsed_time(e1) for e0, e1 in pairs]) * 1e3 / (replays_per_sample * calls_per_replay)
    return {"median_us": float(np.median(us)), "p10_us": float(np.percentile(us, 10)),
            "p90_us": float(np.percentile(us, 90)), "samples": samples,
            "calls_per_sample": replays_per_sample * calls_per_replay}


ATTENTION_CONFIGS = (   # (key, configuration, num_splits, samples)
    ("1_tiny", 1, 0, 200), ("2_8b_verify_layer", 2, 0, 200), ("3_drafter_blocks", 3, 0, 200),
    ("4_batched_paged", 4, 0, 30), ("5_long_context_16_chunks", 5, 16, 30), ("5_long_context_library_chunks", 5, 0, 30))


def time_attention_config(torch, sb, which, num_splits, samples):
    """sb_tree_attention on one benchmark configuration, standing alone: a CUDA graph walks copies of the
    K/V caches whose total exceeds twice the L2 size, so every call streams its keys and values from HBM."""
    import numpy as np
    from paper_2605_07243_b200 import device_inputs as dev
    from paper_2605_07243_b200 import workloads as W
    case = {1: lambda: W.config1_tiny()[0], 2: W.config2_verify_layer, 3: lambda: W.config3_drafter()[0],
            4: lambda: W.config4_batched(with_logits=False)[0], 5: lambda: W.config5_long(with_logits=False)[0]}[which]()
    kv_bytes = case.k.nbytes + case.v.nbytes
    l2 = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size
    n_sets = max(2, min(32, int(np.ceil(2 * l2 / kv_bytes))))
    tb, q, kw = dev.attention_args(case)
    sets = [(tb.k_cache, tb.v_cache)] + [(tb.k_cache.clone(), tb.v_cache.clone()) for _ in range(n_sets - 1)]
    out = torch.empty_like(q)
    lse = torch.empty((q.shape[0], case.n_q_heads), dtype=torch.float32, device="cuda")
    status = torch.empty(case.batch, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(256, sb.sb_tree_attention_workspace_bytes(tb, q.shape[0], num_splits)), dtype=torch.uint8,
                     device="cuda")

    def walk():
        for k, v in sets:
            sb.sb_tree_attention(tb, q, out, lse, num_splits=num_splits, workspace=ws, status=status, k_cache=k,
                                 v_cache=v, **kw)

    walk()
    torch.cuda.synchronize()
    assert int(status.max()) == 0
    graph = capture(torch, walk)
    st = sample_graph(torch, graph, samples, 1, n_sets)
    hbm, tflops, kind = measured_peaks()
    nbytes, flops = case.algorithmic_bytes(), case.flops()
    t_hbm, t_tc = nbytes / (hbm * 1e9) * 1e6, flops / (tflops * 1e12) * 1e6
    us = st["median_us"]
    res = {"us": us, "p10_us": st["p10_us"], "p90_us": st["p90_us"], "samples": samples, "kv_sets_rotated": n_sets,
           "num_splits": num_splits, "algorithmic_bytes": nbytes, "flops": flops, "GBps": nbytes / us / 1e3,
           "TFLOPps": flops / us / 1e6, "bound": "hbm" if t_hbm >= t_tc else "tensor",
           "roof_us": max(t_hbm, t_tc), "frac": max(t_hbm, t_tc) / us,
           "peak": f"{kind}: " + (f"{hbm} GB/s HBM copy" if t_hbm >= t_tc else f"{tflops} TFLOP/s sustained dense bf16")}
    del sets, graph, tb, q, out, ws
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    from paper_2605_07243_b200 import binding as sb
    from paper_2605_07243_b200.pipeline import VerifyStep

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist_on = world > 1
    torch.cuda.set_device(local_rank)
    if dist_on:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sb.load()

    par, layers, ver, exp = build_workload(rank, N_LAYERS)
    step = VerifyStep(layers, ver, exp, num_splits=args.num_splits, keep_host=True)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        # eager once: sets kernel attributes, counts launches, checks the status words
        launches_per_step = step.launches_per_step()
        side.synchronize()
        assert int(step.attn_status.max()) == 0 and int(step.accept["status"].max()) == 0
        assert int(step.compact_status.max()) == 0 and int(step.expand["status"][0]) == 0
        assert int(step.accept["accept_len"][0]) == int(ver.planted_len[0])
        g_step = capture(torch, step.run_device)
        g_attn = capture(torch, step.run_attention)
        g_expand = capture(torch, step.run_expand)
        g_accept = capture(torch, step.run_accept)
        g_expand_cold = g_accept_cold = None
        if not args.step_only:
            step.run_expand_cold()
            step.run_accept_cold()
            side.synchronize()
            assert int(step.expand["cold_n_nodes"].min()) == int(step.expand["n_nodes"][0])
            g_expand_cold = capture(torch, step.run_expand_cold)
            g_accept_cold = capture(torch, step.run_accept_cold)
        g_compact = capture(torch, step.run_compact)
        extras = []   # pieces outside the step (the "next" rows), timed on their own
        if not args.step_only:
            for name, fn in (("rank_features_not_in_step", step.run_rank_features),
                             ("expand_and_rank_features_one_pass_not_in_step", step.run_expand_features),
                             ("verifier_signal_not_in_step", step.run_signal),
                             ("verify_sample_T1_not_in_step", step.run_sample),
                             ("shift_project_32x4096_not_in_step", step.run_shift_all),
                             ("fuse_project_8x4x4096_not_in_step", step.run_fuse_all)):
                fn()
                extras.append((name, capture(torch, fn)))
            # one whole iteration (two drafter blocks growing the tree on the device, then the verify forward on it)
            from paper_2605_07243_b200.iteration import build_8b_iteration
            iteration = build_8b_iteration(layers, ver.logits, ver.max_depth, num_splits=args.num_splits)
            iteration.run()
            side.synchronize()
            assert int(iteration.attn_status.max()) == 0 and int(iteration.accept["status"].max()) == 0
            assert all(int(e["status"][0]) == 0 for e in iteration.blocks)
            extras.append(("whole_iteration_2_blocks_32_layers_not_in_step", capture(torch, iteration.run)))

        for _ in range(max(args.warmup, 3)):
            g_step.replay()
        side.synchronize()
        sampler = ClockSampler(local_rank)
        sampler.start()

        def keep_busy(seconds):
            if args.quick:
                return
            # same work as the timed region, untimed: gives the 100 ms clock sampler a load to see
            t_end = time.perf_counter() + seconds
            while time.perf_counter() < t_end:
                for _ in range(20):
                    g_step.replay()
                side.synchronize()

        keep_busy(0.7)
        launches0 = sb.sb_kernel_launch_count()
        ms_total = time_graph(torch, g_step, args.steps, dist_on)
        gpu_launches = launches_per_step * args.steps
        # the dominant kernel (tree attention): 32 launches on 32 distinct KV buffers per replay
        attn_iters = max(args.steps, 10)
        ms_attn = time_graph(torch, g_attn, attn_iters, dist_on)
        # distributions that do not depend on --steps: one sample = one replay of the step / the 32 layers
        n_samples = 20 if args.quick else 200
        step_stats = sample_graph(torch, g_step, n_samples)
        attn_stats = sample_graph(torch, g_attn, n_samples, 1, N_LAYERS)
        keep_busy(0.4)
        clocks = sampler.stop()
        parts_stats = {}
        calls = {"shift_project_32x4096_not_in_step": step.SHIFT_SETS, "fuse_project_8x4x4096_not_in_step": step.FUSE_SETS,
                 "expand": step.COLD_SETS, "accept": step.COLD_SETS}
        # expand / accept: one graph walks COLD_SETS copies of the scores / logits (more than twice the L2 size), one
        # call each, so every call streams its matrix from HBM and the replay's own cost (about 4 us) is shared by all
        # of them -- what a call costs inside an iteration; the *_single_call_graph entries replay ONE call on the same
        # matrix (L2-warm, the whole replay cost on it)
        cold = [] if args.step_only else [("expand", g_expand_cold), ("accept", g_accept_cold)]
        for name, g in cold + [("expand_single_call_graph", g_expand), ("accept_single_call_graph", g_accept),
                               ("compact", g_compact)] + extras:
            # short graphs: ten replays per sample keep the event pair's own cost out of the figure
            reps = 1 if name.startswith("whole_iteration") or name in ("expand", "accept") else 10
            parts_stats[name] = sample_graph(torch, g, n_samples, reps, calls.get(name, 1))
        parts_ms = {k: v["median_us"] * 1e-3 for k, v in parts_stats.items()}
        configs = None
        if world == 1 and not args.quick and not args.step_only:
            configs = {key: time_attention_config(torch, sb, which, splits, n)
                       for key, which, splits, n in ATTENTION_CONFIGS}

        # end to end: inputs in pinned host memory, results back to pinned host memory
        e2e_steps = 1 if args.quick else max(3, min(args.steps, 5))
        step.run_from_host()
        side.synchronize()
        if dist_on:
            torch.distributed.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            step.run_from_host()
        e1.record()
        side.synchronize()
        ms_e2e = e0.elapsed_time(e1) / e2e_steps
    del launches0

    ms_step = ms_total / args.steps
    ms_attn_launch = ms_attn / attn_iters / N_LAYERS
    ms_step, ms_attn_launch, ms_e2e = max_over_ranks(torch, [ms_step, ms_attn_launch, ms_e2e], "cuda")

    parts = step.algorithmic_bytes()
    total_bytes = parts["total"]
    value = world * total_bytes / (ms_step * 1e-3) / 1e9
    e2e_value = world * total_bytes / (ms_e2e * 1e-3) / 1e9
    h2d, d2h = step.host_bytes()
    peak, _tflops, peak_kind = measured_peaks()
    attn_bytes = parts["attention_per_layer"]
    achieved = attn_bytes / (ms_attn_launch * 1e-3) / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "8B-shaped verify step (configs[1]): batch 1 per GPU, 32 query / 8 KV heads, "
                               "D=128, contiguous bf16 KV prefix 2048, 60-node K=4/M=2 block tree, 32 layers, "
                               "bf16 logits vocab 128256 (accept_len 3), fp32 drafter scores 32x128256",
                   "step_contents": "ancestor masks, the drafter's top-k expansion of the next block (32 x 128256 "
                                    "scores: part of the iteration, not of the verify forward proper), 32 attention "
                                    "layers, greedy acceptance, compaction of 32 layers",
                   "l2": "inputs larger than L2: 32 distinct KV buffers (276 MB) stream through per step",
                   "launch": "whole step captured in one CUDA graph", "num_splits": args.num_splits},
        "us_per_verify_step": ms_step * 1e3,
        "pct_of_nominal_hbm_peak": 100.0 * value / world / NOMINAL_HBM_GBS,
        "step_algorithmic_bytes": total_bytes,
        "breakdown_us": {"attention_32_layers": ms_attn_launch * N_LAYERS * 1e3,
                         "attention_per_layer": ms_attn_launch * 1e3,
                         **{k: v * 1e3 for k, v in parts_ms.items()}},
        "step_us_stats": step_stats,
        "breakdown_us_stats": {"attention_per_layer": attn_stats, **parts_stats},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e},
        "gpu_launches": gpu_launches,
        "roofline": {"bound": "hbm", "kernel": "sb::attn_tc_kernel<128, 6> (tcgen05), one launch per layer",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"{peak_kind} HBM copy bandwidth", "traffic": ATTN_DRAM_TRAFFIC_BYTES,
                     "algorithmic_bytes_per_launch": attn_bytes,
                     "pct_of_nominal_8TBps": 100.0 * achieved / NOMINAL_HBM_GBS},
    }
    if configs is not None:
        line["configs"] = configs
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.quick:
        import oracle
        t0 = time.perf_counter()
        nb = oracle_sample_step(layers, ver, exp, N_LAYERS)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": nb / dt / 1e9, "unit": "GB/s", "cores": oracle.num_threads(),
                                "kind": "oracle", "seconds": dt,
                                "sample": "one whole step (all 32 attention layers, acceptance, expansion, "
                                          "compaction) on the fp64 oracle, once"}
    if rank == 0 and world == 1 and args.oracle_configs:
        # The oracle's tree attention on each of the five benchmark configurations, once, on the host
        # cores (the counterpart of the "configs" key); a baseline only.
        import oracle
        from paper_2605_07243_b200 import workloads as W
        makers = {1: lambda: W.config1_tiny()[0], 2: W.config2_verify_layer, 3: lambda: W.config3_drafter()[0],
                  4: lambda: W.config4_batched(with_logits=False)[0], 5: lambda: W.config5_long(with_logits=False)[0]}
        by_config = {}
        for c in [int(x) for x in args.oracle_configs.split(",")]:
            case = makers[c]()
            t0 = time.perf_counter()
            oracle.tree_attention(**case.oracle_kwargs())
            dt = time.perf_counter() - t0
            by_config[str(c)] = {"seconds": dt, "GB/s": case.algorithmic_bytes() / dt / 1e9,
                                 "GFLOP/s": case.flops() / dt / 1e9}
        line["cpu_baseline_attention_by_config"] = {"cores": oracle.num_threads(), "kind": "oracle", "configs": by_config}
    if dist_on:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--oracle-configs", default="",
                    help="also time the CPU oracle's tree attention on these benchmark configurations (e.g. 1,2,3,4,5)")
    ap.add_argument("--step-only", action="store_true",
                    help="profiling aid: leave out the pieces timed outside the step (their kernels then do not appear)")
    ap.add_argument("--attention-config", default="",
                    help="profiling aid: time sb_tree_attention on ONE benchmark configuration and print its entry of "
                         "the \"configs\" key, e.g. 5 or 5:16 (configuration:num_splits); nothing else runs")
    ap.add_argument("--samples", type=int, default=30, help="samples for --attention-config")
    ap.add_argument("--quick", action="store_true",
                    help="profiling aid: no clock-sampling busy loops, a single end-to-end step, no CPU baseline")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.attention_config:
        import torch
        from paper_2605_07243_b200 import binding as sb
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
        sb.load()
        which, _, splits = args.attention_config.partition(":")
        with torch.cuda.stream(torch.cuda.Stream()):
            print(json.dumps(time_attention_config(torch, sb, int(which), int(splits or 0), args.samples)))
        return 0
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
