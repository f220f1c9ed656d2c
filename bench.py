#!/usr/bin/env python
"""Benchmark of the POP hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl pop|reference] [--workload NAME]

One *step* is one pass of the whole hot path over one batch of synthetic input: for each of
`--layers` FFN layers (distinct weights, so that the decode working set is far larger than L2)
a prefill partition (prompt scoring, rank-select, repack; the input-independent weight statistics
are prepared once per layer, outside the step), then `--tokens` decode tokens, each running
through all layers (every layer reads the token's x: an FFN block's input comes out of a
normalisation layer, and chaining y into x without one overflows within a few layers), i.e.
layers x tokens decode layer-steps.

The headline metric is the decode throughput in layer-steps per second at batch 1 on the
Llama-2-7B-shaped FFN (hidden 4096, intermediate 11008, bf16, FFN sparsity 20 %, gamma 0.1),
with its reciprocal (us per layer-step) and the achieved fraction of HBM bandwidth on the bytes
the step has to read.  The same JSON line carries the other workloads (`per_workload`), the
method's variants and the partition-fraction sweep (`variants`), and a CUDA-graph replay of the
decode loop beside the eager launches.  N > 1 runs N independent replicas (the path does not
shard): started under torchrun the ranks come from the environment, otherwise `--gpus N` starts
them itself.
"""
import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

WORKLOADS = {
    # name: (d, N, dtype, prompt tokens, batch, FFN sparsity r)
    "llama2_7b_ffn_r20_b1": (4096, 11008, "bf16", 512, 1, 0.2),
    "llama2_7b_ffn_r40_b1": (4096, 11008, "bf16", 512, 1, 0.4),
    "mixtral_expert_r20_b1": (4096, 14336, "bf16", 512, 1, 0.2),
    "llama2_13b_ffn_r40_b1": (5120, 13824, "bf16", 704, 1, 0.4),
    "llama2_13b_ffn_r40_b8": (5120, 13824, "bf16", 704, 8, 0.4),
    "small_f32": (512, 1376, "f32", 64, 1, None),
}
GAMMA = 0.1


def ratios_of(name):
    d, N, dt, L, B, r = WORKLOADS[name]
    if r is None:
        return (0.30, 0.40, 0.30)
    return (1.0 - r - GAMMA / 2, GAMMA, r - GAMMA / 2)


def algorithmic_bytes_per_layer_step(d, es, n_ret, n_cand, k, B):
    """Bytes one decode layer-step has to read/write: gate+up rows of R u C, down rows of
    R + selected, plus the small vectors (x, y, candidate norms, h round trip)."""
    weights = es * d * (2 * (n_ret + n_cand) + (n_ret + k))
    small = 2 * B * d * es + 8 * n_cand + 2 * 4 * B * (n_ret + n_cand)
    return weights + small


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for (_, r) in self.rows]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- oracle leg (CPU)
def oracle_sample(name, seed=0, prompt_sample=64, decode_sample=4, one_thread=False):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the prefill
    partition from the first `prompt_sample` prompt tokens and `decode_sample` decode steps."""
    from oracle import pop_oracle as po
    from paper_2602_06822_b200 import workloads as wl
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    d, N, dt, L, B, r = WORKLOADS[name]
    ratios = ratios_of(name)
    cfg = wl.FFNConfig(name, d=d, N=N, dtype=dt, prompt_tokens=min(L, prompt_sample), decode_steps=decode_sample,
                       batch=B, ratios=wl.Ratios(*ratios), seed=seed)
    w = wl.make_ffn_workload(cfg)
    Wh = [np.asarray(a.values, dtype=np.float64) for a in (w.weights.Wg, w.weights.Wu, w.weights.Wd)]
    X = np.asarray(w.X.values, dtype=np.float64)
    xs = np.asarray(w.xs.values, dtype=np.float64)
    t0 = time.perf_counter()
    part = po.prefill_partition(X, *Wh, ratios)
    t1 = time.perf_counter()
    k = part["C"].size // 2
    for t in range(decode_sample):
        po.decode_step(xs[t], *Wh, part["R"], part["C"], k)
    t2 = time.perf_counter()
    per_step = (t2 - t1) / decode_sample
    out = {"value": 1.0 / per_step, "unit": "layer-steps/s", "cores": int(threads), "kind": "oracle",
           "sample": f"1 layer: prefill partition on {X.shape[0]} of {L * B} prompt tokens ({t1 - t0:.2f} s), "
                     f"then {decode_sample} decode layer-steps ({per_step * 1e3:.1f} ms each)",
           "prefill_s": t1 - t0, "decode_s_per_layer_step": per_step}
    if one_thread:
        # the same decode step with the numerical library held to one thread
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                t3 = time.perf_counter()
                po.decode_step(xs[0], *Wh, part["R"], part["C"], k)
                t4 = time.perf_counter()
            out["value_one_thread"] = 1.0 / (t4 - t3)
            out["sample"] += f"; one more step on 1 thread ({(t4 - t3) * 1e3:.0f} ms)"
        except ImportError:
            pass
    return out


def run_reference(args):
    """`--impl reference`: there is no reference implementation of the paper; the arm is the CPU
    oracle timed on the host cores on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    vals = []
    for i in range(args.warmup + args.steps):
        o = oracle_sample(name, seed=i, prompt_sample=32, decode_sample=2)
        if i >= args.warmup:
            vals.append(o)
    per = statistics.mean(v["decode_s_per_layer_step"] for v in vals)
    total = sum(v["decode_s_per_layer_step"] * 2 + v["prefill_s"] for v in vals)
    d, N, dt, L, B, r = WORKLOADS[name]
    from oracle import pop_oracle as po
    nr, nc, _np = po.region_sizes(N, ratios_of(name))
    kd = nc // 2
    value = 1.0 / per
    line = {"impl": "reference", "metric": "pop_decode_layer_steps_per_s", "value": value, "unit": "layer-steps/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "d": d, "N": N, "batch": B, "prompt_tokens": L * B, "ratios": list(ratios_of(name)),
                       "n_ret": int(nr), "n_cand": int(nc), "k": int(kd), "layers": args.layers, "tokens": args.tokens,
                       "sample_per_step": "one layer: prefill partition on 32 prompt tokens + 2 decode layer-steps"},
            "cpu_baseline": {"value": value, "unit": "layer-steps/s", "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": "per step: prefill partition on 32 prompt tokens + 2 decode layer-steps of one layer"},
            "e2e": {"value": value, "unit": "layer-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "us_per_layer_step": per * 1e6}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- measured DRAM traffic
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode kernel from an ncu capture, kept with the
# profiles.  The figure belongs to one version of the kernel's source: it is reported only while the source file
# still hashes to what it was when the counters were taken, and is null otherwise.
NCU_TRAFFIC = {
    "llama2_7b_ffn_r20_b1": {"bytes": 235.6e6, "kernel_source": "paper_2602_06822_b200/csrc/pop_decode_stream.cu",
                             "sha256_16": "3dead4f2bd36d12a", "summary": "profiles/pop_decode_stream_kernel_llama2_7b_r20_b1.md"},
}


def source_hash(rel):
    try:
        return hashlib.sha256(open(os.path.join(ROOT, rel), "rb").read()).hexdigest()[:16]
    except OSError:
        return None


def ncu_traffic(workload, decode_kernel_auto=True):
    """(bytes or None, where the figure comes from)."""
    rec = NCU_TRAFFIC.get(workload)
    if rec is None or not decode_kernel_auto:
        return None, "no stored capture for this workload and kernel"
    if source_hash(rec["kernel_source"]) != rec["sha256_16"]:
        return None, f"stored ncu capture ({rec['summary']}) predates the current {rec['kernel_source']}"
    return rec["bytes"], f"stored ncu capture, {rec['summary']} (not measured in this run)"


# ----------------------------------------------------------------------------- multi-rank arithmetic
def max_over_ranks(v, world, device):
    """The slowest rank's time: every rank contributes its own device-measured duration."""
    if world == 1:
        return v
    import torch
    import torch.distributed as dist
    t = torch.tensor([v], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, units_per_rank, max_ms):
    """Replicas only (the path does not shard): every rank processes `units_per_rank` layer-steps of its own
    seeded workload; the job's throughput is all of them over the slowest rank's time."""
    return world * units_per_rank / (max_ms * 1e-3)


# ----------------------------------------------------------------------------- GPU arm
def make_layers(torch, pop, g, dev, d, N, dtype, layers):
    """Seeded synthetic weights of `layers` distinct FFN layers (~ N(0, 0.02^2)) and their prepared statistics."""
    W, WT = [], []
    for _ in range(layers):
        Wg = (torch.randn(N, d, generator=g, device=dev, dtype=torch.float32) * 0.02).to(dtype)
        Wu = (torch.randn(N, d, generator=g, device=dev, dtype=torch.float32) * 0.02).to(dtype)
        Wd = (torch.randn(d, N, generator=g, device=dev, dtype=torch.float32) * 0.02).to(dtype)
        W.append((Wg, Wu, Wd))
        WT.append(pop.Weights(Wg, Wu, Wd))
    return W, WT


def time_decode(torch, pop, parts, xs, k, act, stream, reps=3):
    """Decode only: one warm-up pass and `reps` - 1 timed passes of tokens x layers layer-steps; ms per pass (list)."""
    tokens, layers = xs.shape[0], len(parts)
    ms = []
    for rep_i in range(reps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        ev[0].record(stream)
        for t in range(tokens):
            for l in range(layers):
                pop.decode_step(parts[l], xs[t], k, y=act[l + 1])
        ev[1].record(stream)
        torch.cuda.synchronize()
        if rep_i:
            ms.append(ev[0].elapsed_time(ev[1]))
    for p_ in parts:
        p_.check()
    return ms


def time_decode_graph(torch, pop, parts, xs, k, act, replays=7):
    """The same decode loop captured once into a CUDA graph and replayed; ms per replay (list), or None with the reason."""
    tokens, layers = xs.shape[0], len(parts)
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for t in range(tokens):
                    for l in range(layers):
                        pop.decode_step(parts[l], xs[t], k, y=act[l + 1], stream=side)
        torch.cuda.synchronize()
        ms = []
        for i in range(replays + 1):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev[0].record()
            graph.replay()
            ev[1].record()
            torch.cuda.synchronize()
            if i:
                ms.append(ev[0].elapsed_time(ev[1]))
        for p_ in parts:
            p_.check()
        del graph
        return ms, None
    except Exception as e:       # capture is an optional second protocol: report why it is missing
        torch.cuda.synchronize()
        return None, f"{type(e).__name__}: {e}"[:200]


def run_pop(args):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as ge
    from paper_2602_06822_b200 import pop

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the POP library has no CPU path")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} needs GPU {local}, the node has {torch.cuda.device_count()}")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        ge.build()
    if world > 1:
        dist.barrier()
    pop.lib()
    # every step builds and destroys one partition per layer: let the library keep all of their memory for the next
    # step (the default keeps 1 GiB), as a serving loop with this many live layers would
    pop.set_config(slab_cache_bytes=16 << 30,
                   decode_kernel={"auto": pop.POP_DECODE_AUTO, "fused": pop.POP_DECODE_FUSED, "simple": pop.POP_DECODE_SIMPLE}[args.decode_kernel])

    name = args.workload
    d, N, dts, L, B, r = WORKLOADS[name]
    dtype = torch.bfloat16 if dts == "bf16" else torch.float32
    es = 2 if dts == "bf16" else 4
    ratios = ratios_of(name)
    n_ret, n_cand, n_pruned, k = pop.region_sizes(N, ratios)
    layers, tokens = args.layers, args.tokens

    # ---- synthetic inputs, seeded, generated on the device (weights ~ N(0, 0.02^2), activations ~ N(0,1))
    g = torch.Generator(device=dev)
    g.manual_seed(1234 + rank)
    W, WT = make_layers(torch, pop, g, dev, d, N, dtype, layers)
    X = torch.randn(B * L, d, generator=g, device=dev, dtype=torch.float32).to(dtype)
    xs = torch.randn(tokens, B, d, generator=g, device=dev, dtype=torch.float32).to(dtype)
    X_host = X.cpu().pin_memory()
    xs_host = xs.cpu().pin_memory()
    y_host = torch.empty(tokens, B, d, dtype=dtype).pin_memory()
    act = [torch.empty(B, d, device=dev, dtype=dtype) for _ in range(layers + 1)]
    X_stage = torch.empty_like(X)
    stream = torch.cuda.current_stream()

    def one_step(e2e, ev):
        """prefill all layers, then tokens x layers decode layer-steps.  ev = (start, mid, end) events."""
        ev[0].record(stream)
        Xin = X
        if e2e:
            X_stage.copy_(X_host, non_blocking=True)
            Xin = X_stage
        parts = [WT[l].prefill_partition(Xin, ratios) for l in range(layers)]
        ev[1].record(stream)
        for t in range(tokens):
            if e2e:
                act[0].copy_(xs_host[t], non_blocking=True)
                cur = act[0]
            else:
                cur = xs[t]
            for l in range(layers):
                pop.decode_step(parts[l], cur, k, y=act[l + 1])
            if e2e:
                y_host[t].copy_(act[layers], non_blocking=True)
                stream.synchronize()          # the token's result is on the host before the next token
        ev[2].record(stream)
        return parts

    def free(parts):
        for p in parts:
            p.destroy()

    def timed(e2e, K, Wn):
        for _ in range(Wn):
            free(one_step(e2e, [torch.cuda.Event(enable_timing=True) for _ in range(3)]))
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
        l0 = pop.kernel_launch_count()
        t0 = time.time()
        for i in range(K):
            parts = one_step(e2e, evs[i])
            torch.cuda.synchronize()
            for p in parts:
                p.check()
            free(parts)
        torch.cuda.synchronize()
        t1 = time.time()
        launches = pop.kernel_launch_count() - l0
        pre = [e[0].elapsed_time(e[1]) for e in evs]      # ms
        dec = [e[1].elapsed_time(e[2]) for e in evs]
        tot = evs[0][0].elapsed_time(evs[-1][2])           # first start -> last end, includes frees between steps
        return {"prefill_ms": sum(pre), "decode_ms": sum(dec), "decode_ms_list": dec, "total_ms": tot,
                "launches": launches, "t0": t0, "t1": t1}

    sampler = ClockSampler(local)
    sampler.start()
    res = timed(False, args.steps, args.warmup)
    clocks = sampler.stop(res["t0"], res["t1"])
    e2e_steps = max(1, args.steps // 2)
    e2e = timed(True, e2e_steps, 1)

    def reduce_max(v):
        return max_over_ranks(v, world, dev)

    # partial probing (Sec. 3.4): the same prefill from every fourth prompt token, outside the timed steps
    probe_ms = None
    if not args.no_variants:
        torch = __import__("torch")
        for rep in range(3):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev[0].record(stream)
            pp = [WT[l].prefill_partition_probe(X, ratios, 4) for l in range(layers)]
            ev[1].record(stream)
            torch.cuda.synchronize()
            for q in pp:
                q.check()
                q.destroy()
            probe_ms = ev[0].elapsed_time(ev[1]) / layers
        probe_ms = reduce_max(probe_ms)

    peaks = {}
    pk_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk_path):
        peaks = json.load(open(pk_path))
    peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_src = "measured (MEASURED_PEAKS.json hbm_gbs)" if "hbm_gbs" in peaks else "fallback 6650 GB/s"

    def decode_row(label, d_, N_, B_, parts, xs_, k_, act_, note=None, graph=False):
        """One decode-only measurement as a row of the JSON line."""
        sizes = parts[0].n_ret, parts[0].n_cand
        ms = time_decode(torch, pop, parts, xs_, k_, act_, stream)
        us = 1e3 * reduce_max(statistics.median(ms)) / (len(parts) * xs_.shape[0])
        vb = algorithmic_bytes_per_layer_step(d_, es, sizes[0], sizes[1], k_, B_)
        row = {"workload": label, "d": d_, "N": N_, "batch": B_, "n_ret": sizes[0], "n_cand": sizes[1], "k": k_,
               "us_per_layer_step": us, "algorithmic_bytes_per_launch": vb, "achieved_GBs": vb / (us * 1e-6) / 1e9,
               "frac_of_measured_hbm": vb / (us * 1e-6) / 1e9 / peak}
        try:
            parts[0].streamed_scores()
            row["kernel"] = "streaming"
        except pop.PopError:
            row["kernel"] = "fused / multi-kernel"
        if note:
            row["note"] = note
        if graph:
            gms, why = time_decode_graph(torch, pop, parts, xs_, k_, act_)
            if gms:
                row["graph_replay_us_per_layer_step"] = 1e3 * reduce_max(statistics.median(gms)) / (len(parts) * xs_.shape[0])
            else:
                row["graph_replay"] = why
        return row

    # ---- the method's variants and the partition-fraction sweep on the headline shape (Sec. 4.6, Table 5, Fig. 4)
    variants = []
    graph_row = None
    if not args.no_variants:
        n_act = n_ret + k

        def variant(label, ratios_v, k_v, note, graph=False):
            parts = [WT[l].prefill_partition(X, ratios_v) for l in range(layers)]
            row = decode_row(label, d, N, B, parts, xs, k_v, act, note, graph)
            free(parts)
            row["variant"] = row.pop("workload")
            return row

        graph_row = variant("POP, gamma 0.1 (the headline setting)", ratios, k,
                            "eager launches and a CUDA-graph replay of the same tokens x layers loop", graph=True)
        variants.append(graph_row)
        variants.append(variant("static mask (Variant 1)", (n_act / N, 0.0, (N - n_act) / N), 0,
                                "mask fixed at prefill: the same active count, no candidate region, no per-step choice"))
        variants.append(variant("all channels candidates (Variant 2)", (0.0, 1.0, 0.0), n_act,
                                "every channel scored at every step"))
        if r is not None:
            for gam in (0.05, 0.2):
                rv = (1.0 - r - gam / 2, gam, r - gam / 2)
                nc_v = pop.region_sizes(N, rv)[1]
                variants.append(variant(f"POP, gamma {gam}", rv, nc_v // 2, "partition-fraction sweep (gamma = |C| / N)"))

    # ---- the other workloads, decode only, each with its own weights
    per_workload = []
    if not args.no_workloads and name == "llama2_7b_ffn_r20_b1":
        for wname in ("llama2_7b_ffn_r40_b1", "mixtral_expert_r20_b1", "llama2_13b_ffn_r40_b1", "llama2_13b_ffn_r40_b8"):
            d2, N2, dts2, L2, B2, r2 = WORKLOADS[wname]
            rat2 = ratios_of(wname)
            if (d2, N2) == (d, N):
                W2, WT2 = W, WT
            else:
                for wt in WT:
                    wt.destroy()
                del W, WT
                torch.cuda.empty_cache()
                W2, WT2 = make_layers(torch, pop, g, dev, d2, N2, dtype, layers)
                W, WT = W2, WT2
                d, N = d2, N2
            X2 = torch.randn(B2 * L2, d2, generator=g, device=dev, dtype=torch.float32).to(dtype)
            xs2 = torch.randn(tokens, B2, d2, generator=g, device=dev, dtype=torch.float32).to(dtype)
            act2 = [torch.empty(B2, d2, device=dev, dtype=dtype) for _ in range(layers + 1)]
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            parts = [WT2[l].prefill_partition(X2, rat2) for l in range(layers)]
            torch.cuda.synchronize()
            free(parts)
            ev[0].record(stream)
            parts = [WT2[l].prefill_partition(X2, rat2) for l in range(layers)]
            ev[1].record(stream)
            torch.cuda.synchronize()
            k2 = parts[0].n_cand // 2
            row = decode_row(wname, d2, N2, B2, parts, xs2, k2, act2)
            row["prefill_partition_ms_per_layer"] = reduce_max(ev[0].elapsed_time(ev[1])) / layers
            row["prompt_tokens"] = B2 * L2
            free(parts)
            per_workload.append(row)
            del X2, xs2, act2
        d, N, dts, L, B, r = WORKLOADS[name]

    dec_ms = reduce_max(res["decode_ms"])
    pre_ms = reduce_max(res["prefill_ms"])
    tot_ms = reduce_max(res["total_ms"])
    e2e_dec_ms = reduce_max(e2e["decode_ms"] + e2e["prefill_ms"])
    layer_steps = layers * tokens * args.steps
    us_per_ls = 1e3 * dec_ms / layer_steps
    us_per_ls_median = 1e3 * reduce_max(statistics.median(res["decode_ms_list"])) / (layers * tokens)
    value = whole_job_value(world, layer_steps, dec_ms)
    e2e_value = whole_job_value(world, layers * tokens * e2e_steps, e2e_dec_ms)

    if rank == 0:
        abytes = algorithmic_bytes_per_layer_step(d, es, n_ret, n_cand, k, B)
        achieved = abytes / (us_per_ls * 1e-6) / 1e9
        cpu = oracle_sample(name, one_thread=True) if world == 1 and not args.no_cpu_baseline else None
        traffic, traffic_src = ncu_traffic(name, pop.get_config().decode_kernel == pop.POP_DECODE_AUTO)
        line = {
            "metric": "pop_decode_layer_steps_per_s", "value": value, "unit": "layer-steps/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dts, "data": "synthetic",
            "config": {"workload": name, "d": d, "N": N, "batch": B, "prompt_tokens": L * B, "ratios": list(ratios),
                       "n_ret": n_ret, "n_cand": n_cand, "k": k, "layers": layers, "tokens": tokens,
                       "slab_cache_bytes": 16 << 30, "decode_kernel": args.decode_kernel,
                       "l2": f"inputs larger than L2: {layers} layers x {abytes / 1e6:.1f} MB of distinct weights per token",
                       "replicas": world},
            "us_per_layer_step": us_per_ls,
            "us_per_layer_step_median_of_steps": us_per_ls_median,
            "tokens_per_s_if_32_such_layers": 1e6 / (32 * us_per_ls),
            "prefill_partition_ms_per_layer": pre_ms / (layers * args.steps),
            "prefill_note": "pop_prefill_partition_prepared: the weight statistics (pop_weights_prepare) are computed once "
                            "per layer before the timed region; scoring on the tensor cores (tcgen05), exact re-scoring "
                            "of the channels near the rank boundaries, ranking, repack",
            "prefill_probe": None if probe_ms is None else {"token_stride": 4, "ms_per_layer": probe_ms,
                                                            "note": "pop_prefill_partition_probe: statistics from every 4th prompt token"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "layer-steps/s",
                    "h2d_bytes_per_step": int(X_host.numel() * es + tokens * B * d * es),
                    "d2h_bytes_per_step": int(tokens * B * d * es),
                    "prefill_ms_per_step": e2e["prefill_ms"] / e2e_steps,
                    "decode_ms_per_step": e2e["decode_ms"] / e2e_steps,
                    "note": "prompt copied from pinned host memory before prefill; per token x copied in, last layer's y "
                            "copied out and the stream synchronised"},
            "gpu_launches": int(res["launches"]),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "traffic_source": traffic_src, "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": abytes, "frac_of_nominal_8TBs": achieved / 8000.0,
                         "kernel": "decode layer-step (all kernels of one pop_decode_step, averaged over the decode region)"},
        }
        if graph_row is not None and "graph_replay_us_per_layer_step" in graph_row:
            gu = graph_row["graph_replay_us_per_layer_step"]
            line["graph_replay"] = {"us_per_layer_step": gu, "achieved_GBs": abytes / (gu * 1e-6) / 1e9,
                                    "frac_of_measured_hbm": abytes / (gu * 1e-6) / 1e9 / peak,
                                    "note": "median of 7 replays of one captured tokens x layers decode loop"}
        if variants:
            line["variants"] = variants
        if per_workload:
            line["per_workload"] = per_workload
        if cpu is not None:
            line["cpu_baseline"] = {k2: cpu[k2] for k2 in ("value", "unit", "cores", "kind", "sample", "value_one_thread") if k2 in cpu}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def free_port():
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_ranks(args, argv):
    """`--gpus N` outside torchrun: start N ranks (one per GPU) of this script and pass their exit code on."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="pop", choices=["pop", "reference"])
    ap.add_argument("--workload", default="llama2_7b_ffn_r20_b1", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--tokens", type=int, default=128)
    ap.add_argument("--decode-kernel", default="auto", choices=["auto", "fused", "simple"],
                    help="decode kernel family (pop_set_config): auto = the streaming kernel where it applies")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the method's variants and the gamma sweep")
    ap.add_argument("--no-workloads", action="store_true", help="skip the per_workload list")
    args = ap.parse_args(argv)
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.impl == "reference":
        run_reference(args)
        return
    world = int(os.environ.get("WORLD_SIZE", "0"))
    if world == 0 and args.gpus > 1:
        raise SystemExit(spawn_ranks(args, argv))
    if world > 1 and world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE is {world}")
    run_pop(args)


if __name__ == "__main__":
    main()
