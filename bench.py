#!/usr/bin/env python
"""Benchmark of the POP hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl pop|reference] [--workload NAME]

One *step* is one pass of the whole hot path over one batch of synthetic input: for each of
`--layers` FFN layers (distinct weights, so that the decode working set is far larger than L2)
a prefill partition (channel norms, prompt scoring, rank-select, repack), then `--tokens`
decode tokens, each running through all layers in sequence (layer l's output is layer l+1's
input), i.e. layers x tokens decode layer-steps.

The headline metric is the decode throughput in layer-steps per second at batch 1 on the
Llama-2-7B-shaped FFN (hidden 4096, intermediate 11008, bf16, FFN sparsity 20 %, gamma 0.1),
with its reciprocal (us per layer-step) and the achieved fraction of HBM bandwidth on the bytes
the step has to read.  N > 1 runs N independent replicas (the path does not shard).
"""
import argparse
import json
import os
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
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode kernel, from an ncu capture of the streaming
# kernel on this workload (226.07 MB read + 9.5 MB written; the summary is kept with the profiles).  Valid for the
# default decode kernel of that workload only; None for anything else, and to be reset to None when that kernel changes.
NCU_TRAFFIC_BYTES = {"llama2_7b_ffn_r20_b1": 235.6e6}


def ncu_traffic(workload):
    if os.environ.get("POP_DECODE_IMPL", "stream") not in ("", "stream"):
        return None
    return NCU_TRAFFIC_BYTES.get(workload)


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
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        ge.build()
    if world > 1:
        dist.barrier()
    pop.lib()

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
    W = []
    for l in range(layers):
        Wg = (torch.randn(N, d, generator=g, device=dev, dtype=torch.float32) * 0.02).to(dtype)
        Wu = (torch.randn(N, d, generator=g, device=dev, dtype=torch.float32) * 0.02).to(dtype)
        Wd = (torch.randn(d, N, generator=g, device=dev, dtype=torch.float32) * 0.02).to(dtype)
        W.append((Wg, Wu, Wd))
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
        parts = [pop.prefill_partition(Xin, *W[l], ratios) for l in range(layers)]
        ev[1].record(stream)
        for t in range(tokens):
            if e2e:
                act[0].copy_(xs_host[t], non_blocking=True)
                cur = act[0]
            else:
                cur = xs[t]
            # Every layer reads the token's x: inputs of an FFN block come out of a normalisation layer, and
            # feeding one block's y into the next without it overflows within a few layers.
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
        w0 = time.perf_counter()
        for i in range(K):
            parts = one_step(e2e, evs[i])
            torch.cuda.synchronize()
            for p in parts:
                p.check()
            free(parts)
        torch.cuda.synchronize()
        w1 = time.perf_counter()
        t1 = time.time()
        launches = pop.kernel_launch_count() - l0
        pre = sum(e[0].elapsed_time(e[1]) for e in evs)      # ms
        dec = sum(e[1].elapsed_time(e[2]) for e in evs)
        tot = evs[0][0].elapsed_time(evs[-1][2])               # first start -> last end, includes frees between steps
        return {"prefill_ms": pre, "decode_ms": dec, "total_ms": tot, "wall_ms": (w1 - w0) * 1e3,
                "launches": launches, "t0": t0, "t1": t1}

    sampler = ClockSampler(local)
    sampler.start()
    res = timed(False, args.steps, args.warmup)
    clocks = sampler.stop(res["t0"], res["t1"])
    e2e = timed(True, max(1, args.steps // 2), 1)
    e2e_steps = max(1, args.steps // 2)

    def timed_variant(label, ratios_v, k_v, note):
        """The method's two limiting variants (Table 5 / Sec. 4.6) through the same two calls, decode only:
        one warm-up pass and two timed passes of `tokens` x `layers` layer-steps."""
        nr, nc, npr, _ = pop.region_sizes(N, ratios_v)
        parts = [pop.prefill_partition(X, *W[l], ratios_v) for l in range(layers)]
        ms = []
        for rep_i in range(3):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev[0].record(stream)
            for t in range(tokens):
                for l in range(layers):
                    pop.decode_step(parts[l], xs[t], k_v, y=act[l + 1])
            ev[1].record(stream)
            torch.cuda.synchronize()
            if rep_i:
                ms.append(ev[0].elapsed_time(ev[1]))
        for p_ in parts:
            p_.check()
        free(parts)
        us = 1e3 * max_over_ranks(sum(ms) / len(ms), world, dev) / (layers * tokens)
        vb = algorithmic_bytes_per_layer_step(d, es, nr, nc, k_v, B)
        return {"variant": label, "n_ret": nr, "n_cand": nc, "k": k_v, "us_per_layer_step": us,
                "algorithmic_bytes_per_launch": vb, "achieved_GBs": vb / (us * 1e-6) / 1e9, "note": note}

    variants = []
    if not args.no_variants:
        n_act = n_ret + k
        variants.append(timed_variant("static mask (Variant 1)", (n_act / N, 0.0, (N - n_act) / N), 0,
                                      "mask fixed at prefill: the same active count, no candidate region, no per-step choice"))
        variants.append(timed_variant("all channels candidates (Variant 2)", (0.0, 1.0, 0.0), n_act,
                                      "every channel scored at every step; served by the fused kernel (the streaming kernel "
                                      "holds up to 1536 candidates)"))

    def reduce_max(v):
        return max_over_ranks(v, world, dev)

    dec_ms = reduce_max(res["decode_ms"])
    pre_ms = reduce_max(res["prefill_ms"])
    tot_ms = reduce_max(res["total_ms"])
    e2e_dec_ms = reduce_max(e2e["decode_ms"] + e2e["prefill_ms"])
    layer_steps = layers * tokens * args.steps
    us_per_ls = 1e3 * dec_ms / layer_steps
    value = whole_job_value(world, layer_steps, dec_ms)
    e2e_value = whole_job_value(world, layers * tokens * e2e_steps, e2e_dec_ms)

    if rank == 0:
        peaks = {}
        pk_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(pk_path):
            peaks = json.load(open(pk_path))
        peak = float(peaks.get("hbm_gbs", 6650.0))
        peak_src = "measured (MEASURED_PEAKS.json hbm_gbs)" if "hbm_gbs" in peaks else "fallback 6650 GB/s"
        abytes = algorithmic_bytes_per_layer_step(d, es, n_ret, n_cand, k, B)
        achieved = abytes / (us_per_ls * 1e-6) / 1e9
        cpu = oracle_sample(name, one_thread=True) if world == 1 and not args.no_cpu_baseline else None
        line = {
            "metric": "pop_decode_layer_steps_per_s", "value": value, "unit": "layer-steps/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dts, "data": "synthetic",
            "config": {"workload": name, "d": d, "N": N, "batch": B, "prompt_tokens": L * B, "ratios": list(ratios),
                       "n_ret": n_ret, "n_cand": n_cand, "k": k, "layers": layers, "tokens": tokens,
                       "l2": f"inputs larger than L2: {layers} layers x {abytes / 1e6:.1f} MB of distinct weights per token",
                       "replicas": world},
            "us_per_layer_step": us_per_ls,
            "tokens_per_s_if_32_such_layers": 1e6 / (32 * us_per_ls),
            "prefill_partition_ms_per_layer": pre_ms / (layers * args.steps),
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
                         "traffic": ncu_traffic(name), "peak_source": peak_src, "algorithmic_bytes_per_launch": abytes,
                         "frac_of_nominal_8TBs": achieved / 8000.0,
                         "kernel": "decode layer-step (all kernels of one pop_decode_step, averaged over the decode region)"},
        }
        if variants:
            line["variants"] = variants
        if cpu is not None:
            line["cpu_baseline"] = {k2: cpu[k2] for k2 in ("value", "unit", "cores", "kind", "sample", "value_one_thread") if k2 in cpu}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="pop", choices=["pop", "reference"])
    ap.add_argument("--workload", default="llama2_7b_ffn_r20_b1", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--tokens", type=int, default=128)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the timing of the method's two limiting variants")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_pop(args)


if __name__ == "__main__":
    main()
