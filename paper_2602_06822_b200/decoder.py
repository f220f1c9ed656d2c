"""Llama-shaped decoder harness around the POP library (the paper applies POP to every FFN of a
decoder and leaves attention unchanged: Sec. 3.3 first paragraph, Sec. 4.4, App. A.1).

This is harness code, not part of the library's hot path: embeddings, RMSNorm (gain 1), rotary
position embeddings (base 10000, rotate-half convention), dense multi-head attention with a KV cache
and the residual stream are plain torch ops in bf16; every FFN goes through the C ABI
(`pop_prefill_partition_with_output` for the prompt, `pop_decode_step` per generated token), or,
for the dense baseline of the latency table, through torch linear layers.

Weights are synthetic (seeded, ~ N(0, 0.02^2)); token ids are a seeded sequence that is fed
teacher-forced, so that no sampling and no LM head are needed.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import torch
import torch.nn.functional as F

from . import pop


@dataclass
class DecoderConfig:
    n_layers: int = 32
    d: int = 4096
    n_heads: int = 32
    N: int = 11008
    vocab: int = 32000
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    seed: int = 3
    weight_std: float = 0.02


def ratios_for(r: float, gamma: float = 0.1):
    """(retained, candidate, pruned) for FFN pruning ratio r with partition fraction gamma = |C| / N."""
    return (1.0 - r - gamma / 2, gamma, r - gamma / 2)


class Decoder:
    """ffn = "pop" (every FFN through the library, ratios given) or "dense" (torch linear layers)."""

    def __init__(self, cfg: DecoderConfig, device="cuda:0", ffn: str = "pop", ratios=None, k: Optional[int] = None):
        self.cfg, self.dev, self.ffn = cfg, torch.device(device), ffn
        g = torch.Generator(device=self.dev)
        g.manual_seed(cfg.seed)

        def rnd(*shape):
            return (torch.randn(*shape, generator=g, device=self.dev, dtype=torch.float32) * cfg.weight_std).bfloat16()

        self.embed = rnd(cfg.vocab, cfg.d)
        self.layers: List[Dict[str, torch.Tensor]] = []
        for _ in range(cfg.n_layers):
            self.layers.append({"Wq": rnd(cfg.d, cfg.d), "Wk": rnd(cfg.d, cfg.d), "Wv": rnd(cfg.d, cfg.d), "Wo": rnd(cfg.d, cfg.d),
                                "Wg": rnd(cfg.N, cfg.d), "Wu": rnd(cfg.N, cfg.d), "Wd": rnd(cfg.d, cfg.N)})
        self.hd = cfg.d // cfg.n_heads
        inv = 1.0 / (cfg.rope_base ** (torch.arange(0, self.hd, 2, device=self.dev, dtype=torch.float32) / self.hd))
        self.inv_freq = inv
        self.ratios = ratios
        self.k = k
        self.weights = [pop.Weights(l["Wg"], l["Wu"], l["Wd"]) for l in self.layers] if ffn == "pop" else None
        self.parts: List[Optional[pop.Partition]] = [None] * cfg.n_layers
        self.kv: List[Optional[tuple]] = [None] * cfg.n_layers
        self.pos = 0
        self.trace = None          # when a dict: (layer, step) -> recorded FFN inputs / outputs, for layer-local parity
        self.timers = None         # when a dict: "attention" / "mlp" -> list of (start, end) CUDA events

    # ------------------------------------------------------------------ pieces
    def rmsnorm(self, h):
        return F.rms_norm(h, (self.cfg.d,), eps=self.cfg.rms_eps)          # gain 1: one fused kernel

    def rope(self, x, pos0):
        """x [T, heads, hd]; positions pos0 .. pos0 + T - 1; rotate-half convention."""
        T = x.shape[0]
        ang = (torch.arange(pos0, pos0 + T, device=self.dev, dtype=torch.float32)[:, None] * self.inv_freq[None, :])
        cos, sin = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
        xf = x.float()
        x1, x2 = xf[..., : self.hd // 2], xf[..., self.hd // 2:]
        return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1).bfloat16()

    def attention(self, li, a, pos0):
        """a [T, d] normalised input; appends to the layer's KV cache; returns the attention block's output [T, d]."""
        L, cfg = self.layers[li], self.cfg
        T = a.shape[0]
        q = self.rope(F.linear(a, L["Wq"]).view(T, cfg.n_heads, self.hd), pos0)
        kx = self.rope(F.linear(a, L["Wk"]).view(T, cfg.n_heads, self.hd), pos0)
        vx = F.linear(a, L["Wv"]).view(T, cfg.n_heads, self.hd)
        if self.kv[li] is None:
            K, V = kx, vx
        else:
            K, V = torch.cat([self.kv[li][0], kx]), torch.cat([self.kv[li][1], vx])
        self.kv[li] = (K, V)
        o = F.scaled_dot_product_attention(q.transpose(0, 1), K.transpose(0, 1), V.transpose(0, 1), is_causal=(T > 1))
        return F.linear(o.transpose(0, 1).reshape(T, cfg.d), L["Wo"])

    def _timed(self, name):
        class _T:
            def __init__(s2, outer):
                s2.o = outer
            def __enter__(s2):
                if s2.o.timers is not None:
                    s2.e0 = torch.cuda.Event(enable_timing=True); s2.e0.record()
            def __exit__(s2, *a):
                if s2.o.timers is not None:
                    e1 = torch.cuda.Event(enable_timing=True); e1.record()
                    s2.o.timers.setdefault(name, []).append((s2.e0, e1))
        return _T(self)

    def dense_ffn(self, li, f):
        L = self.layers[li]
        return F.linear(F.silu(F.linear(f, L["Wg"])) * F.linear(f, L["Wu"]), L["Wd"])

    # ------------------------------------------------------------------ the two stages
    def prefill(self, ids: torch.Tensor):
        """ids [T] prompt token ids -> hidden states [T, d] after the last layer.  Builds every layer's partition."""
        assert self.pos == 0
        h = self.embed[ids]
        for li in range(self.cfg.n_layers):
            with self._timed("attention"):
                h = h + self.attention(li, self.rmsnorm(h), 0)
            f = self.rmsnorm(h)
            with self._timed("mlp"):
                if self.ffn == "pop":
                    if self.parts[li] is not None:
                        self.parts[li].destroy()
                    kk = self.k if self.k is not None else pop.region_sizes(self.cfg.N, self.ratios)[3]
                    self.parts[li], y = self.weights[li].prefill_partition_with_output(f, self.ratios, kk)
                else:
                    y = self.dense_ffn(li, f)
            if self.trace is not None:
                self.trace[("prefill", li)] = (f.clone(), y.clone())
            h = h + y
        self.pos = ids.shape[0]
        return h

    def decode(self, tok: torch.Tensor, step: int = 0):
        """One teacher-forced token id [1] -> hidden state [1, d]."""
        h = self.embed[tok]
        for li in range(self.cfg.n_layers):
            with self._timed("attention"):
                h = h + self.attention(li, self.rmsnorm(h), self.pos)
            f = self.rmsnorm(h)
            with self._timed("mlp"):
                if self.ffn == "pop":
                    p = self.parts[li]
                    kk = self.k if self.k is not None else p.n_cand // 2
                    want = self.trace is not None and self.trace.get("want", lambda l, s: True)(li, step)
                    if want:
                        mask = torch.empty(p.n_cand, dtype=torch.uint8, device=self.dev)
                        sel = torch.empty(kk, dtype=torch.int32, device=self.dev)
                        y = pop.decode_step(p, f, kk, mask_out=mask, sel_out=sel)
                        self.trace[(li, step)] = (f.clone(), y.clone(), mask, sel)
                    else:
                        y = pop.decode_step(p, f, kk)
                else:
                    y = self.dense_ffn(li, f)
            h = h + y
        self.pos += 1
        return h

    # ------------------------------------------------------------------ static-shape decode (CUDA-graph capturable)
    def begin_static(self, ids_all: torch.Tensor, max_len: int):
        """After prefill: moves the KV cache into preallocated [max_len] buffers and keeps the position and the
        teacher-forced token ids on the device, so that one decode step is a fixed sequence of launches."""
        cfg = self.cfg
        self.max_len = max_len
        self.ids_dev = ids_all.to(self.dev)
        self.pos_t = torch.tensor([self.pos], device=self.dev, dtype=torch.int64)
        self.kv_static = []
        for li in range(cfg.n_layers):
            K = torch.zeros(max_len, cfg.n_heads, self.hd, device=self.dev, dtype=torch.bfloat16)
            V = torch.zeros_like(K)
            if self.kv[li] is not None:
                K[: self.pos] = self.kv[li][0]
                V[: self.pos] = self.kv[li][1]
            self.kv_static.append((K, V))
        self.arange = torch.arange(max_len, device=self.dev)
        self.y_static = torch.zeros(1, cfg.d, device=self.dev, dtype=torch.bfloat16)

    def step_static(self, attention: bool = True, mlp: bool = True):
        """One teacher-forced token at the device-side position; no host-side value enters the launches."""
        cfg = self.cfg
        h = self.embed.index_select(0, self.ids_dev.index_select(0, self.pos_t))
        ang = self.pos_t.float()[:, None] * self.inv_freq[None, :]
        cos, sin = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
        mask = (self.arange <= self.pos_t)[None, None, :]

        def rope1(x):
            xf = x.float()
            x1, x2 = xf[..., : self.hd // 2], xf[..., self.hd // 2:]
            return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1).bfloat16()

        for li in range(cfg.n_layers):
            L = self.layers[li]
            if attention:
                a = self.rmsnorm(h)
                q = rope1(F.linear(a, L["Wq"]).view(1, cfg.n_heads, self.hd))
                kx = rope1(F.linear(a, L["Wk"]).view(1, cfg.n_heads, self.hd))
                vx = F.linear(a, L["Wv"]).view(1, cfg.n_heads, self.hd)
                K, V = self.kv_static[li]
                K.index_copy_(0, self.pos_t, kx)
                V.index_copy_(0, self.pos_t, vx)
                o = F.scaled_dot_product_attention(q.transpose(0, 1), K.transpose(0, 1), V.transpose(0, 1), attn_mask=mask)
                h = h + F.linear(o.transpose(0, 1).reshape(1, cfg.d), L["Wo"])
            if mlp:
                f = self.rmsnorm(h)
                if self.ffn == "pop":
                    p = self.parts[li]
                    y = pop.decode_step(p, f, self.k if self.k is not None else p.n_cand // 2, y=self.y_static,
                                        stream=torch.cuda.current_stream())
                else:
                    y = self.dense_ffn(li, f)
                h = h + y
        self.pos_t += 1
        return h

    def reset(self):
        self.kv = [None] * self.cfg.n_layers
        self.pos = 0

    def close(self):
        for p in self.parts:
            if p is not None:
                p.destroy()
        self.parts = [None] * self.cfg.n_layers
        if self.weights:
            for w in self.weights:
                w.destroy()
            self.weights = None


def seeded_ids(cfg: DecoderConfig, n: int, seed: int, device) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randint(0, cfg.vocab, (n,), generator=g).to(device)


def _replay_ms(graph, n, pos_t, pos0):
    pos_t.fill_(pos0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def latency_table(cfg: Optional[DecoderConfig] = None, n_in: int = 128, n_out: int = 128, device="cuda:0", reps: int = 3):
    """Attention / MLP / end-to-end latency of `n_in` prompt tokens + `n_out` generated tokens, dense and with POP
    at the paper's two MLP channel ratios for Llama-2-7B (29.9 % and 59.8 %: App. A.1), gamma 0.1: the shape of the
    paper's Table 4 (which was measured on an RTX A6000 with trained weights, module times by CUDA events).
    Here the prompt pass is timed eagerly with CUDA events; a decode step is captured once into a CUDA graph and
    replayed n_out times (so the figures are device time, not launch overhead), and the module shares come from
    two more graphs of the same step with the other module left out.  Returns a list of rows (times in ms over
    all layers and tokens, best of `reps`)."""
    cfg = cfg or DecoderConfig()
    rows = []
    for label, ffn, r in (("dense", "dense", None), ("POP, MLP ratio 29.9 %", "pop", 0.299), ("POP, MLP ratio 59.8 %", "pop", 0.598)):
        m = Decoder(cfg, device, ffn=ffn, ratios=ratios_for(r) if r is not None else None)
        ids = seeded_ids(cfg, n_in + n_out + 1, 17, m.dev)
        prefill_ms = []
        for rep in range(2):
            m.reset()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            m.prefill(ids[:n_in])
            e1.record()
            torch.cuda.synchronize()
            prefill_ms.append(e0.elapsed_time(e1))
        m.begin_static(ids, n_in + n_out + 8)
        graphs = {}
        side = torch.cuda.Stream()
        for name, att, mlp in (("e2e", True, True), ("attention", True, False), ("mlp", False, True)):
            m.pos_t.fill_(n_in)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                m.step_static(att, mlp)                   # warm-up outside capture (lazy initialisations)
            torch.cuda.synchronize()
            m.pos_t.fill_(n_in)
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph, stream=side):
                m.step_static(att, mlp)
            graphs[name] = gph
        torch.cuda.synchronize()
        t = {name: min(_replay_ms(gph, n_out, m.pos_t, n_in) for _ in range(reps)) for name, gph in graphs.items()}
        if ffn == "pop":
            for p in m.parts:
                p.check()
        rows.append({"model": label, "prefill_ms": min(prefill_ms), "decode_e2e_ms": t["e2e"], "decode_attention_ms": t["attention"],
                     "decode_mlp_ms": t["mlp"], "e2e_ms": min(prefill_ms) + t["e2e"],
                     "mlp_us_per_layer_step": 1e3 * t["mlp"] / (n_out * cfg.n_layers),
                     "attention_us_per_layer_step": 1e3 * t["attention"] / (n_out * cfg.n_layers)})
        del graphs
        m.close()
        del m
        torch.cuda.empty_cache()
    base = rows[0]
    for rw in rows:
        rw["mlp_speedup"] = base["decode_mlp_ms"] / rw["decode_mlp_ms"]
        rw["e2e_speedup"] = base["e2e_ms"] / rw["e2e_ms"]
    return rows


if __name__ == "__main__":
    import argparse
    import json
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import __graft_entry__ as ge
    ap = argparse.ArgumentParser(description="Table-4-shaped latency breakdown on the Llama-2-7B-shaped decoder")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--n-in", type=int, default=128)
    ap.add_argument("--n-out", type=int, default=128)
    a = ap.parse_args()
    ge.build()
    for rw in latency_table(DecoderConfig(n_layers=a.layers), a.n_in, a.n_out):
        print(json.dumps(rw))
