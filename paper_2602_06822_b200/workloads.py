"""Seeded synthetic inputs for the POP hot path.

This module only *draws numbers*: it holds none of the method's arithmetic
(no scoring, no partitioning, no FFN math), so both the CPU oracle's tests and
the CUDA path can consume the very same arrays without sharing any code that
matters for parity.

Every array is produced on the host with ``numpy.random.Generator(PCG64(seed))``.
For the bf16 workloads the fp32 draws are rounded to bf16 (round to nearest
even) once; the 16-bit patterns go to the GPU and the *same values*, widened
back to fp32, go to the oracle.

The shapes follow the paper's models (Llama-2-7B / 13B FFN blocks, a
Mixtral-shaped expert layer, a VLM-style prompt of visual + text tokens) and
its settings (pruning ratio 20 % / 40 %, partition fraction gamma = 0.1, Sec. 4
"Implementation Details").  They stand in for the paper's trained checkpoints
and evaluation suites, which are not available offline.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

F32 = "f32"
BF16 = "bf16"


# --------------------------------------------------------------------------- bf16 packing
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest even); returns the uint16 patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 patterns (uint16) to the fp32 values they denote (exact)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Array:
    """One input array in both of its forms.

    ``values``  fp32 array holding exactly the numbers the device sees
                (bf16-representable when ``dtype == 'bf16'``) - for the oracle.
    ``raw``     what is copied to the device: the same fp32 array, or the
                uint16 bf16 patterns.
    """
    values: np.ndarray
    raw: np.ndarray
    dtype: str

    @property
    def shape(self):
        return self.values.shape


def as_array(a: np.ndarray, dtype: str) -> Array:
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == F32:
        return Array(a, a, F32)
    if dtype == BF16:
        bits = f32_to_bf16_bits(a)
        return Array(bf16_bits_to_f32(bits), bits, BF16)
    raise ValueError(f"unknown dtype {dtype!r}")


# --------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class Ratios:
    """Fractions of the N intermediate channels put in each region."""
    retained: float
    candidate: float
    pruned: float

    def astuple(self) -> Tuple[float, float, float]:
        return (self.retained, self.candidate, self.pruned)


def ratios_for(r: float, gamma: float = 0.1) -> Ratios:
    """Region fractions for an FFN pruning ratio ``r`` and partition fraction
    ``gamma``: the candidate band has width gamma centred on the pruning
    threshold (Sec. 3.3, thresholds at the r-delta and r+delta quantiles with
    gamma = 2 delta)."""
    half = gamma / 2.0
    return Ratios(retained=1.0 - r - half, candidate=gamma, pruned=r - half)


@dataclass(frozen=True)
class FFNConfig:
    name: str
    d: int                 # hidden size
    N: int                 # intermediate size (the prunable channels)
    dtype: str
    prompt_tokens: int     # L per prompt
    decode_steps: int
    batch: int = 1         # decode batch B (prompts folded into L at prefill)
    ratios: Ratios = Ratios(0.30, 0.40, 0.30)
    seed: int = 0
    activation: str = "normal"      # "normal" | "vlm" (heavy-tailed visual rows + text rows)
    visual_tokens: int = 0
    weight_std: float = 0.02
    k: Optional[int] = None         # None => floor(n_C / 2)


def config1() -> FFNConfig:
    """Small fp32 layer the oracle finishes in seconds."""
    return FFNConfig("cfg1_small_f32", d=512, N=1376, dtype=F32, prompt_tokens=64,
                     decode_steps=16, ratios=Ratios(0.30, 0.40, 0.30), seed=0, k=275)


def config2(r: float = 0.2, steps: int = 128) -> FFNConfig:
    """Llama-2-7B-shaped FFN, bf16, batch 1, FFN sparsity r, gamma = 0.1."""
    return FFNConfig(f"cfg2_llama7b_r{int(round(r * 100))}", d=4096, N=11008, dtype=BF16,
                     prompt_tokens=512, decode_steps=steps, ratios=ratios_for(r, 0.1), seed=2)


def config4_expert(r: float = 0.2, steps: int = 128) -> FFNConfig:
    """One expert of the Mixtral-shaped layer (hidden 4096, expert intermediate 14336)."""
    return FFNConfig(f"cfg4_mixtral_expert_r{int(round(r * 100))}", d=4096, N=14336, dtype=BF16,
                     prompt_tokens=512, decode_steps=steps, ratios=ratios_for(r, 0.1), seed=4)


def config5(batch: int = 1, steps: int = 256) -> FFNConfig:
    """Llama-2-13B-shaped FFN with a VLM-style prompt: 576 visual-patch-like
    rows whose hidden channels have heavy-tailed scales, then 128 text rows."""
    return FFNConfig(f"cfg5_llama13b_vlm_b{batch}", d=5120, N=13824, dtype=BF16,
                     prompt_tokens=704, decode_steps=steps, batch=batch,
                     ratios=ratios_for(0.4, 0.1), seed=5, activation="vlm", visual_tokens=576)


def scaled(cfg: FFNConfig, **kw) -> FFNConfig:
    """A copy of ``cfg`` with some fields replaced (reduced test sizes)."""
    d = dict(cfg.__dict__)
    d.update(kw)
    return FFNConfig(**d)


# --------------------------------------------------------------------------- generators
@dataclass
class FFNWeights:
    Wg: Array      # [N, d]  gate projection, row i = channel i
    Wu: Array      # [N, d]  up projection
    Wd: Array      # [d, N]  down projection, column i = channel i


def make_weights(N: int, d: int, dtype: str, seed: int, std: float = 0.02) -> FFNWeights:
    rng = np.random.Generator(np.random.PCG64([seed, 101]))
    Wg = rng.standard_normal((N, d), dtype=np.float32) * np.float32(std)
    Wu = rng.standard_normal((N, d), dtype=np.float32) * np.float32(std)
    Wd = rng.standard_normal((d, N), dtype=np.float32) * np.float32(std)
    return FFNWeights(as_array(Wg, dtype), as_array(Wu, dtype), as_array(Wd, dtype))


def make_prompt(cfg: FFNConfig, prompt_id: int = 0) -> np.ndarray:
    """fp32 [L, d] prompt activations feeding the FFN (before dtype rounding)."""
    rng = np.random.Generator(np.random.PCG64([cfg.seed, 202, prompt_id]))
    L, d = cfg.prompt_tokens, cfg.d
    X = rng.standard_normal((L, d), dtype=np.float32)
    if cfg.activation == "vlm":
        # visual rows: per-hidden-channel scale a_c = |t_3| drawn once (a few
        # massive channels), times N(0,1); the trailing text rows stay N(0,1).
        a = np.abs(rng.standard_t(3.0, size=d)).astype(np.float32)
        nv = min(cfg.visual_tokens, L)
        X[:nv] *= a[None, :]
    elif cfg.activation != "normal":
        raise ValueError(cfg.activation)
    return X


def make_prefill_input(cfg: FFNConfig) -> Array:
    """Prompt activations with the batch folded into the token axis: [B*L, d]."""
    Xs = [make_prompt(cfg, p) for p in range(cfg.batch)]
    return as_array(np.concatenate(Xs, axis=0), cfg.dtype)


def make_decode_inputs(cfg: FFNConfig, steps: Optional[int] = None) -> Array:
    """Step-wise FFN inputs x_t, [steps, B, d] ~ N(0,1), different at every step."""
    steps = cfg.decode_steps if steps is None else steps
    rng = np.random.Generator(np.random.PCG64([cfg.seed, 303]))
    x = rng.standard_normal((steps, cfg.batch, cfg.d), dtype=np.float32)
    return as_array(x, cfg.dtype)


@dataclass
class FFNWorkload:
    cfg: FFNConfig
    weights: FFNWeights
    X: Array            # [B*L, d]
    xs: Array           # [steps, B, d]


def make_ffn_workload(cfg: FFNConfig, steps: Optional[int] = None) -> FFNWorkload:
    return FFNWorkload(cfg, make_weights(cfg.N, cfg.d, cfg.dtype, cfg.seed, cfg.weight_std),
                       make_prefill_input(cfg), make_decode_inputs(cfg, steps))


def make_adversarial_case(kind: str, d: int, N: int, L: int, steps: int, batch: int = 1, seed: int = 0) -> FFNWorkload:
    """Inputs built to strain reduced-precision accumulation (they only draw and arrange numbers):
      "heavy_tail"        activations scaled per hidden channel by |t_3| (a few massive channels), at prefill AND at
                          every decode step, the last step i.i.d. t_3;
      "cancellation"      gate / up rows whose first half is about +c and second half about -c against activations
                          near 1: partial sums of several hundred that cancel to order one;
      "mixed_magnitudes"  activations alternating between about 1e-3 and about 1e3 along the hidden axis.
    """
    rng = np.random.Generator(np.random.PCG64([seed, 909]))
    cfg = FFNConfig(f"adv_{kind}", d=d, N=N, dtype=BF16, prompt_tokens=L, decode_steps=steps, batch=batch,
                    ratios=Ratios(0.45, 0.25, 0.30), seed=seed)
    Wg = rng.standard_normal((N, d), dtype=np.float32) * np.float32(0.02)
    Wu = rng.standard_normal((N, d), dtype=np.float32) * np.float32(0.02)
    Wd = rng.standard_normal((d, N), dtype=np.float32) * np.float32(0.02)
    X = rng.standard_normal((L * batch, d), dtype=np.float32)
    xs = rng.standard_normal((steps, batch, d), dtype=np.float32)
    if kind == "heavy_tail":
        a = np.abs(rng.standard_t(3.0, size=d)).astype(np.float32)
        X *= a[None, :]
        xs *= a[None, None, :]
        xs[-1] = rng.standard_t(3.0, size=(batch, d)).astype(np.float32)
    elif kind == "cancellation":
        sign = np.where(np.arange(d) < d // 2, 1.0, -1.0).astype(np.float32)
        Wg = Wg + np.float32(0.5) * sign[None, :]
        Wu = Wu + np.float32(0.25) * sign[None, :]
        X = np.float32(1.0) + np.float32(0.01) * X
        xs = np.float32(1.0) + np.float32(0.01) * xs
    elif kind == "mixed_magnitudes":
        scale = np.where(np.arange(d) % 2 == 0, 1e-3, 1e3).astype(np.float32)
        X *= scale[None, :]
        xs *= scale[None, None, :]
    else:
        raise ValueError(kind)
    return FFNWorkload(cfg, FFNWeights(as_array(Wg, BF16), as_array(Wu, BF16), as_array(Wd, BF16)),
                       as_array(X, BF16), as_array(xs, BF16))


# --------------------------------------------------------------------------- MoE layer (config 4)
@dataclass
class MoEWorkload:
    cfg: FFNConfig                  # per-expert FFN shape
    n_experts: int
    top_k: int
    experts: List[FFNWeights]
    X: Array                        # [L, d] prompt activations
    xs: Array                       # [steps, 1, d]
    prompt_logits: np.ndarray       # [L, E] fp32 router logits ~ N(0,1)
    decode_logits: np.ndarray       # [steps, E]


def make_moe_workload(cfg: FFNConfig, n_experts: int = 8, top_k: int = 2,
                      steps: Optional[int] = None) -> MoEWorkload:
    steps = cfg.decode_steps if steps is None else steps
    experts = [make_weights(cfg.N, cfg.d, cfg.dtype, cfg.seed * 1000 + 7 * e + 1, cfg.weight_std)
               for e in range(n_experts)]
    rng = np.random.Generator(np.random.PCG64([cfg.seed, 404]))
    pl = rng.standard_normal((cfg.prompt_tokens, n_experts), dtype=np.float32)
    dl = rng.standard_normal((steps, n_experts), dtype=np.float32)
    return MoEWorkload(cfg, n_experts, top_k, experts, make_prefill_input(cfg),
                       make_decode_inputs(cfg, steps), pl, dl)


# --------------------------------------------------------------------------- adversarial small cases
def make_tie_case(N: int = 48, d: int = 16, L: int = 8, seed: int = 7, dtype: str = F32) -> FFNWorkload:
    """A small layer with duplicated channels (exact score ties) and a few
    all-zero channels (zero scores), to exercise the index tie-break."""
    cfg = FFNConfig("ties", d=d, N=N, dtype=dtype, prompt_tokens=L, decode_steps=4,
                    ratios=Ratios(0.25, 0.5, 0.25), seed=seed)
    w = make_weights(N, d, dtype, seed)
    Wg, Wu, Wd = (np.array(a.values) for a in (w.Wg, w.Wu, w.Wd))
    for src, dst in ((1, 5), (1, 9), (2, 30), (7, 8), (20, 41)):
        Wg[dst] = Wg[src]; Wu[dst] = Wu[src]; Wd[:, dst] = Wd[:, src]
    for z in (0, 13, 47):
        Wg[z] = 0.0
    weights = FFNWeights(as_array(Wg, dtype), as_array(Wu, dtype), as_array(Wd, dtype))
    return FFNWorkload(cfg, weights, make_prefill_input(cfg), make_decode_inputs(cfg))
