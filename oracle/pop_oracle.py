"""CPU oracle for POP (partition-guided online pruning) of a SwiGLU FFN block.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
method computes; it exists so that the CUDA library can be checked against it.
Nothing in the product path may import it (only the tests, the smoke check and
the benchmark's CPU-baseline leg do), and it imports nothing from the CUDA
package.  Everything is numpy in float64; a matrix product (``@``) and a stable
sort are the only library primitives used as steps.

POP is a heuristic that defines its own result, so the functions below take the
paper's steps in the paper's order:

  prefill (Sec. 3.3 "Prefilling Stage", Sec. 3.4 Eq. 3)
    H   = f(X)                     intermediate activations of the whole prompt
    s_i = || H[:, :, i] ||_2       norm over batch and sequence          (Eq. 3, right)
    I_i = || W[:, i] (.) s ||_2    W = the linear layer that consumes H  (Eq. 3, left)
    R, C, P from the quantile band around the pruning threshold     (Sec. 3.3)
  decode step t (Sec. 3.3 "Decoding Stage", Sec. 3.4 last paragraph)
    H_t  = f(X_t; R u C)           forward over retained + candidate channels
    I_i(t) for i in C only         same formula, evaluated from H_t
    pick candidates so that the active count matches the target ratio
    final computation over R u selected only

Notation: d hidden size, N intermediate size; the prunable *channels* are the N
intermediate dimensions (Sec. 3.1, last paragraph: an FFN "output channel" is one
dimension of the intermediate representation shared by consecutive linear
layers).  Wg, Wu are [N, d] (row i = channel i), Wd is [d, N] (column i =
channel i).  f(x) = silu(Wg x) * (Wu x)  (SwiGLU; the paper writes a generic f).

Readings taken where the paper is silent or garbled (each also listed in the
design notes of the repository):

 1. Eq. 3 indexes the *column* W[:, i] and multiplies it by a vector indexed by
    the input channel; with W in R^{C_out x C_in} that cannot be an output
    channel of W.  Reading: W is the down projection, whose input channel i is
    the FFN intermediate channel i; s is the per-channel norm of the tensor that
    enters it (H, after activation and gating), broadcast so that
    I_i = sqrt(sum_j (Wd[j, i] * s_i)^2).
 2. gamma ("partition fraction", Sec. 4) versus delta ("partition width",
    Sec. 3.3): gamma = |C| / N = 2 delta.
 3. Quantiles and ties: regions are taken by rank with exact sizes
    n_P = floor(pruned * N + 1e-9), n_C = floor(candidate * N + 1e-9),
    n_R = N - n_P - n_C; identical to the threshold form whenever the two
    boundary scores are distinct.
 4. k (how many candidates are switched on) is an explicit argument; the default
    floor(n_C / 2) centres the active count on the target ratio.
 5. Ties: order by (score descending, channel index ascending).
 6. Batch > 1: Eq. 3's norm runs over batch *and* sequence, so one partition is
    built from all prompt tokens and one mask per step is shared by the batch.
 7. The prefill pass's own output uses R plus the top-k candidates by *prefill*
    score (a static mask at the target ratio; this is also "Variant (1)" of the
    ablation when reused for every decoding step).
 8. MoE: softmax over all router logits, top-2 (ties to the lower expert id),
    renormalised; expert e's partition is built from the prompt tokens routed
    to e, unweighted.

Parity pins (tests/test_oracle_*.py): dense-FFN special case against
torch's CPU linear/silu; closed forms of Eq. 3; a hand-worked 6-channel example
(tests/golden/hand_case.txt); brute-force sorting on tiny inputs; region
invariants; permutation equivariance; Variant (1)/(2) special cases; Table 5's
overhead ratio.  "parity unpinned" (fixed by the readings above only): batch-
shared mask (6), prefill output mask (7), MoE routing of the statistic (8), and
the rounding of k (4).
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=F64)


# ----------------------------------------------------------------------------- FFN pieces
def silu(z: np.ndarray) -> np.ndarray:
    """silu(z) = z / (1 + exp(-z))."""
    z = _f64(z)
    return z / (1.0 + np.exp(-z))


def intermediate(X, Wg, Wu, channels: Optional[np.ndarray] = None) -> np.ndarray:
    """H[t, c] = silu(Wg[i_c] . X[t]) * (Wu[i_c] . X[t]) for the listed channels
    (all N when ``channels`` is None).  Sec. 3.4: H_t = f(X_t; R u C)."""
    X, Wg, Wu = _f64(X), _f64(Wg), _f64(Wu)
    if X.ndim == 1:
        X = X[None, :]
    if channels is not None:
        Wg, Wu = Wg[channels], Wu[channels]
    G = X @ Wg.T
    U = X @ Wu.T
    return silu(G) * U


def dense_ffn(x, Wg, Wu, Wd) -> np.ndarray:
    """Plain SwiGLU FFN, y = Wd (silu(Wg x) * (Wu x)); x is [B, d] or [d]."""
    x = _f64(x)
    one = x.ndim == 1
    H = intermediate(x, Wg, Wu)
    y = H @ _f64(Wd).T
    return y[0] if one else y


def masked_ffn(x, Wg, Wu, Wd, active: np.ndarray) -> np.ndarray:
    """FFN restricted to the channels in ``active`` (ascending ids):
    y[b] = sum_{i in active} Wd[:, i] * h[b, i]."""
    x = _f64(x)
    one = x.ndim == 1
    active = np.asarray(active, dtype=np.int64)
    H = intermediate(x, Wg, Wu, active)
    y = H @ _f64(Wd)[:, active].T
    return y[0] if one else y


# ----------------------------------------------------------------------------- Eq. 3
def activation_norms(H: np.ndarray) -> np.ndarray:
    """s_k = || H[:, :, k] ||_2 over every leading axis (batch and sequence)."""
    H = _f64(H)
    lead = tuple(range(H.ndim - 1))
    return np.sqrt((H * H).sum(axis=lead))


def channel_importance(W_cols: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Eq. 3 under reading 1: I_i = || W[:, i] * s_i ||_2 for the columns given
    (W_cols is [d, n], s is [n])."""
    W_cols, s = _f64(W_cols), _f64(s)
    T = W_cols * s[None, :]
    return np.sqrt((T * T).sum(axis=0))


def prefill_scores(X, Wg, Wu, Wd) -> np.ndarray:
    """I_i for all N channels from the whole prompt X [L, d] (batch folded in)."""
    H = intermediate(X, Wg, Wu)
    return channel_importance(Wd, activation_norms(H))


# ----------------------------------------------------------------------------- regions
def default_ratios(r: float, gamma: float = 0.1) -> Tuple[float, float, float]:
    """(retained, candidate, pruned) fractions for FFN pruning ratio r: the band
    between the (r - delta) and (r + delta) quantiles with gamma = 2 delta."""
    delta = gamma / 2.0
    return (1.0 - r - delta, gamma, r - delta)


def region_sizes(N: int, ratios: Sequence[float]) -> Tuple[int, int, int]:
    """(n_R, n_C, n_P) by reading 3."""
    ret, cand, pruned = (float(v) for v in ratios)
    if min(ret, cand, pruned) < 0 or ret + cand + pruned > 1.0 + 1e-9 or cand + pruned > 1.0 + 1e-9:
        raise ValueError("ratios must be non-negative and sum to at most 1")
    n_P = int(np.floor(pruned * N + 1e-9))
    n_C = int(np.floor(cand * N + 1e-9))
    n_R = N - n_P - n_C
    return n_R, n_C, n_P


def default_k(n_C: int) -> int:
    return n_C // 2


def rank_order(scores: np.ndarray, ids: Optional[np.ndarray] = None) -> np.ndarray:
    """Positions sorted by (score descending, id ascending)."""
    scores = _f64(scores)
    if not np.all(np.isfinite(scores)):
        raise ValueError("non-finite importance score")
    ids = np.arange(scores.shape[0], dtype=np.int64) if ids is None else np.asarray(ids, dtype=np.int64)
    return np.lexsort((ids, -scores))


def partition_from_scores(I: np.ndarray, ratios: Sequence[float]) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """R, C, P (each ascending by channel id) from the importance scores."""
    N = I.shape[0]
    n_R, n_C, n_P = region_sizes(N, ratios)
    order = rank_order(I)
    R = np.sort(order[:n_R]).astype(np.int32)
    C = np.sort(order[n_R:n_R + n_C]).astype(np.int32)
    P = np.sort(order[n_R + n_C:]).astype(np.int32)
    return R, C, P


def prefill_partition(X, Wg, Wu, Wd, ratios: Sequence[float]) -> Dict[str, np.ndarray]:
    """Prefilling stage: scores from the full prompt, then the three regions."""
    I = prefill_scores(X, Wg, Wu, Wd)
    R, C, P = partition_from_scores(I, ratios)
    return {"scores": I, "R": R, "C": C, "P": P}


def prefill_partition_probe(X, Wg, Wu, Wd, ratios: Sequence[float], token_stride: int) -> Dict[str, np.ndarray]:
    """Prefilling stage from "partial probing prompt activations" (Sec. 3.4, which does not define the subset): read as
    every token_stride-th prompt token, rows 0, s, 2s, ... of X.  Eq. 3 over those tokens only; stride 1 is the
    whole prompt."""
    if token_stride < 1:
        raise ValueError("token_stride must be at least 1")
    out = prefill_partition(_f64(X)[::token_stride], Wg, Wu, Wd, ratios)
    out["tokens"] = np.arange(0, np.asarray(X).shape[0], token_stride)
    return out


# ----------------------------------------------------------------------------- decode step
def candidate_scores(H_C: np.ndarray, Wd, C: np.ndarray) -> np.ndarray:
    """I_i(t), i in C, from this step's activations H_C [B, n_C] (Eq. 3 with the
    norm over the batch axis; the sequence axis has length 1)."""
    return channel_importance(_f64(Wd)[:, np.asarray(C, dtype=np.int64)], activation_norms(H_C))


def select_candidates(scores: np.ndarray, C: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Top-k of C by (score descending, channel id ascending).  Returns the mask
    over C's slots (uint8) and the selected channel ids, ascending."""
    C = np.asarray(C, dtype=np.int64)
    if not 0 <= k <= C.shape[0]:
        raise ValueError("k out of range")
    order = rank_order(scores, C)
    mask = np.zeros(C.shape[0], dtype=np.uint8)
    mask[order[:k]] = 1
    return mask, C[mask.astype(bool)].astype(np.int32)


def decode_step(x, Wg, Wu, Wd, R: np.ndarray, C: np.ndarray, k: int) -> Dict[str, np.ndarray]:
    """One decoding step for x [B, d] (or [d]): forward over R u C, score C,
    select k candidates, finish over R u selected."""
    x = _f64(x)
    one = x.ndim == 1
    xb = x[None, :] if one else x
    R = np.asarray(R, dtype=np.int64)
    C = np.asarray(C, dtype=np.int64)
    H_R = intermediate(xb, Wg, Wu, R)                  # [B, n_R]
    H_C = intermediate(xb, Wg, Wu, C)                  # [B, n_C]
    sc = candidate_scores(H_C, Wd, C)
    mask, sel = select_candidates(sc, C, k)
    on = mask.astype(bool)
    active = np.concatenate([R, C[on]])
    H_act = np.concatenate([H_R, H_C[:, on]], axis=1)
    asc = np.argsort(active, kind="stable")            # sum in ascending channel order
    y = H_act[:, asc] @ _f64(Wd)[:, active[asc]].T
    return {"y": y[0] if one else y, "mask": mask, "sel": sel, "scores": sc,
            "H_R": H_R, "H_C": H_C}


# ----------------------------------------------------------------------------- static mask / prefill output (reading 7)
def static_selection(I: np.ndarray, C: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """The k candidates with the largest *prefill* score (Variant (1) of the
    ablation: the mask from prefilling reused at every step)."""
    C = np.asarray(C, dtype=np.int64)
    return select_candidates(_f64(I)[C], C, k)


def prefill_output(X, Wg, Wu, Wd, R, C, I, k: int) -> np.ndarray:
    """The prompt's own FFN output "under the resulting pruning structure"."""
    _, sel = static_selection(I, C, k)
    active = np.sort(np.concatenate([np.asarray(R, dtype=np.int64), sel.astype(np.int64)]))
    return masked_ffn(X, Wg, Wu, Wd, active)


# ----------------------------------------------------------------------------- MoE (reading 8)
def moe_route(logits: np.ndarray, top_k: int = 2) -> Tuple[np.ndarray, np.ndarray]:
    """softmax over all experts, top_k by (prob descending, expert id ascending),
    renormalised.  Returns (expert ids [T, top_k], weights [T, top_k])."""
    z = _f64(logits)
    z = z - z.max(axis=-1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=-1, keepdims=True)
    T, E = p.shape
    ids = np.empty((T, top_k), dtype=np.int64)
    for t in range(T):
        ids[t] = rank_order(p[t])[:top_k]
    w = np.take_along_axis(p, ids, axis=1)
    w /= w.sum(axis=1, keepdims=True)
    return ids, w


def moe_prefill_partitions(X, experts, prompt_logits, ratios, top_k: int = 2):
    """One partition per expert from the prompt tokens routed to it."""
    ids, _ = moe_route(prompt_logits, top_k)
    X = _f64(X)
    parts = []
    for e, (Wg, Wu, Wd) in enumerate(experts):
        tok = np.nonzero((ids == e).any(axis=1))[0]
        parts.append(dict(prefill_partition(X[tok], Wg, Wu, Wd, ratios), tokens=tok))
    return parts


def moe_decode_step(x, experts, parts, logits, k: int, top_k: int = 2):
    """y = sum_e p_e * decode_step_e(x) over the routed experts of one token."""
    ids, w = moe_route(np.asarray(logits)[None, :], top_k)
    y = 0.0
    per = []
    for j in range(top_k):
        e = int(ids[0, j])
        Wg, Wu, Wd = experts[e]
        out = decode_step(x, Wg, Wu, Wd, parts[e]["R"], parts[e]["C"], k)
        y = y + w[0, j] * out["y"]
        per.append((e, float(w[0, j]), out))
    return {"y": y, "experts": ids[0], "weights": w[0], "per_expert": per}


# ----------------------------------------------------------------------------- cost model (Sec. 5, Table 5)
def scoring_overhead_fraction(N: int, n_scored: int) -> float:
    """Multiply-accumulates spent by the literal Eq. 3 evaluation on n_scored
    channels (one pass over d x n_scored entries of the down projection) as a
    fraction of the dense FFN's three d x N projections."""
    return (n_scored / float(N)) / 3.0
