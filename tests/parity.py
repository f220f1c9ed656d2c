"""Helpers shared by the GPU parity tests: upload of seeded inputs, and the comparison rules.

Comparison rules (stated here once, used by every parity test):
  * index sets (regions, selected candidates) must be equal arrays, except that ids may swap
    across a rank boundary when their ORACLE scores lie within 1e-6 relative of the oracle's
    score at that boundary (allowance for near-ties: such scores are equal for every practical purpose);
  * outputs: err_j = |y_j - yref_j| / max(|yref_j|, floor * max_j |yref_j|); max_j err_j must be
    <= 1e-4 for fp32 and <= 2e-2 for bf16.  The floor keeps the measure meaningful for outputs
    that happen to lie near zero, where an fp32 accumulation has an absolute, not a relative,
    error.  bf16 results are gated with floor = 1e-3; fp32 results with floor = 1e-2: an fp32
    accumulation of n products carries an absolute error of about sqrt(n) 2^-24 of the terms'
    root-sum-square, i.e. a few 1e-6 of a typical |y_j|, which measured against 1e-3 of the
    largest output is already of the order of the 1e-4 gate itself.  The full-size tests print the
    worst error under both floors and the normwise error.
"""
import numpy as np
import torch

from paper_2602_06822_b200 import workloads as wl

TOL = {wl.F32: 1e-4, wl.BF16: 2e-2}
FLOOR = {wl.F32: 1e-2, wl.BF16: 1e-3}
SWAP_RTOL = 1e-6


def to_dev(a: wl.Array, dev="cuda:0", index=None):
    raw = a.raw if index is None else a.raw[index]
    t = torch.from_numpy(np.ascontiguousarray(raw))
    if a.dtype == wl.BF16:
        t = t.view(torch.bfloat16)
    return t.to(dev)


def host_values(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_err(y: np.ndarray, yref: np.ndarray, floor: float = 1e-3) -> float:
    yref = np.asarray(yref, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    scale = np.max(np.abs(yref))
    if scale == 0.0:
        return float(np.max(np.abs(y)))
    den = np.maximum(np.abs(yref), floor * scale)
    return float(np.max(np.abs(y - yref) / den))


def bf16_ulp_distance(a: torch.Tensor, b: torch.Tensor) -> int:
    """Largest distance, in bf16 representable values, between corresponding elements of two bf16 tensors."""
    def ordinal(t):
        v = t.contiguous().view(torch.int16).to(torch.int32) & 0xFFFF
        return torch.where(v >= 0x8000, 0x8000 - v, v)          # negative values below zero, in order
    return int((ordinal(a) - ordinal(b)).abs().max())


def normwise_err(y, yref) -> float:
    yref = np.asarray(yref, dtype=np.float64)
    s = np.max(np.abs(yref))
    return float(np.max(np.abs(np.asarray(y, np.float64) - yref)) / (s if s > 0 else 1.0))


def check_set(got: np.ndarray, want: np.ndarray, score_of, boundary_scores, what: str) -> int:
    """Equal sets, up to swaps of ids whose oracle score is within SWAP_RTOL of a boundary score.
    Returns the number of swapped pairs."""
    got = np.asarray(got).astype(np.int64)
    want = np.asarray(want).astype(np.int64)
    assert got.shape == want.shape, f"{what}: size {got.shape} != {want.shape}"
    assert np.all(np.diff(got) > 0), f"{what}: not strictly ascending"
    if np.array_equal(got, want):
        return 0
    diff = np.setxor1d(got, want)
    for i in diff:
        s = score_of(int(i))
        ok = any(abs(s - b) <= SWAP_RTOL * abs(b) for b in boundary_scores)
        assert ok, f"{what}: id {i} differs and its score {s!r} is not within {SWAP_RTOL} of a boundary {boundary_scores}"
    return diff.size // 2


def check_regions(part, ref) -> int:
    """GPU partition (paper_2602_06822_b200.pop.Partition) against the oracle's dict."""
    R, C, P = part.indices()
    I = ref["scores"]
    allc = np.concatenate([R, C, P])
    assert np.array_equal(np.sort(allc), np.arange(I.shape[0])), "regions do not partition the channels"
    bounds = []
    if ref["R"].size and (ref["C"].size or ref["P"].size):
        rest = np.concatenate([ref["C"], ref["P"]])
        bounds += [I[ref["R"]].min(), I[rest].max()]
    if ref["P"].size and (ref["C"].size or ref["R"].size):
        rest = np.concatenate([ref["C"], ref["R"]])
        bounds += [I[ref["P"]].max(), I[rest].min()]
    sw = 0
    for got, key in ((R, "R"), (C, "C"), (P, "P")):
        sw += check_set(got, ref[key], lambda i: I[i], bounds, f"region {key}")
    return sw


def check_selection(sel: np.ndarray, mask: np.ndarray, C: np.ndarray, o: dict, k: int) -> int:
    """GPU mask / selected ids of one step against the oracle's step output `o`."""
    C = np.asarray(C)
    assert mask.shape == (C.size,) and int(mask.sum()) == k
    assert np.array_equal(C[mask.astype(bool)], sel), "mask and sel_out disagree"
    sc = dict(zip(C.tolist(), o["scores"].tolist()))
    on = o["mask"].astype(bool)
    bounds = []
    if 0 < k < C.size:
        bounds = [o["scores"][on].min(), o["scores"][~on].max()]
    return check_set(sel, o["sel"], lambda i: sc[i], bounds, "selected candidates")
