"""Pins for the CPU oracle: each test ties one part of oracle/pop_oracle.py to
something other than the oracle itself - a library routine, a closed form, a
hand-worked example, brute force, or an invariant the paper states."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import pop_oracle as po
from paper_2602_06822_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def small(N=96, d=40, L=24, B=1, seed=3, dtype=wl.F32, ratios=wl.Ratios(0.3, 0.4, 0.3)):
    cfg = wl.FFNConfig("t", d=d, N=N, dtype=dtype, prompt_tokens=L, decode_steps=3, batch=B,
                       ratios=ratios, seed=seed)
    return wl.make_ffn_workload(cfg)


def W(w):
    return w.weights.Wg.values, w.weights.Wu.values, w.weights.Wd.values


# ------------------------------------------------------------------ dense FFN == library SwiGLU
def test_dense_ffn_matches_torch_library():
    w = small(B=3)
    Wg, Wu, Wd = W(w)
    x = w.xs.values[0]
    tx = torch.from_numpy(np.asarray(x, dtype=np.float64))
    tg, tu, td = (torch.from_numpy(np.asarray(a, dtype=np.float64)) for a in (Wg, Wu, Wd))
    ref = torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(tx, tg)) * torch.nn.functional.linear(tx, tu), td)
    got = po.dense_ffn(x, Wg, Wu, Wd)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-12, atol=1e-15)


def test_zero_pruning_reproduces_dense_ffn():
    w = small(B=2)
    Wg, Wu, Wd = W(w)
    part = po.prefill_partition(w.X.values, Wg, Wu, Wd, (1.0, 0.0, 0.0))
    assert part["R"].tolist() == list(range(w.cfg.N)) and part["C"].size == 0 and part["P"].size == 0
    for x in w.xs.values:
        out = po.decode_step(x, Wg, Wu, Wd, part["R"], part["C"], 0)
        np.testing.assert_allclose(out["y"], po.dense_ffn(x, Wg, Wu, Wd), rtol=1e-12, atol=1e-16)


def test_k_extremes_reduce_to_restricted_ffn():
    w = small()
    Wg, Wu, Wd = W(w)
    part = po.prefill_partition(w.X.values, Wg, Wu, Wd, w.cfg.ratios.astuple())
    R, C = part["R"], part["C"]
    x = w.xs.values[0]
    tW = [torch.from_numpy(np.asarray(a, dtype=np.float64)) for a in (Wg, Wu, Wd)]
    tx = torch.from_numpy(np.asarray(x, dtype=np.float64))

    def lib(act):
        act = torch.from_numpy(np.asarray(act, dtype=np.int64))
        h = torch.nn.functional.silu(tx @ tW[0][act].T) * (tx @ tW[1][act].T)
        return (h @ tW[2][:, act].T).numpy()

    full = po.decode_step(x, Wg, Wu, Wd, R, C, C.size)
    np.testing.assert_allclose(full["y"], lib(np.sort(np.concatenate([R, C]))), rtol=1e-11, atol=1e-15)
    assert full["mask"].all()
    none = po.decode_step(x, Wg, Wu, Wd, R, C, 0)
    np.testing.assert_allclose(none["y"], lib(R), rtol=1e-11, atol=1e-15)
    assert not none["mask"].any() and none["sel"].size == 0


# ------------------------------------------------------------------ Eq. 3 closed forms
def test_eq3_factorises_into_activation_norm_times_column_norm():
    w = small(B=1)
    Wg, Wu, Wd = W(w)
    H = po.intermediate(w.X.values, Wg, Wu)
    I = po.prefill_scores(w.X.values, Wg, Wu, Wd)
    s = np.linalg.norm(H, axis=0)
    n = np.linalg.norm(np.asarray(Wd, dtype=np.float64), axis=0)
    np.testing.assert_allclose(I, s * n, rtol=1e-13)
    # element-level statement: I_i^2 = sum_t sum_j (Wd[j,i] * H[t,i])^2
    i = 17
    brute = math.sqrt(sum((float(Wd[j, i]) * float(H[t, i])) ** 2 for t in range(H.shape[0]) for j in range(Wd.shape[0])))
    assert abs(I[i] - brute) <= 1e-12 * brute


def test_decode_score_is_column_norm_times_abs_h_at_batch_one():
    w = small()
    Wg, Wu, Wd = W(w)
    part = po.prefill_partition(w.X.values, Wg, Wu, Wd, w.cfg.ratios.astuple())
    out = po.decode_step(w.xs.values[0, 0], Wg, Wu, Wd, part["R"], part["C"], 5)
    n = np.linalg.norm(np.asarray(Wd, dtype=np.float64)[:, part["C"]], axis=0)
    np.testing.assert_allclose(out["scores"], n * np.abs(out["H_C"][0]), rtol=1e-13)


def test_batch_norm_runs_over_batch_and_sequence():
    # Eq. 3: s_k = ||X[:, :, k]||_2 - folding the batch into the token axis must not matter.
    w = small(B=2, L=10)
    Wg, Wu, Wd = W(w)
    X = w.X.values
    I_all = po.prefill_scores(X, Wg, Wu, Wd)
    I_a = po.prefill_scores(X[:10], Wg, Wu, Wd)
    I_b = po.prefill_scores(X[10:], Wg, Wu, Wd)
    np.testing.assert_allclose(I_all ** 2, I_a ** 2 + I_b ** 2, rtol=1e-12)


# ------------------------------------------------------------------ hand-worked example
def _gold(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split(":", 1)
            rows = [[float(t) for t in r.split()] for r in val.split(";")]
            out[key.strip()] = np.array(rows if len(rows) > 1 else rows[0])
    return out


def test_hand_worked_example():
    g = _gold(os.path.join(GOLD, "hand_case.txt"))
    a = math.log(3.0)
    a2 = a * a
    Wg, Wu, Wd = g["Wg"], g["Wu"], g["Wd"]
    X = g["X_over_a"] * a
    H = po.intermediate(X, Wg, Wu)
    np.testing.assert_allclose(H, g["H_over_a2"] * a2, rtol=1e-13, atol=1e-15)
    part = po.prefill_partition(X, Wg, Wu, Wd, g["ratios"])
    np.testing.assert_allclose(part["scores"] ** 2, g["I2_over_a4"] * a2 * a2, rtol=1e-13)
    assert part["R"].tolist() == g["R"].astype(int).tolist()
    assert part["C"].tolist() == g["C"].astype(int).tolist()
    assert part["P"].tolist() == g["P"].astype(int).tolist()
    R, C = part["R"], part["C"]
    x1 = g["x1_over_a"] * a
    o = po.decode_step(x1, Wg, Wu, Wd, R, C, 1)
    np.testing.assert_allclose(o["H_R"][0], g["h1_over_a2_R"] * a2, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(o["H_C"][0], g["h1_over_a2_C"] * a2, rtol=1e-13)
    np.testing.assert_allclose(o["scores"], g["score1_over_a2"] * a2, rtol=1e-13)
    assert o["mask"].tolist() == g["k1_mask"].astype(int).tolist()
    assert o["sel"].tolist() == [int(g["k1_sel"][0])]
    np.testing.assert_allclose(o["y"], g["y1_k1_over_a2"] * a2, rtol=1e-13)
    np.testing.assert_allclose(po.decode_step(x1, Wg, Wu, Wd, R, C, 2)["y"], g["y1_k2_over_a2"] * a2, rtol=1e-13)
    np.testing.assert_allclose(po.decode_step(x1, Wg, Wu, Wd, R, C, 0)["y"], g["y1_k0_over_a2"] * a2, rtol=1e-13)
    x2 = g["x2_over_a"] * a
    o2 = po.decode_step(x2, Wg, Wu, Wd, R, C, 1)
    np.testing.assert_allclose(o2["scores"] ** 2, g["score2_sq_over_a4"] * a2 * a2, rtol=1e-13)
    np.testing.assert_allclose(o2["y"], g["y2_k1_over_a2"] * a2, rtol=1e-13)


# ------------------------------------------------------------------ regions
@pytest.mark.parametrize("N,ratios", [
    (1376, (0.30, 0.40, 0.30)), (11008, (0.75, 0.10, 0.15)), (11008, (0.55, 0.10, 0.35)),
    (14336, (0.75, 0.10, 0.15)), (14336, (0.55, 0.10, 0.35)), (13824, (0.55, 0.10, 0.35)),
    (97, (0.5, 0.25, 0.25)), (7, (0.0, 1.0, 0.0)), (5, (1.0, 0.0, 0.0)),
])
def test_region_sizes_follow_the_ratios(N, ratios):
    n_R, n_C, n_P = po.region_sizes(N, ratios)
    assert n_R + n_C + n_P == N
    assert abs(n_C - ratios[1] * N) < 1 and abs(n_P - ratios[2] * N) < 1 and abs(n_R - ratios[0] * N) < 2
    assert n_C == math.floor(ratios[1] * N + 1e-9) and n_P == math.floor(ratios[2] * N + 1e-9)


def test_region_sizes_at_the_benchmark_shapes():
    # sizes quoted in the design notes for the five workloads
    assert po.region_sizes(1376, (0.30, 0.40, 0.30)) == (414, 550, 412)
    assert po.region_sizes(11008, po.default_ratios(0.2)) == (8257, 1100, 1651)
    assert po.region_sizes(11008, po.default_ratios(0.4)) == (6056, 1100, 3852)
    assert po.region_sizes(14336, po.default_ratios(0.2)) == (10753, 1433, 2150)
    assert po.region_sizes(13824, po.default_ratios(0.4)) == (7604, 1382, 4838)


def test_regions_are_disjoint_exhaustive_and_ordered_by_threshold():
    w = small(N=257, d=24, L=16)
    Wg, Wu, Wd = W(w)
    part = po.prefill_partition(w.X.values, Wg, Wu, Wd, (0.45, 0.2, 0.35))
    R, C, P, I = part["R"], part["C"], part["P"], part["scores"]
    allc = np.concatenate([R, C, P])
    assert np.array_equal(np.sort(allc), np.arange(257))
    for a in (R, C, P):
        assert np.all(np.diff(a) > 0)
    # threshold form of Sec. 3.3: R >= tau_high > C > tau_low >= P
    assert I[R].min() > I[C].max() and I[C].min() > I[P].max()
    # quantile form: tau_low / tau_high are order statistics of the scores
    srt = np.sort(I)
    assert I[P].max() == srt[P.size - 1] and I[R].min() == srt[257 - R.size]


def test_bad_ratios_rejected():
    with pytest.raises(ValueError):
        po.region_sizes(10, (0.5, 0.5, 0.5))
    with pytest.raises(ValueError):
        po.region_sizes(10, (-0.1, 0.5, 0.5))


# ------------------------------------------------------------------ top-k by brute force
def test_selection_matches_brute_force_sort_with_ties():
    rng = np.random.default_rng(11)
    for trial in range(200):
        n = int(rng.integers(1, 13))
        C = np.sort(rng.choice(40, size=n, replace=False))
        scores = rng.integers(0, 4, size=n).astype(np.float64)     # many exact ties
        k = int(rng.integers(0, n + 1))
        mask, sel = po.select_candidates(scores, C, k)
        ranked = sorted(range(n), key=lambda j: (-scores[j], C[j]))
        want = sorted(int(C[j]) for j in ranked[:k])
        assert sel.tolist() == want
        assert mask.sum() == k and [int(c) for c, m in zip(C, mask) if m] == want


def test_partition_matches_brute_force_sort_with_ties():
    rng = np.random.default_rng(12)
    for trial in range(100):
        N = int(rng.integers(3, 30))
        I = rng.integers(0, 5, size=N).astype(np.float64)
        ratios = (0.4, 0.3, 0.3)
        n_R, n_C, n_P = po.region_sizes(N, ratios)
        ranked = sorted(range(N), key=lambda i: (-I[i], i))
        R, C, P = po.partition_from_scores(I, ratios)
        assert R.tolist() == sorted(ranked[:n_R])
        assert C.tolist() == sorted(ranked[n_R:n_R + n_C])
        assert P.tolist() == sorted(ranked[n_R + n_C:])


def test_tie_case_prefers_lower_channel_index():
    w = wl.make_tie_case()
    Wg, Wu, Wd = W(w)
    I = po.prefill_scores(w.X.values, Wg, Wu, Wd)
    assert I[1] == I[5] == I[9] and I[0] == 0.0 and I[13] == 0.0 and I[47] == 0.0
    R, C, P = po.partition_from_scores(I, w.cfg.ratios.astuple())
    region = np.empty(w.cfg.N, dtype=int)
    region[R], region[C], region[P] = 0, 1, 2
    # equal scores: the lower id never lands in a worse region than the higher id
    for lo, hi in ((1, 5), (5, 9), (2, 30), (7, 8), (20, 41), (0, 13), (13, 47)):
        assert region[lo] <= region[hi]


# ------------------------------------------------------------------ whole-method properties
def test_permuting_channels_permutes_indices_and_keeps_outputs():
    w = small(N=64, d=32, L=12)
    Wg, Wu, Wd = W(w)
    perm = np.random.default_rng(5).permutation(64)
    inv = np.argsort(perm)
    Wg2, Wu2, Wd2 = Wg[perm], Wu[perm], Wd[:, perm]
    ratios = (0.4, 0.3, 0.3)
    p1 = po.prefill_partition(w.X.values, Wg, Wu, Wd, ratios)
    p2 = po.prefill_partition(w.X.values, Wg2, Wu2, Wd2, ratios)
    np.testing.assert_allclose(p2["scores"], p1["scores"][perm], rtol=1e-13)
    for key in ("R", "C", "P"):
        assert sorted(perm[p2[key]].tolist()) == p1[key].tolist()
    x = w.xs.values[1, 0]
    o1 = po.decode_step(x, Wg, Wu, Wd, p1["R"], p1["C"], 9)
    o2 = po.decode_step(x, Wg2, Wu2, Wd2, p2["R"], p2["C"], 9)
    assert sorted(perm[o2["sel"]].tolist()) == o1["sel"].tolist()
    np.testing.assert_allclose(o2["y"], o1["y"], rtol=1e-10, atol=1e-14)


def test_active_count_matches_target_ratio():
    # Sec. 3.3: the number of active channels per step matches the pruning ratio r.
    N, r = 11008, 0.2
    n_R, n_C, n_P = po.region_sizes(N, po.default_ratios(r, 0.1))
    k = po.default_k(n_C)
    assert abs((n_R + k) - (1 - r) * N) <= 1.5


def test_variant2_all_channels_rescored_is_global_topk():
    # Ablation Variant (2): every channel is a candidate; the step keeps the
    # top (1-r)N channels by this step's own score.
    w = small(N=80, d=32, L=12)
    Wg, Wu, Wd = W(w)
    part = po.prefill_partition(w.X.values, Wg, Wu, Wd, (0.0, 1.0, 0.0))
    assert part["C"].size == 80 and part["R"].size == 0
    x = w.xs.values[0, 0]
    k = 80 - int(0.25 * 80)
    out = po.decode_step(x, Wg, Wu, Wd, part["R"], part["C"], k)
    h = po.intermediate(x, Wg, Wu)[0]
    n = np.linalg.norm(np.asarray(Wd, dtype=np.float64), axis=0)
    want = np.sort(np.argsort(-(n * np.abs(h)), kind="stable")[:k])
    assert out["sel"].tolist() == want.tolist()
    np.testing.assert_allclose(out["y"], (np.asarray(Wd, np.float64)[:, want] * h[want]).sum(axis=1), rtol=1e-10)


def test_variant1_static_mask_is_topk_of_prefill_scores():
    # Ablation Variant (1): the prefill mask reused; equals the top (n_R + k) channels by prefill score.
    w = small(N=90, d=32, L=12)
    Wg, Wu, Wd = W(w)
    part = po.prefill_partition(w.X.values, Wg, Wu, Wd, (0.5, 0.2, 0.3))
    k = 9
    _, sel = po.static_selection(part["scores"], part["C"], k)
    active = np.sort(np.concatenate([part["R"], sel]))
    top = np.sort(np.argsort(-part["scores"], kind="stable")[:part["R"].size + k])
    assert active.tolist() == top.tolist()
    Y = po.prefill_output(w.X.values, Wg, Wu, Wd, part["R"], part["C"], part["scores"], k)
    np.testing.assert_allclose(Y, po.masked_ffn(w.X.values, Wg, Wu, Wd, top), rtol=1e-12)


def test_scoring_overhead_matches_table5():
    # Table 5: online scoring costs 2.85 % (Llama-2-7B) / 3.48 % (Llama-3.1-8B) of the
    # FFN FLOPs at gamma = 0.1, and 33.1 % / 33.3 % when all channels are re-scored.
    with open(os.path.join(GOLD, "table5_overhead.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for model, N, pop_pct, all_pct in rows:
        N = int(N)
        n_C = po.region_sizes(N, po.default_ratios(0.2, 0.1))[1]
        assert abs(100 * po.scoring_overhead_fraction(N, N) - float(all_pct)) < 0.5
        assert abs(100 * po.scoring_overhead_fraction(N, n_C) - float(pop_pct)) < 0.6
        # gamma = 2 * delta reading: the ratio of the two overheads is the candidate fraction
        assert abs(float(pop_pct) / float(all_pct) - 0.1) < 0.02


# ------------------------------------------------------------------ MoE routing
def test_moe_route_matches_torch_softmax_topk():
    rng = np.random.default_rng(2)
    logits = rng.standard_normal((50, 8))
    ids, wts = po.moe_route(logits, 2)
    p = torch.softmax(torch.from_numpy(logits), dim=-1)
    tv, ti = torch.topk(p, 2, dim=-1)
    assert np.array_equal(ids, ti.numpy())
    np.testing.assert_allclose(wts, (tv / tv.sum(-1, keepdim=True)).numpy(), rtol=1e-12)
    # exact tie -> lower expert id first
    ids2, _ = po.moe_route(np.array([[0.0, 1.0, 1.0, -1.0]]), 2)
    assert ids2.tolist() == [[1, 2]]


def test_moe_partitions_use_only_routed_tokens():
    cfg = wl.FFNConfig("m", d=24, N=40, dtype=wl.F32, prompt_tokens=30, decode_steps=2, seed=9,
                       ratios=wl.Ratios(0.5, 0.25, 0.25))
    m = wl.make_moe_workload(cfg, n_experts=4, top_k=2)
    ex = [(e.Wg.values, e.Wu.values, e.Wd.values) for e in m.experts]
    parts = po.moe_prefill_partitions(m.X.values, ex, m.prompt_logits, cfg.ratios.astuple(), 2)
    ids, _ = po.moe_route(m.prompt_logits, 2)
    assert sum(p["tokens"].size for p in parts) == 2 * 30
    for e, p in enumerate(parts):
        assert all(e in ids[t] for t in p["tokens"])
        ref = po.prefill_partition(m.X.values[p["tokens"]], *ex[e], cfg.ratios.astuple())
        assert np.array_equal(ref["R"], p["R"]) and np.array_equal(ref["C"], p["C"])
    out = po.moe_decode_step(m.xs.values[0, 0], ex, parts, m.decode_logits[0], 5, 2)
    e0, e1 = out["experts"]
    y = out["weights"][0] * po.decode_step(m.xs.values[0, 0], *ex[e0], parts[e0]["R"], parts[e0]["C"], 5)["y"] \
        + out["weights"][1] * po.decode_step(m.xs.values[0, 0], *ex[e1], parts[e1]["R"], parts[e1]["C"], 5)["y"]
    np.testing.assert_allclose(out["y"], y, rtol=1e-13)


# ------------------------------------------------------------------ planted mistakes (in the oracle, on the CPU)
@pytest.mark.parametrize("mutation", ["relu_for_silu", "drop_gate", "norm_l1", "ascending_rank", "score_without_weight"])
def test_pins_catch_planted_mistakes(monkeypatch, mutation):
    """Each plausible mistake, planted into the oracle, must fail the hand-worked example."""
    if mutation == "relu_for_silu":
        monkeypatch.setattr(po, "silu", lambda z: np.maximum(np.asarray(z, dtype=np.float64), 0.0))
    elif mutation == "drop_gate":
        monkeypatch.setattr(po, "silu", lambda z: np.ones_like(np.asarray(z, dtype=np.float64)))
    elif mutation == "norm_l1":
        monkeypatch.setattr(po, "activation_norms", lambda H: np.abs(np.asarray(H, np.float64)).reshape(-1, H.shape[-1]).sum(axis=0))
    elif mutation == "ascending_rank":
        orig = po.rank_order
        monkeypatch.setattr(po, "rank_order", lambda s, ids=None: orig(-np.asarray(s, np.float64), ids))
    elif mutation == "score_without_weight":
        monkeypatch.setattr(po, "channel_importance", lambda Wc, s: np.asarray(s, np.float64))
    with pytest.raises(AssertionError):
        test_hand_worked_example()


def test_partial_probing_is_the_statistic_over_the_probe_tokens():
    """Reading of Sec. 3.4 "partial probing": every s-th token.  Stride 1 is the whole prompt; a stride of L leaves the
    first token alone, for which Eq. 3 is |h_i(x_0)| * |Wd[:, i]| written out; a channel that is active only on skipped
    tokens scores zero."""
    rng = np.random.default_rng(5)
    L, d, N = 9, 6, 12
    X = rng.standard_normal((L, d)); Wg = rng.standard_normal((N, d)); Wu = rng.standard_normal((N, d)); Wd = rng.standard_normal((d, N))
    ratios = (0.5, 0.25, 0.25)
    full = po.prefill_partition(X, Wg, Wu, Wd, ratios)
    one = po.prefill_partition_probe(X, Wg, Wu, Wd, ratios, 1)
    assert np.array_equal(full["scores"], one["scores"]) and np.array_equal(one["tokens"], np.arange(L))
    first = po.prefill_partition_probe(X, Wg, Wu, Wd, ratios, L)
    g, u = Wg @ X[0], Wu @ X[0]
    h = g / (1.0 + np.exp(-g)) * u
    assert np.allclose(first["scores"], np.abs(h) * np.linalg.norm(Wd, axis=0), rtol=1e-12)
    assert np.array_equal(first["tokens"], [0])
    third = po.prefill_partition_probe(X, Wg, Wu, Wd, ratios, 3)
    assert np.array_equal(third["tokens"], [0, 3, 6])
    Xz = X.copy(); Xz[[0, 3, 6]] = 0.0                      # the probe tokens silent: every score is zero
    assert np.all(po.prefill_partition_probe(Xz, Wg, Wu, Wd, ratios, 3)["scores"] == 0.0)
    assert np.any(po.prefill_partition(Xz, Wg, Wu, Wd, ratios)["scores"] > 0.0)
    with pytest.raises(ValueError):
        po.prefill_partition_probe(X, Wg, Wu, Wd, ratios, 0)
