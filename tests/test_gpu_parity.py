"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Regions / masks / selected ids bit-exact (near-tie swaps per tests/parity.py),
outputs within 1e-4 (fp32) / 2e-2 (bf16)."""
import numpy as np
import pytest
import torch

import __graft_entry__ as ge
from oracle import pop_oracle as po
from paper_2602_06822_b200 import pop, workloads as wl
from tests import parity as pr

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    ge.build()
    pop.lib()


@pytest.fixture(autouse=True, params=["fused", "stream"])
def decode_impl(request):
    """Every case runs with both decode kernel families (the choice is made when a partition is created;
    shapes the streaming kernel does not take use the fused / simple kernels either way)."""
    old = pop.set_config(decode_kernel=pop.POP_DECODE_FUSED if request.param == "fused" else pop.POP_DECODE_AUTO)
    yield request.param
    pop.set_config(decode_kernel=old.decode_kernel, launch_mode=old.launch_mode, wait_budget_us=old.wait_budget_us,
                   slab_cache_bytes=old.slab_cache_bytes)


def weights_dev(w):
    return pr.to_dev(w.weights.Wg), pr.to_dev(w.weights.Wu), pr.to_dev(w.weights.Wd)


def weights_host(w):
    return tuple(np.asarray(a.values, dtype=np.float64) for a in (w.weights.Wg, w.weights.Wu, w.weights.Wd))


def check_streamed_bounds(part, o, k):
    """Streaming kernel only: the bound it attaches to every streamed candidate score must cover the distance to
    the exact score (the selection relies on it: Sec. 3.3 ranks by the exact scores), with room to spare."""
    if part.n_cand == 0 or k <= 0 or k >= part.n_cand:
        return                      # nothing is ranked: the kernel does not look at the scores
    try:
        a, m = part.streamed_scores()
    except pop.PopError as e:
        assert e.status == pop.POP_ERR_UNSUPPORTED
        return                      # served by the fused / simple kernels, which score in fp64
    exact = np.asarray(o["scores"], dtype=np.float64)
    err = np.abs(a.astype(np.float64) - exact)
    assert np.all(np.isfinite(m)) and np.all(m >= 0)
    bad = err > m
    assert not bad.any(), f"error bound violated for {int(bad.sum())} candidates (worst ratio {np.max(err / np.maximum(m, 1e-300)):.3g})"
    # the bounds are meant to be loose by a wide factor (the model doubles the worst case twice)
    assert np.max(err / np.maximum(m, 1e-300)) <= 0.25


def check_prefill_scores(part, ref, dtype):
    """Prefill scores (Eq. 3) against the oracle's.  fp32 partitions and every channel the library scored again in
    fp64 (bound 0: the channels near the two rank boundaries) must agree to fp64 rounding; a score streamed through
    the tensor cores must lie within its own bound of the exact score, with room to spare (the regions rely on it)."""
    sc, bd = part.scores(), part.score_bounds()
    exact = np.asarray(ref["scores"], dtype=np.float64)
    assert np.all(np.isfinite(sc)) and np.all(np.isfinite(bd)) and np.all(bd >= 0)
    err = np.abs(sc - exact)
    ex = bd == 0
    if dtype == wl.F32:
        assert ex.all()
    assert np.all(err[ex] <= 1e-9 * exact[ex] + 1e-300), f"exactly scored channels off by {np.max(err[ex] / np.maximum(exact[ex], 1e-300)):.3g}"
    if (~ex).any():
        ratio = float(np.max(err[~ex] / bd[~ex]))
        assert ratio <= 0.25, f"streamed prefill score outside a quarter of its bound (ratio {ratio:.3g})"
    return int(ex.sum())


def run_decode_parity(w, part, R, C, steps, k, Wh, floor=None):
    cfg = w.cfg
    dev = torch.device("cuda:0")
    mask = torch.empty(max(part.n_cand, 1), dtype=torch.uint8, device=dev)[:part.n_cand]
    sel = torch.empty(max(k, 1), dtype=torch.int32, device=dev)[:k]
    worst, swaps = 0.0, 0
    worst_other, worst_norm = 0.0, 0.0
    floor = pr.FLOOR[cfg.dtype] if floor is None else floor
    for t in range(steps):
        x = pr.to_dev(w.xs, index=t)
        mask.fill_(7)
        sel.fill_(-1)
        y = pop.decode_step(part, x, k, mask_out=mask, sel_out=sel)
        torch.cuda.synchronize()
        part.check()                 # a bounded device wait that expired is reported before any comparison
        o = po.decode_step(w.xs.values[t], *Wh, R, C, k)
        m, s = mask.cpu().numpy(), sel.cpu().numpy()
        sw = pr.check_selection(s, m, C, o, k)
        yref = o["y"]
        if sw:   # an allowed near-tie swap: compare y with the oracle run under the GPU's mask
            active = np.sort(np.concatenate([R, s]))
            yref = po.masked_ffn(w.xs.values[t], *Wh, active)
        swaps += sw
        yh = pr.host_values(y)
        worst = max(worst, pr.rel_err(yh, yref, floor))
        worst_other = max(worst_other, pr.rel_err(yh, yref, 1e-3 if floor != 1e-3 else 1e-2))
        worst_norm = max(worst_norm, pr.normwise_err(yh, yref))
        check_streamed_bounds(part, o, k)
    part.check()
    print(f"[{cfg.name} d={cfg.d} N={cfg.N} B={cfg.batch} steps={steps}] worst output error: {worst:.2e} (floor {floor:g}), "
          f"{worst_other:.2e} (floor {1e-3 if floor != 1e-3 else 1e-2:g}), normwise {worst_norm:.2e}; near-tie swaps {swaps}")
    assert worst <= pr.TOL[cfg.dtype], f"max relative output error {worst:.3e}"
    return worst, swaps


def run_case(cfg, steps=None, k=None, check_scores=True):
    w = wl.make_ffn_workload(cfg, steps)
    steps = w.xs.values.shape[0]
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, cfg.ratios.astuple())
    ref = po.prefill_partition(w.X.values, *Wh, cfg.ratios.astuple())
    assert (part.n_ret, part.n_cand, part.n_pruned) == (ref["R"].size, ref["C"].size, ref["P"].size)
    if check_scores:
        check_prefill_scores(part, ref, cfg.dtype)
    pr.check_regions(part, ref)
    R, C, _ = part.indices()
    if k is None:
        k = cfg.k if cfg.k is not None else part.n_cand // 2
    out = run_decode_parity(w, part, R, C, steps, k, Wh)
    part.destroy()
    return out


# ------------------------------------------------------------------ config 1 (full, fp32)
def test_config1_full():
    cfg = wl.config1()
    assert pop.region_sizes(cfg.N, cfg.ratios.astuple()) == (414, 550, 412, 275)
    run_case(cfg)


# ------------------------------------------------------------------ small shapes, several tiles + ragged tails
@pytest.mark.parametrize("d,N,L,B,dtype", [
    (256, 640, 40, 1, wl.BF16),
    (264, 1000, 33, 1, wl.BF16),      # d not a multiple of 256; N, L ragged
    (1024, 1111, 70, 2, wl.BF16),
    (512, 777, 65, 3, wl.BF16),
    (320, 900, 20, 8, wl.BF16),
    (100, 333, 19, 1, wl.F32),
    (768, 1500, 50, 4, wl.F32),
    # bf16 with d a multiple of 1024: tiled layout + streaming kernel (units of 8 / 16 channels, ragged tails)
    (2048, 403, 24, 1, wl.BF16),
    (2048, 777, 17, 2, wl.BF16),
    (2048, 1210, 20, 3, wl.BF16),
    (2048, 650, 12, 4, wl.BF16),
    (2048, 500, 12, 5, wl.BF16),
    (2048, 333, 9, 8, wl.BF16),
    (4096, 1500, 16, 1, wl.BF16),
    (5120, 900, 16, 2, wl.BF16),
    # N a multiple of 8: W_d is repacked by the kernel that stages channel spans in shared memory
    (2048, 1208, 20, 3, wl.BF16),
    (4096, 1504, 16, 1, wl.BF16),
    (1024, 2056, 30, 2, wl.BF16),
])
def test_small_shapes(d, N, L, B, dtype):
    cfg = wl.FFNConfig(f"s{d}x{N}", d=d, N=N, dtype=dtype, prompt_tokens=L, decode_steps=5, batch=B,
                       ratios=wl.Ratios(0.45, 0.25, 0.30), seed=d + N)
    run_case(cfg)


@pytest.mark.parametrize("ratios", [(0.05, 0.25, 0.70), (0.02, 0.08, 0.90), (0.90, 0.05, 0.05)])
def test_sparse_and_dense_retained_regions_tiled(ratios):
    """Few retained channels: the channel span of one group of retained slots is wider than the repacking kernel's
    staging buffer and it reads W_d directly; many: narrow spans."""
    cfg = wl.FFNConfig("span", d=2048, N=4096, dtype=wl.BF16, prompt_tokens=20, decode_steps=3, batch=2,
                       ratios=wl.Ratios(*ratios), seed=29)
    run_case(cfg)


# ------------------------------------------------------------------ degenerate settings
@pytest.mark.parametrize("ratios,kfrac", [
    ((1.0, 0.0, 0.0), 0.0),     # nothing pruned: dense FFN
    ((0.0, 1.0, 0.0), 0.6),     # every channel a candidate (ablation Variant (2))
    ((0.0, 0.5, 0.5), 0.5),     # no retained channels
    ((0.5, 0.0, 0.5), 0.0),     # no candidates: static mask
    ((0.4, 0.3, 0.3), 0.0),     # k = 0
    ((0.4, 0.3, 0.3), 1.0),     # k = n_C
])
@pytest.mark.parametrize("dtype,d", [(wl.F32, 256), (wl.BF16, 256), (wl.BF16, 2048)])
def test_degenerate_regions(ratios, kfrac, dtype, d):
    cfg = wl.FFNConfig("deg", d=d, N=500, dtype=dtype, prompt_tokens=24, decode_steps=3, batch=2,
                       ratios=wl.Ratios(*ratios), seed=17)
    n_C = po.region_sizes(cfg.N, ratios)[1]
    run_case(cfg, k=int(round(kfrac * n_C)))


def test_zero_pruning_equals_dense_ffn_on_gpu():
    cfg = wl.FFNConfig("dense", d=512, N=1376, dtype=wl.F32, prompt_tokens=16, decode_steps=2, batch=1,
                       ratios=wl.Ratios(1.0, 0.0, 0.0), seed=3)
    w = wl.make_ffn_workload(cfg)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, (1.0, 0.0, 0.0))
    x = pr.to_dev(w.xs, index=0)
    y = pop.decode_step(part, x, 0)
    ref = torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(x.double(), Wg.double()))
        * torch.nn.functional.linear(x.double(), Wu.double()), Wd.double())
    assert pr.rel_err(pr.host_values(y), ref.cpu().numpy(), pr.FLOOR[wl.F32]) <= 1e-4
    part.destroy()


@pytest.mark.parametrize("dtype,d", [(wl.F32, 16), (wl.BF16, 2048)])
def test_exact_ties_break_by_lower_channel_index(dtype, d):
    w = wl.make_tie_case(d=d, dtype=dtype)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, w.cfg.ratios.astuple())
    ref = po.prefill_partition(w.X.values, *Wh, w.cfg.ratios.astuple())
    R, C, P = part.indices()
    # exact equality, no allowance: duplicated channels have bit-equal scores on both sides
    assert np.array_equal(R, ref["R"]) and np.array_equal(C, ref["C"]) and np.array_equal(P, ref["P"])
    sc = part.scores()
    assert sc[1] == sc[5] == sc[9] and sc[0] == 0.0 and sc[13] == 0.0
    part.destroy()
    # decode ties: make every channel a candidate so the duplicated channels compete directly
    ret = np.array([3, 4], dtype=np.int32)
    cand = np.array([i for i in range(w.cfg.N) if i not in (3, 4, 40)], dtype=np.int32)
    part = pop.partition_from_indices(Wg, Wu, Wd, ret, cand)
    for k in (0, 1, 7, 20, cand.size - 1, cand.size):
        mask = torch.zeros(cand.size, dtype=torch.uint8, device="cuda:0")
        sel = torch.zeros(max(k, 1), dtype=torch.int32, device="cuda:0")[:k]
        for t in range(w.xs.values.shape[0]):
            y = pop.decode_step(part, pr.to_dev(w.xs, index=t), k, mask_out=mask, sel_out=sel)
            o = po.decode_step(w.xs.values[t], *Wh, ret, cand, k)
            assert np.array_equal(sel.cpu().numpy(), o["sel"])
            assert np.array_equal(mask.cpu().numpy(), o["mask"])
            assert pr.rel_err(pr.host_values(y), o["y"], pr.FLOOR[dtype]) <= pr.TOL[dtype]
    part.check()
    part.destroy()


def test_partition_from_indices_and_argument_errors():
    cfg = wl.FFNConfig("fi", d=128, N=200, dtype=wl.BF16, prompt_tokens=8, decode_steps=2, seed=21)
    w = wl.make_ffn_workload(cfg)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    rng = np.random.default_rng(0)
    perm = rng.permutation(200)
    ret, cand = np.sort(perm[:90]).astype(np.int32), np.sort(perm[90:150]).astype(np.int32)
    part = pop.partition_from_indices(Wg, Wu, Wd, ret, cand)
    R, C, P = part.indices()
    assert np.array_equal(R, ret) and np.array_equal(C, cand) and np.array_equal(P, np.sort(perm[150:]))
    run_decode_parity(w, part, R, C, 2, 30, Wh)
    x = pr.to_dev(w.xs, index=0)
    for bad_k in (-1, 61):
        with pytest.raises(pop.PopError) as e:
            pop.decode_step(part, x, bad_k)
        assert e.value.status == pop.POP_ERR_INVALID_ARG
    with pytest.raises(pop.PopError) as e:
        pop.decode_step(part, torch.zeros(9, 128, dtype=torch.bfloat16, device="cuda:0"), 3)
    assert e.value.status == pop.POP_ERR_UNSUPPORTED
    part.destroy()
    for bad in ((np.array([5, 3], np.int32), cand), (np.array([1, 1], np.int32), cand),
                (np.array([cand[0]], np.int32), cand), (np.array([200], np.int32), cand)):
        with pytest.raises(pop.PopError) as e:
            pop.partition_from_indices(Wg, Wu, Wd, *bad)
        assert e.value.status == pop.POP_ERR_INVALID_ARG
    with pytest.raises(pop.PopError) as e:
        pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, (0.5, 0.6, 0.6))
    assert e.value.status == pop.POP_ERR_INVALID_ARG


@pytest.mark.parametrize("d", [512, 2048])
def test_repeated_steps_are_bit_identical_in_mask_and_within_two_ulps_in_output(d):
    """The same step twice: equal masks, and outputs that differ by at most two bf16 values (the partial sums reach the
    fp32 accumulator in the order the SMs deliver them, so the last bit of an fp32 sum, and with it a rounding to
    bf16, may differ; anything larger would point at a race)."""
    cfg = wl.FFNConfig("rep", d=d, N=1024, dtype=wl.BF16, prompt_tokens=32, decode_steps=1, seed=5)
    w = wl.make_ffn_workload(cfg)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, (0.5, 0.3, 0.2))
    x = pr.to_dev(w.xs, index=0)
    k = part.n_cand // 2
    m1 = torch.zeros(part.n_cand, dtype=torch.uint8, device="cuda:0")
    y1 = pop.decode_step(part, x, k, mask_out=m1).clone()
    for rep in range(8):
        m2 = torch.zeros_like(m1)
        y2 = pop.decode_step(part, x, k, mask_out=m2).clone()
        assert torch.equal(m1, m2)
        assert pr.bf16_ulp_distance(y1, y2) <= 2
    part.destroy()


# ------------------------------------------------------------------ full-size workloads
@pytest.mark.parametrize("r", [0.2, 0.4])
def test_config2_full_size(r, decode_impl):
    cfg = wl.config2(r)
    assert po.region_sizes(cfg.N, cfg.ratios.astuple())[:2] == ((8257, 1100) if r == 0.2 else (6056, 1100))
    run_case(cfg, steps=32 if decode_impl == "stream" else 6)


@pytest.mark.parametrize("batch", [1, 8])
def test_config5_full_size(batch):
    cfg = wl.config5(batch)
    run_case(cfg, steps=3)


# ------------------------------------------------------------------ Mixtral-shaped MoE layer (composition of the two calls)
def run_moe_case(cfg, n_experts, steps):
    """One partition per expert from the prompt tokens routed to it, then per decode token the two routed
    experts' decode steps combined with the renormalised router weights.  The router (softmax, top-2) and the
    weighted sum are harness code in torch; every FFN step goes through the C ABI."""
    m = wl.make_moe_workload(cfg, n_experts=n_experts, top_k=2, steps=steps)
    dev = torch.device("cuda:0")
    ratios = cfg.ratios.astuple()
    ex_host = [tuple(np.asarray(a.values, dtype=np.float64) for a in (e.Wg, e.Wu, e.Wd)) for e in m.experts]
    ref_parts = po.moe_prefill_partitions(m.X.values, ex_host, m.prompt_logits, ratios, 2)
    # harness routing on the device
    pl = torch.from_numpy(m.prompt_logits).to(dev)
    top = torch.topk(torch.softmax(pl.double(), dim=-1), 2, dim=-1).indices
    Xd = pr.to_dev(m.X)
    parts = []
    for e in range(n_experts):
        tok = torch.nonzero((top == e).any(dim=1)).flatten()
        assert np.array_equal(tok.cpu().numpy(), ref_parts[e]["tokens"])
        Wg, Wu, Wd = (pr.to_dev(a) for a in (m.experts[e].Wg, m.experts[e].Wu, m.experts[e].Wd))
        part = pop.prefill_partition(Xd[tok].contiguous(), Wg, Wu, Wd, ratios)
        pr.check_regions(part, ref_parts[e])
        parts.append(part)
        del Wg, Wu, Wd
    k = parts[0].n_cand // 2
    worst = 0.0
    for t in range(steps):
        x = pr.to_dev(m.xs, index=t)
        dl = torch.from_numpy(m.decode_logits[t]).to(dev).double()
        p = torch.softmax(dl, dim=-1)
        wts, ids = torch.topk(p, 2)
        wts = wts / wts.sum()
        o = po.moe_decode_step(m.xs.values[t, 0], ex_host, ref_parts, m.decode_logits[t], k, 2)
        assert np.array_equal(np.sort(ids.cpu().numpy()), np.sort(o["experts"]))
        y = torch.zeros(1, cfg.d, dtype=torch.float64, device=dev)
        for j in range(2):
            e = int(ids[j])
            R, C, _ = parts[e].indices()
            mask = torch.empty(parts[e].n_cand, dtype=torch.uint8, device=dev)
            sel = torch.empty(k, dtype=torch.int32, device=dev)
            ye = pop.decode_step(parts[e], x, k, mask_out=mask, sel_out=sel)
            torch.cuda.synchronize()
            parts[e].check()
            oe = [po_e for po_e in o["per_expert"] if po_e[0] == e][0][2]
            pr.check_selection(sel.cpu().numpy(), mask.cpu().numpy(), C, oe, k)
            assert pr.rel_err(pr.host_values(ye), oe["y"], pr.FLOOR[cfg.dtype]) <= pr.TOL[cfg.dtype]
            y += float(wts[j]) * ye.double()
        # The combined output: every expert output arrives rounded to bf16 (2^-9 of its own magnitude), which is
        # an absolute error for the weighted sum where the experts cancel; it is judged normwise.
        worst = max(worst, pr.normwise_err(y.cpu().numpy()[0], o["y"]))
    assert worst <= 1e-2, f"MoE output error {worst:.3e}"
    for part in parts:
        part.destroy()


def test_moe_batched_decode_groups_tokens_per_expert():
    """Batched MoE decoding: the tokens of one step are grouped by routed expert and every group is one decode
    step of that expert's partition, with one mask per group (candidate energy summed over the group's tokens, as
    for any batch).  Checked group by group against the oracle's batched decode step, and token by token against the
    router-weighted sum of the oracle's group outputs."""
    cfg = wl.FFNConfig("moe_batch", d=2048, N=600, dtype=wl.BF16, prompt_tokens=48, decode_steps=8,
                       ratios=wl.Ratios(0.5, 0.2, 0.3), seed=23)
    n_experts = 4
    m = wl.make_moe_workload(cfg, n_experts=n_experts, top_k=2, steps=8)
    dev = torch.device("cuda:0")
    ratios = cfg.ratios.astuple()
    ex_host = [tuple(np.asarray(a.values, dtype=np.float64) for a in (e.Wg, e.Wu, e.Wd)) for e in m.experts]
    ref_parts = po.moe_prefill_partitions(m.X.values, ex_host, m.prompt_logits, ratios, 2)
    Xd = pr.to_dev(m.X)
    parts = []
    for e in range(n_experts):
        tok = torch.from_numpy(np.asarray(ref_parts[e]["tokens"])).to(dev)
        Wg, Wu, Wd = (pr.to_dev(a) for a in (m.experts[e].Wg, m.experts[e].Wu, m.experts[e].Wd))
        part = pop.prefill_partition(Xd[tok].contiguous(), Wg, Wu, Wd, ratios)
        pr.check_regions(part, ref_parts[e])
        parts.append(part)
    k = parts[0].n_cand // 2
    xs = pr.to_dev(m.xs)[:, 0, :].contiguous()                      # the step's 8 tokens
    xs_host = m.xs.values[:, 0, :]
    ids, wts = po.moe_route(m.decode_logits, 2)                      # [8, 2] expert ids and renormalised weights
    y = torch.zeros(8, cfg.d, dtype=torch.float64, device=dev)
    y_ref = np.zeros((8, cfg.d))
    groups = 0
    for e in range(n_experts):
        tok = np.nonzero((ids == e).any(axis=1))[0]
        if tok.size == 0:
            continue
        groups += 1
        R, C, _ = parts[e].indices()
        mask = torch.empty(parts[e].n_cand, dtype=torch.uint8, device=dev)
        sel = torch.empty(k, dtype=torch.int32, device=dev)
        ye = pop.decode_step(parts[e], xs[torch.from_numpy(tok).to(dev)].contiguous(), k, mask_out=mask, sel_out=sel)
        torch.cuda.synchronize()
        parts[e].check()
        oe = po.decode_step(xs_host[tok], *ex_host[e], ref_parts[e]["R"], ref_parts[e]["C"], k)
        pr.check_selection(sel.cpu().numpy(), mask.cpu().numpy(), C, oe, k)
        assert pr.rel_err(pr.host_values(ye), oe["y"], pr.FLOOR[cfg.dtype]) <= pr.TOL[cfg.dtype]
        for g, t in enumerate(tok):
            wt = float(wts[t][ids[t] == e][0])
            y[t] += wt * ye[g].double()
            y_ref[t] += wt * oe["y"][g]
    assert groups >= 2
    for t in range(8):
        assert pr.normwise_err(y[t].cpu().numpy(), y_ref[t]) <= 1e-2
    for part in parts:
        part.destroy()


def test_moe_small():
    cfg = wl.FFNConfig("moe_small", d=2048, N=600, dtype=wl.BF16, prompt_tokens=48, decode_steps=3,
                       ratios=wl.Ratios(0.5, 0.2, 0.3), seed=11)
    run_moe_case(cfg, n_experts=4, steps=3)


@pytest.mark.parametrize("r", [0.2, 0.4])
def test_config4_moe_full_size(r):
    cfg = wl.config4_expert(r)
    run_moe_case(cfg, n_experts=8, steps=4)


@pytest.mark.gpu
@pytest.mark.parametrize("d,dtype", [(2048, wl.BF16), (128, wl.F32)])
def test_all_candidate_scores_equal(d, dtype):
    """x = 0 makes every candidate score 0: nothing separates the candidates, so the top-k is decided by the
    tie-break alone (lowest channel ids, Sec. 3.3 ranking read as a total order) and y is exactly 0.  In the
    streaming kernel this is the case where no candidate is decided by the streamed scores."""
    cfg = wl.FFNConfig("zeros", d=d, N=384, dtype=dtype, prompt_tokens=16, decode_steps=1,
                       ratios=wl.Ratios(0.4, 0.35, 0.25), seed=5)
    w = wl.make_ffn_workload(cfg)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, cfg.ratios.astuple())
    R, C, _ = part.indices()
    x0 = np.zeros_like(w.xs.values[0])
    x = torch.zeros_like(pr.to_dev(w.xs, index=0))
    for k in (1, part.n_cand // 2, part.n_cand - 1):
        mask = torch.full((part.n_cand,), 9, dtype=torch.uint8, device="cuda:0")
        sel = torch.full((k,), -1, dtype=torch.int32, device="cuda:0")
        y = pop.decode_step(part, x, k, mask_out=mask, sel_out=sel)
        torch.cuda.synchronize()
        part.check()
        o = po.decode_step(x0, *Wh, R, C, k)
        assert np.array_equal(o["sel"], C[:k])                       # the oracle's own tie-break, stated
        assert np.array_equal(sel.cpu().numpy(), o["sel"])
        assert np.array_equal(mask.cpu().numpy(), o["mask"])
        assert float(y.float().abs().max()) == 0.0
    part.destroy()


def _stream_case():
    cfg = wl.FFNConfig("modes", d=2048, N=1536, dtype=wl.BF16, prompt_tokens=24, decode_steps=3,
                       ratios=wl.Ratios(0.5, 0.25, 0.25), seed=11)
    w = wl.make_ffn_workload(cfg)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, cfg.ratios.astuple())
    part.streamed_scores()          # raises unless the streaming kernel serves this partition
    return w, Wh, part


def _check_steps(w, Wh, part, steps):
    R, C, _ = part.indices()
    k = part.n_cand // 2
    mask = torch.zeros(part.n_cand, dtype=torch.uint8, device="cuda:0")
    for t in range(steps):
        y = pop.decode_step(part, pr.to_dev(w.xs, index=t), k, mask_out=mask)
        torch.cuda.synchronize()
        part.check()
        o = po.decode_step(w.xs.values[t], *Wh, R, C, k)
        assert np.array_equal(mask.cpu().numpy(), o["mask"])
        assert pr.rel_err(pr.host_values(y), o["y"]) <= pr.TOL[wl.BF16]


@pytest.mark.parametrize("mode", ["pdl", "coop", "plain"])
def test_streaming_kernel_launch_modes(mode, decode_impl):
    """The launch mode is a process-wide setting read at every step: the same partition is stepped in each mode."""
    if decode_impl != "stream":
        pytest.skip("launch modes belong to the streaming kernel")
    w, Wh, part = _stream_case()
    code = {"pdl": pop.POP_LAUNCH_PDL, "coop": pop.POP_LAUNCH_COOPERATIVE, "plain": pop.POP_LAUNCH_PLAIN}[mode]
    old = pop.set_config(launch_mode=code)
    try:
        assert pop.get_config().launch_mode == code
        _check_steps(w, Wh, part, 3)
    finally:
        pop.set_config(launch_mode=old.launch_mode)
    part.destroy()


def test_a_wait_that_runs_out_is_reported_and_the_partition_stays_usable(decode_impl):
    """Failure detection without a fault: with a wait budget of zero every device-side wait that is not satisfied
    within its first polls gives up, the step winds down (all CTAs drain and leave), pop_partition_check reports
    POP_ERR_TIMEOUT, and with the budget restored the next steps on the same partition are correct again."""
    if decode_impl != "stream":
        pytest.skip("the streaming kernel is the one whose CTAs wait on one another")
    w, Wh, part = _stream_case()
    old = pop.set_config(wait_budget_us=0)
    try:
        timed_out = 0
        for t in range(3):
            pop.decode_step(part, pr.to_dev(w.xs, index=t), part.n_cand // 2)
            try:
                part.check()
            except pop.PopError as e:
                assert e.status == pop.POP_ERR_TIMEOUT
                timed_out += 1
    finally:
        pop.set_config(wait_budget_us=old.wait_budget_us)
    assert timed_out > 0, "no wait ran out with a zero budget"
    _check_steps(w, Wh, part, 3)
    part.destroy()


def test_config_rejects_bad_values_and_cache_can_be_released():
    c = pop.get_config()
    for bad in ({"decode_kernel": 7}, {"launch_mode": -1}):
        with pytest.raises(pop.PopError) as e:
            pop.set_config(**bad)
        assert e.value.status == pop.POP_ERR_INVALID_ARG
    assert pop.get_config().launch_mode == c.launch_mode
    pop.release_cached_memory()


@pytest.mark.parametrize("d,N,L,dtype", [(512, 1500, 70, wl.BF16), (2048, 900, 40, wl.BF16), (264, 777, 33, wl.F32)])
def test_prepared_weights_give_the_same_partition(d, N, L, dtype):
    """pop_weights_prepare + pop_prefill_partition_prepared against pop_prefill_partition: same regions and scores, bit
    for bit, for two prompts on one prepared weight set."""
    cfg = wl.FFNConfig("prep", d=d, N=N, dtype=dtype, prompt_tokens=L, decode_steps=1, ratios=wl.Ratios(0.5, 0.2, 0.3), seed=41)
    w = wl.make_ffn_workload(cfg)
    Wg, Wu, Wd = weights_dev(w)
    wts = pop.Weights(Wg, Wu, Wd)
    X = pr.to_dev(w.X)
    for Xi in (X, X[: L // 2].contiguous()):
        a = pop.prefill_partition(Xi, Wg, Wu, Wd, cfg.ratios.astuple())
        b = wts.prefill_partition(Xi, cfg.ratios.astuple())
        for ia, ib in zip(a.indices(), b.indices()):
            assert np.array_equal(ia, ib)
        assert np.array_equal(a.scores(), b.scores()) and np.array_equal(a.score_bounds(), b.score_bounds())
        a.destroy(); b.destroy()
    wts.destroy()


@pytest.mark.parametrize("d,N,L,stride,dtype", [(512, 1500, 70, 3, wl.BF16), (2048, 904, 200, 4, wl.BF16), (264, 777, 33, 2, wl.F32),
                                                  (4096, 11008, 512, 4, wl.BF16), (1024, 1112, 64, 1, wl.BF16), (1024, 1112, 5, 7, wl.BF16)])
def test_partial_probing_scores_every_s_th_token(d, N, L, stride, dtype):
    """pop_prefill_partition_probe (Sec. 3.4 "partial probing prompt activations", read as every s-th prompt token): the
    regions are those the oracle finds on rows 0, s, 2 s, ... of the prompt, the scores agree with it as those of a
    whole prompt do, and the partition is the one pop_prefill_partition_prepared gives for those rows alone, bit for bit."""
    cfg = wl.FFNConfig("probe", d=d, N=N, dtype=dtype, prompt_tokens=L, decode_steps=1, ratios=wl.Ratios(0.5, 0.2, 0.3), seed=d + stride)
    w = wl.make_ffn_workload(cfg)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    wts = pop.Weights(Wg, Wu, Wd)
    X = pr.to_dev(w.X)
    a = wts.prefill_partition_probe(X, cfg.ratios.astuple(), stride)
    ref = po.prefill_partition_probe(w.X.values, *Wh, cfg.ratios.astuple(), stride)
    check_prefill_scores(a, ref, dtype)
    pr.check_regions(a, ref)
    b = wts.prefill_partition(X[::stride].contiguous(), cfg.ratios.astuple())
    for ia, ib in zip(a.indices(), b.indices()):
        assert np.array_equal(ia, ib)
    assert np.array_equal(a.scores(), b.scores()) and np.array_equal(a.score_bounds(), b.score_bounds())
    with pytest.raises(pop.PopError):
        wts.prefill_partition_probe(X, cfg.ratios.astuple(), 0)
    a.destroy(); b.destroy(); wts.destroy()


# ------------------------------------------------------------------ the prompt's own output under the pruned structure
@pytest.mark.parametrize("d,N,L,kfrac", [(512, 1504, 70, 0.5), (2048, 904, 40, 0.25), (320, 648, 200, 1.0), (1024, 1112, 130, 0.0)])
def test_prefill_output_small(d, N, L, kfrac):
    """pop_prefill_partition_with_output against the oracle's prefill_output (Sec. 3.4: Retained + the k best Candidates
    by prefill score), several token and channel tiles with ragged tails; the partition it returns is the usual one."""
    cfg = wl.FFNConfig("pout", d=d, N=N, dtype=wl.BF16, prompt_tokens=L, decode_steps=1, ratios=wl.Ratios(0.5, 0.2, 0.3), seed=d + L)
    run_prefill_output_case(cfg, kfrac)


def run_prefill_output_case(cfg, kfrac):
    w = wl.make_ffn_workload(cfg, 1)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    wts = pop.Weights(Wg, Wu, Wd)
    ref = po.prefill_partition(w.X.values, *Wh, cfg.ratios.astuple())
    k = int(round(kfrac * ref["C"].size))
    part, Y = wts.prefill_partition_with_output(pr.to_dev(w.X), cfg.ratios.astuple(), k)
    torch.cuda.synchronize()
    part.check()
    pr.check_regions(part, ref)
    check_prefill_scores(part, ref, cfg.dtype)
    yref = po.prefill_output(w.X.values, *Wh, ref["R"], ref["C"], ref["scores"], k)
    err = pr.rel_err(pr.host_values(Y), yref)
    assert err <= pr.TOL[wl.BF16], f"prompt output error {err:.3e}"
    part.destroy()
    wts.destroy()
    return err


def test_prefill_output_config2_full_size():
    run_prefill_output_case(wl.config2(0.2), 0.5)


def test_prefill_output_rejects_what_it_does_not_take():
    cfg = wl.FFNConfig("pout32", d=256, N=640, dtype=wl.F32, prompt_tokens=16, decode_steps=1, seed=3)
    w = wl.make_ffn_workload(cfg, 1)
    wts = pop.Weights(*weights_dev(w))
    with pytest.raises(pop.PopError) as e:
        wts.prefill_partition_with_output(pr.to_dev(w.X), cfg.ratios.astuple(), 10)
    assert e.value.status == pop.POP_ERR_UNSUPPORTED
    wts.destroy()
    cfg = wl.FFNConfig("poutk", d=256, N=640, dtype=wl.BF16, prompt_tokens=16, decode_steps=1, seed=3)
    w = wl.make_ffn_workload(cfg, 1)
    wts = pop.Weights(*weights_dev(w))
    with pytest.raises(pop.PopError) as e:
        wts.prefill_partition_with_output(pr.to_dev(w.X), cfg.ratios.astuple(), 10 ** 6)
    assert e.value.status == pop.POP_ERR_INVALID_ARG
    wts.destroy()


# ------------------------------------------------------------------ inputs built to strain the error bounds
@pytest.mark.parametrize("batch", [1, 3])
@pytest.mark.parametrize("kind", ["heavy_tail", "cancellation", "mixed_magnitudes"])
def test_error_bounds_hold_on_adversarial_inputs(kind, batch):
    """Regions and masks are decided on scores that went through the tensor cores in reduced precision, each with a bound
    of its error; exactness rests on those bounds.  Here they meet heavy-tailed activations at decode time, rows whose
    terms cancel from partial sums of several hundred down to order one, and activations that mix 1e-3 with 1e3.
    Prefill scores must lie within a quarter of their bounds and the regions equal the oracle's; at every decode step
    the masks equal the oracle's and, under the streaming kernel, |streamed - exact| stays within a quarter of the
    streamed bound.  The outputs of these constructed cases sum terms of very different magnitude (the cancellation
    case reaches 2.3e-2 on one near-zero output under the 1e-3 floor, 4.5e-3 under 1e-2, 2.7e-3 normwise), so they
    are judged with the 1e-2 floor."""
    w = wl.make_adversarial_case(kind, d=2048, N=768, L=40, steps=4, batch=batch, seed=23)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, w.cfg.ratios.astuple())
    ref = po.prefill_partition(w.X.values, *Wh, w.cfg.ratios.astuple())
    check_prefill_scores(part, ref, wl.BF16)
    pr.check_regions(part, ref)
    R, C, _ = part.indices()
    run_decode_parity(w, part, R, C, 4, part.n_cand // 2, Wh, floor=1e-2)
    part.destroy()


# ------------------------------------------------------------------ wide candidate regions (partition fraction 0.2 and more)
@pytest.mark.parametrize("B", [1, 4])
def test_many_candidates_on_the_streaming_kernel(B, decode_impl):
    """More than 1536 and up to 3072 candidates: still the streaming kernel (its selection warp holds 96 keys per lane)."""
    cfg = wl.FFNConfig("wideC", d=2048, N=4000, dtype=wl.BF16, prompt_tokens=24, decode_steps=3, batch=B,
                       ratios=wl.Ratios(0.25, 0.65, 0.10), seed=77)
    assert po.region_sizes(cfg.N, cfg.ratios.astuple())[1] == 2600
    run_case(cfg)


def test_config2_gamma02_full_size(decode_impl):
    """Sec. 5 "Partition Fraction": gamma = 0.2 at Llama-2-7B shapes is 2201 candidates."""
    cfg = wl.scaled(wl.config2(0.2), ratios=wl.ratios_for(0.2, 0.2), name="cfg2_llama7b_r20_gamma20")
    assert po.region_sizes(cfg.N, cfg.ratios.astuple())[:2] == (7707, 2201)
    w = wl.make_ffn_workload(cfg, 4)
    Wh = weights_host(w)
    Wg, Wu, Wd = weights_dev(w)
    part = pop.prefill_partition(pr.to_dev(w.X), Wg, Wu, Wd, cfg.ratios.astuple())
    if decode_impl == "stream":
        part.streamed_scores()          # raises unless the streaming kernel serves this partition
    ref = po.prefill_partition(w.X.values, *Wh, cfg.ratios.astuple())
    pr.check_regions(part, ref)
    R, C, _ = part.indices()
    run_decode_parity(w, part, R, C, 4, part.n_cand // 2, Wh)
    part.destroy()
