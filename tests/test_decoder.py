"""The Llama-2-7B-shaped decoder with POP on every FFN (dense attention unchanged): layer-local parity.

A random-init bf16 network amplifies rounding from layer to layer, so an end-to-end index comparison would say
nothing.  Instead every checked layer-step hands the oracle exactly what the library saw: the layer's actual bf16
FFN input and its partition.  Masks must be equal (near-tie swaps as in tests/parity.py), outputs within 2e-2.
The prompt side is checked the same way per layer: regions and the prompt's own output from the layer's actual
normalised input.  An end-to-end cosine against an fp64 run of the same model is reported for a short run, not gated.
"""
import numpy as np
import pytest
import torch

import __graft_entry__ as ge
from oracle import pop_oracle as po
from paper_2602_06822_b200 import decoder as dec, pop, workloads as wl
from tests import parity as pr

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    ge.build()
    pop.lib()


def host64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def layer_weights64(m, li):
    L = m.layers[li]
    return host64(L["Wg"]), host64(L["Wu"]), host64(L["Wd"])


def check_layer_prefill(m, li, ratios, k):
    f, y = m.trace[("prefill", li)]
    Wh = layer_weights64(m, li)
    ref = po.prefill_partition(host64(f), *Wh, ratios)
    pr.check_regions(m.parts[li], ref)
    yref = po.prefill_output(host64(f), *Wh, ref["R"], ref["C"], ref["scores"], k)
    err = pr.rel_err(host64(y), yref)
    assert err <= pr.TOL[wl.BF16], f"layer {li}: prompt output error {err:.3e}"
    return Wh


def check_layer_step(m, li, step, Wh, k):
    f, y, mask, sel = m.trace[(li, step)]
    R, C, _ = m.parts[li].indices()
    o = po.decode_step(host64(f), *Wh, R, C, k)
    s = sel.cpu().numpy()
    sw = pr.check_selection(s, mask.cpu().numpy(), C, o, k)
    yref = o["y"] if not sw else po.masked_ffn(host64(f), *Wh, np.sort(np.concatenate([R, s])))
    err = pr.rel_err(host64(y), yref)
    assert err <= pr.TOL[wl.BF16], f"layer {li} step {step}: output error {err:.3e}"
    return err


def reference_run_fp64(m, ids, n_in, n_out, ratios, k):
    """The same model in fp64 on the CPU with the oracle's FFN (regions from the fp64 activations): final hidden states."""
    cfg = m.cfg
    hd = cfg.d // cfg.n_heads
    inv = 1.0 / (cfg.rope_base ** (torch.arange(0, hd, 2, dtype=torch.float64) / hd))

    def rms(h):
        return h * torch.rsqrt(h.pow(2).mean(-1, keepdim=True) + cfg.rms_eps)

    def rope(x, pos0):
        T = x.shape[0]
        ang = torch.arange(pos0, pos0 + T, dtype=torch.float64)[:, None] * inv[None, :]
        c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
        x1, x2 = x[..., : hd // 2], x[..., hd // 2:]
        return torch.cat([x1 * c - x2 * s, x2 * c + x1 * s], dim=-1)

    Wl = [{n: t.detach().double().cpu() for n, t in L.items()} for L in m.layers]
    emb = m.embed.detach().double().cpu()
    kv = [None] * cfg.n_layers
    parts = [None] * cfg.n_layers
    outs = []
    pos = 0
    for chunk in [ids[:n_in].cpu()] + [ids[n_in + s: n_in + s + 1].cpu() for s in range(n_out)]:
        h = emb[chunk]
        T = h.shape[0]
        for li, L in enumerate(Wl):
            a = rms(h)
            q = rope((a @ L["Wq"].T).view(T, cfg.n_heads, hd), pos)
            kx = rope((a @ L["Wk"].T).view(T, cfg.n_heads, hd), pos)
            vx = (a @ L["Wv"].T).view(T, cfg.n_heads, hd)
            K, V = (kx, vx) if kv[li] is None else (torch.cat([kv[li][0], kx]), torch.cat([kv[li][1], vx]))
            kv[li] = (K, V)
            att = torch.einsum("thd,shd->hts", q, K) / np.sqrt(hd)
            if T > 1:
                att = att + torch.triu(torch.full((T, K.shape[0]), float("-inf"), dtype=torch.float64), diagonal=1 + K.shape[0] - T)
            o = torch.einsum("hts,shd->thd", torch.softmax(att, dim=-1), V).reshape(T, cfg.d)
            h = h + o @ L["Wo"].T
            f = rms(h).numpy()
            W3 = (L["Wg"].numpy(), L["Wu"].numpy(), L["Wd"].numpy())
            if T > 1:
                parts[li] = po.prefill_partition(f, *W3, ratios)
                y = po.prefill_output(f, *W3, parts[li]["R"], parts[li]["C"], parts[li]["scores"], k)
            else:
                y = po.decode_step(f, *W3, parts[li]["R"], parts[li]["C"], k)["y"]
            h = h + torch.from_numpy(np.asarray(y, dtype=np.float64)).view(T, cfg.d)
        pos += T
        outs.append(h[-1])
    return torch.stack(outs)


def test_reduced_decoder_every_layer_step():
    cfg = dec.DecoderConfig(n_layers=3, d=2048, n_heads=16, N=2816, vocab=512, seed=5)
    ratios = dec.ratios_for(0.2)
    n_in, n_out = 48, 4
    m = dec.Decoder(cfg, ffn="pop", ratios=ratios)
    k = pop.region_sizes(cfg.N, ratios)[3]
    ids = dec.seeded_ids(cfg, n_in + n_out, 9, m.dev)
    m.trace = {}
    hs = [m.prefill(ids[:n_in])[-1]]
    for s in range(n_out):
        hs.append(m.decode(ids[n_in + s: n_in + s + 1], s)[0])
    torch.cuda.synchronize()
    for p in m.parts:
        p.check()
    worst = 0.0
    for li in range(cfg.n_layers):
        Wh = check_layer_prefill(m, li, ratios, k)
        for s in range(n_out):
            worst = max(worst, check_layer_step(m, li, s, Wh, k))
    # reported, not gated: the whole model against an fp64 run of it
    ref = reference_run_fp64(m, ids, n_in, n_out, ratios, k)
    got = torch.stack(hs).double().cpu()
    cos = torch.nn.functional.cosine_similarity(got, ref, dim=-1)
    print(f"reduced decoder: worst layer-step output error {worst:.2e}; end-to-end cosine of the final hidden state vs fp64: "
          f"min {float(cos.min()):.6f} mean {float(cos.mean()):.6f}")
    m.close()


def test_config3_full_decoder_sampled_layer_steps():
    """32 layers, hidden 4096, 32 heads, FFN 11008, prompt 1024, 256 teacher-forced steps, r = 0.2; the oracle checks
    the prompt side of two layers and a sample of decode layer-steps (each costs it a few hundred milliseconds)."""
    cfg = dec.DecoderConfig()
    ratios = dec.ratios_for(0.2)
    n_in, n_out = 1024, 256
    layers_checked, steps_checked = (0, 13, 31), (0, 1, 100, 255)
    m = dec.Decoder(cfg, ffn="pop", ratios=ratios)
    k = pop.region_sizes(cfg.N, ratios)[3]
    assert (m.weights[0] is not None) and k == 550
    ids = dec.seeded_ids(cfg, n_in + n_out, 21, m.dev)
    m.trace = {"want": lambda li, s: li in layers_checked and s in steps_checked}
    keep_prefill = {}
    h = m.prefill(ids[:n_in])
    for li in list(range(cfg.n_layers)):
        if li in (0, 31):
            keep_prefill[li] = m.trace[("prefill", li)]
        del m.trace[("prefill", li)]
    for s in range(n_out):
        h = m.decode(ids[n_in + s: n_in + s + 1], s)
    torch.cuda.synchronize()
    assert torch.isfinite(h.float()).all()
    for p in m.parts:
        p.check()
        assert (p.n_ret, p.n_cand) == (8257, 1100)
    worst = 0.0
    for li in layers_checked:
        if li in keep_prefill:
            m.trace[("prefill", li)] = keep_prefill[li]
            Wh = check_layer_prefill(m, li, ratios, k)
        else:
            Wh = layer_weights64(m, li)
        for s in steps_checked:
            worst = max(worst, check_layer_step(m, li, s, Wh, k))
    print(f"config 3: worst sampled layer-step output error {worst:.2e}")
    m.close()


def test_static_decode_step_matches_the_eager_one_and_replays_as_a_graph():
    """The graph-capturable decode step (preallocated KV cache, device-side position) against the eager one on the same
    model and tokens, first launched eagerly, then captured once and replayed."""
    cfg = dec.DecoderConfig(n_layers=2, d=2048, n_heads=16, N=2816, vocab=256, seed=7)
    ratios = dec.ratios_for(0.2)
    n_in, n_out = 24, 6
    ids = dec.seeded_ids(cfg, n_in + n_out + 1, 4, "cuda:0")
    m = dec.Decoder(cfg, ffn="pop", ratios=ratios)
    m.prefill(ids[:n_in])
    want = [m.decode(ids[n_in + s: n_in + s + 1], s)[0].float().clone() for s in range(n_out)]
    m.reset()
    m.prefill(ids[:n_in])
    m.begin_static(ids, n_in + n_out + 4)
    got = [m.step_static()[0].float().clone() for _ in range(2)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        out = m.step_static()
    for s in range(2, n_out):
        graph.replay()
        torch.cuda.synchronize()
        got.append(out[0].float().clone())
    for p in m.parts:
        p.check()
    for s in range(n_out):
        cos = float(torch.nn.functional.cosine_similarity(got[s], want[s], dim=0))
        assert cos > 0.9999, f"step {s}: cosine {cos}"
    m.close()
