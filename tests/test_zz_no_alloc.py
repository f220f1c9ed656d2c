"""pop_prefill_scores_noalloc against pop_prefill_partition's scores and against the oracle's.

The entry point serves callers that may not allocate device memory when they need the prefill
scores (a fixed memory pool, a hot loop that bans allocator calls); its temporaries sit in a fixed
array inside the library that every call on the device shares and that keeps the last call's
contents.  So it is called here twice in a row, on two different layers (the second smaller, so
that stale entries of the first call lie behind it), and each result is compared with the scores
the allocating entry point gives for the same inputs, within the tolerance the other score tests use:
fp64 rounding where that entry point scored in fp64 (error bound 0), its own stated bound where it
streamed the score through the tensor cores.  The no-allocation call always scores in fp64, so it is
also held to the oracle's Eq. 3 scores at fp64 rounding.

This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
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


def _layer(d, N, L, dtype, seed):
    cfg = wl.FFNConfig("noalloc", d=d, N=N, dtype=dtype, prompt_tokens=L, decode_steps=1,
                       ratios=wl.Ratios(0.5, 0.2, 0.3), seed=seed)
    w = wl.make_ffn_workload(cfg)
    exact = po.prefill_scores(w.X.values, w.weights.Wg.values, w.weights.Wu.values, w.weights.Wd.values)
    return (cfg, pr.to_dev(w.X), pr.to_dev(w.weights.Wg), pr.to_dev(w.weights.Wu), pr.to_dev(w.weights.Wd)), exact


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    made = [_layer(512, 1500, 70, wl.BF16, 31), _layer(264, 777, 33, wl.F32, 32)]
    layers, exact = [m[0] for m in made], [m[1] for m in made]
    outs = [torch.full((cfg.N,), -1.0, dtype=torch.float64, device="cuda:0") for cfg, *_ in layers]
    # both calls back to back on one stream, nothing in between
    for (cfg, X, Wg, Wu, Wd), out in zip(layers, outs):
        pop.prefill_scores_noalloc(X, Wg, Wu, Wd, out)
    torch.cuda.synchronize()
    for (cfg, X, Wg, Wu, Wd), out, ex in zip(layers, outs, exact):
        part = pop.prefill_partition(X, Wg, Wu, Wd, cfg.ratios.astuple())
        want, bound = part.scores(), part.score_bounds()
        part.destroy()
        got = out.cpu().numpy()
        assert np.all(got >= 0.0) and np.all(np.isfinite(got))
        assert np.all(np.abs(got - want) <= bound + 1e-9 * np.abs(want)), "differs from the allocating entry point"
        np.testing.assert_allclose(got, ex, rtol=1e-9, atol=1e-300)


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    (cfg, X, Wg, Wu, Wd), _ = _layer(128, 64, 8, wl.BF16, 33)
    out = torch.zeros(64, dtype=torch.float64, device="cuda:0")
    too_big = pop.POP_NOALLOC_MAX_N + 1
    # rejected on the host before anything is launched, so the short arrays are never read
    rc = pop.lib().pop_prefill_scores_noalloc(X.data_ptr(), 8, 128, Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(),
                                              too_big, pop.POP_BF16, out.data_ptr(), None)
    assert rc == pop.POP_ERR_UNSUPPORTED
    assert "POP_NOALLOC_MAX_N" in pop.lib().pop_last_cuda_error().decode()
    torch.cuda.synchronize()
    assert float(out.abs().sum()) == 0.0
