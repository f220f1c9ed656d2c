"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and its host-only logic agrees with the oracle.  No GPU compute is called here."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as ge
from oracle import pop_oracle as po
from paper_2602_06822_b200 import pop

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ge.build()
    return pop.lib()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "pop.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(pop_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert "pop_prefill_partition" in names and "pop_decode_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in pop.h but not exported"
        assert n in pop.SIGNATURES, f"{n} has no binding"
    assert sorted(pop.SIGNATURES) == names


def test_version_and_status_strings(lib):
    assert "sm_100a" in pop.version()
    assert pop.status_string(0) == "POP_OK"
    assert pop.status_string(pop.POP_ERR_TIMEOUT) == "POP_ERR_TIMEOUT"
    assert pop.status_string(-99) == "POP_ERR_UNKNOWN"


@pytest.mark.parametrize("N,ratios", [
    (1376, (0.30, 0.40, 0.30)), (11008, (0.75, 0.10, 0.15)), (11008, (0.55, 0.10, 0.35)),
    (14336, (0.75, 0.10, 0.15)), (13824, (0.55, 0.10, 0.35)), (6, (1 / 3, 1 / 3, 1 / 3)),
    (97, (0.5, 0.25, 0.25)), (7, (0.0, 1.0, 0.0)), (5, (1.0, 0.0, 0.0)), (10, (0.2, 0.2, 0.2)),
])
def test_region_sizes_agree_with_oracle(lib, N, ratios):
    n_ret, n_cand, n_pruned, k = pop.region_sizes(N, ratios)
    assert (n_ret, n_cand, n_pruned) == po.region_sizes(N, ratios)
    assert k == po.default_k(n_cand)


def test_region_sizes_rejects_bad_input(lib):
    for N, r in ((0, (0.5, 0.2, 0.3)), (10, (0.5, 0.5, 0.5)), (10, (-0.1, 0.5, 0.5)), (10, (0.1, 0.6, 0.6))):
        with pytest.raises(pop.PopError) as e:
            pop.region_sizes(N, r)
        assert e.value.status == pop.POP_ERR_INVALID_ARG


def test_null_arguments_are_rejected_without_touching_the_device(lib):
    out = C.c_void_p()
    r = pop.Ratios(0.5, 0.2, 0.3)
    assert lib.pop_prefill_partition(None, 4, 8, None, None, None, 16, 0, r, None, C.byref(out)) == pop.POP_ERR_INVALID_ARG
    assert lib.pop_prefill_partition(None, 4, 8, None, None, None, 16, 0, r, None, None) == pop.POP_ERR_INVALID_ARG
    assert lib.pop_decode_step(None, None, 1, 0, None, None, None, None) == pop.POP_ERR_INVALID_ARG
    assert lib.pop_partition_sizes(None, None, None, None) == pop.POP_ERR_INVALID_ARG
    assert lib.pop_partition_destroy(None) == pop.POP_ERR_INVALID_ARG
    assert lib.pop_partition_check(None) == pop.POP_ERR_INVALID_ARG
    assert lib.pop_partition_from_indices(None, None, None, 16, 8, 0, None, 0, None, 0, None, C.byref(out)) == pop.POP_ERR_INVALID_ARG


def test_binding_refuses_to_run_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(RuntimeError):
        pop._torch()
