"""Host-side checks that need no GPU: the library loads, exports what the header declares,
and rejects bad arguments before touching CUDA."""
import ctypes as C

import pytest

from paper_2601_16986_b200 import build as lib_build
from paper_2601_16986_b200 import declared_symbols, load_library
from paper_2601_16986_b200.binding import _Cfg


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return load_library()


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"crystalkv_create", "crystalkv_prefill", "crystalkv_decode_step", "crystalkv_rebudget",
            "crystalkv_get_retained"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def good():
    return _Cfg(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=1, dtype=1, budget_per_head=64,
                min_budget=0, max_budget=0, max_answer_tokens=0, max_context=256, top_p=0.9, lam=0.6,
                sm_scale=0.0, mode=0, device=0)


@pytest.mark.parametrize("field,value", [("head_dim", 64), ("dtype", 7), ("n_layers", 0), ("n_q_heads", 7),
                                         ("n_q_heads", 32), ("mode", 3), ("max_context", 1),
                                         ("budget_per_head", 0), ("max_budget", 8), ("min_budget", 65),
                                         ("top_p", 1.5), ("lam", 1.2), ("device", -1), ("batch", 0)])
def test_create_rejects_bad_config_before_cuda(lib, field, value):
    c = good()
    setattr(c, field, value)
    h = C.c_void_p()
    assert lib.crystalkv_create(C.byref(c), C.byref(h)) == -1
    assert not h.value
    assert len(lib.crystalkv_last_error(None)) > 0


def test_null_arguments(lib):
    h = C.c_void_p()
    assert lib.crystalkv_create(None, C.byref(h)) == -1
    assert lib.crystalkv_create(C.byref(good()), None) == -1
    assert lib.crystalkv_destroy(None) == 0
    assert lib.crystalkv_set_stage(None, 0) == -1
    assert lib.crystalkv_rebudget(None, None) == -1
    assert lib.crystalkv_decode_step(None, 0, None, None, None, None, None) == -1
    assert lib.crystalkv_time(None, 0) == -1
    for code in (0, -1, -2, -3, -4, -5):
        assert lib.crystalkv_strerror(code)


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    from paper_2601_16986_b200 import Config, CrystalKV, CrystalKVError
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(CrystalKVError):
        CrystalKV(Config(n_layers=1, n_q_heads=2, n_kv_heads=1, batch=1, budget_per_head=8, max_context=32))


def _place_runs_one_by_one(whole, runs):
    """Best fit, longest first, one run at a time: the placement the planner performs."""
    free = []            # free warps of every open CTA
    for s in range(7, 0, -1):
        for _ in range(runs[s]):
            fits = [c for c in free if c >= s]
            if fits:
                c = min(fits)
                free.remove(c)
            else:
                c = 8
            if c - s:
                free.append(c - s)
            if c == 8:
                whole += 1   # a CTA was opened
    return whole


def test_the_planners_count_equals_placing_the_runs_one_by_one(lib):
    """The launch planner counts the CTAs a placement needs by moving whole classes of CTAs at
    once; the placement itself goes run by run.  The two must agree for every mix of run lengths,
    or a plan could be chosen that then does not fit the grid."""
    import numpy as np
    rng = np.random.default_rng(7)
    cases = [[0] * 8, [0, 1, 0, 0, 0, 0, 0, 0], [0, 0, 0, 0, 0, 0, 0, 5], [0, 9, 0, 0, 0, 0, 0, 3],
             [0, 0, 4, 0, 0, 0, 2, 0], [0, 3, 3, 3, 3, 3, 3, 3]]
    for _ in range(400):
        top = int(rng.integers(1, 40))
        cases.append([0] + [int(x) for x in rng.integers(0, top, size=7)])
    for runs in cases:
        arr = (C.c_int32 * 8)(*runs)
        for whole in (0, 3):
            got = lib.crystalkv_debug_ctas_needed(whole, arr)
            assert got == _place_runs_one_by_one(whole, runs), (whole, runs, got)
    assert lib.crystalkv_debug_ctas_needed(0, None) == -1
    bad = (C.c_int32 * 8)(0, -1, 0, 0, 0, 0, 0, 0)
    assert lib.crystalkv_debug_ctas_needed(0, bad) == -1
    assert lib.crystalkv_debug_ctas_needed(-1, (C.c_int32 * 8)()) == -1
