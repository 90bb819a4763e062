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
