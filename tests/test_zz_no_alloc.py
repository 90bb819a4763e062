"""crystalkv_validate_static: the slot-ownership check for callers that cannot allocate.

Some users of this library run where a cudaMalloc is not an option: an inference server
whose memory pool has already claimed the whole GPU, or a loop that cannot afford the
device-wide stall of an allocation.
For them the library offers crystalkv_validate_static, which keeps its per-slot counters in
an array built into the library instead of a temporary.  These tests call it through the C
ABI and hold it against crystalkv_validate, the allocating entry point: same verdict on the
same handle, on two calls in a row (the array is shared and keeps the last call's contents,
so a second call only passes if the first one's leftovers are cleared), on a handle of a
different size afterwards, and a clear refusal for a handle too large for the array.

The file name sorts last on purpose: a run that stops at the first failure has then already
gone through every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2601_16986_b200 import Config, CrystalKV, CrystalKVError
from synth import Workload

pytestmark = pytest.mark.gpu


def _run(wl, n_steps, rebudget_at=()):
    """A handle that went through a prefill and `n_steps` decode steps of every layer."""
    ctx = wl.prompt + n_steps + 16
    kv = CrystalKV(Config(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                          batch=wl.batch, budget_per_head=wl.budget_per_head, max_context=ctx,
                          top_p=wl.top_p, lam=wl.lam))
    for l in range(wl.n_layers):
        k, v = wl.prompt_kv(l, device="cuda")
        kv.prefill(l, k, v, wl.queries(l, [wl.prompt - 1], device="cuda")[:, 0].contiguous())
    for s in range(n_steps):
        for l in range(wl.n_layers):
            kv.decode_step(l, *wl.step_inputs(l, wl.prompt + s, device="cuda"))
        if s + 1 in rebudget_at:
            kv.rebudget()
    return kv


def _verdict(call):
    """(status code, counts) of one of the two entry points; 0 = sound."""
    try:
        out = call()
        return 0, (None if out is None else tuple(int(x) for x in out))
    except CrystalKVError as e:
        return e.code, None


def test_static_check_agrees_with_the_allocating_one_twice_in_a_row():
    wl = Workload(name="na", seed=41, n_layers=3, n_q_heads=8, n_kv_heads=2, batch=3, prompt=40,
                  think_steps=60, budget_per_head=48, outlier="perhead", outlier_lo=0.01, outlier_hi=0.2)
    kv = _run(wl, 60, rebudget_at=(24, 48))      # evictions, slot reuse and two reallocations happened
    ref_code, _ = _verdict(kv.validate)          # the existing entry point (allocates a temporary)
    assert ref_code == 0
    for _ in range(2):                           # two calls in a row share the built-in array
        code, counts = _verdict(kv.validate_static)
        assert code == ref_code
        assert counts == (0, 0)
    # more steps, then both again: the verdicts still agree
    for s in range(60, 70):
        for l in range(wl.n_layers):
            kv.decode_step(l, *wl.step_inputs(l, wl.prompt + s, device="cuda"))
    assert _verdict(kv.validate)[0] == 0
    assert _verdict(kv.validate_static) == (0, (0, 0))
    kv.check()
    kv.close()


def test_static_check_after_a_larger_handle_used_the_array():
    """A small handle checked right after a larger one: slots the larger one marked must not
    leak into the smaller one's verdict."""
    big = Workload(name="na_big", seed=42, n_layers=2, n_q_heads=4, n_kv_heads=4, batch=4, prompt=100,
                   think_steps=8, budget_per_head=128)
    small = Workload(name="na_small", seed=43, n_layers=1, n_q_heads=2, n_kv_heads=1, batch=1, prompt=10,
                     think_steps=8, budget_per_head=16)
    kb, ks = _run(big, 8), _run(small, 8)
    assert _verdict(kb.validate_static) == (0, (0, 0))
    assert _verdict(ks.validate_static) == (0, (0, 0))
    assert _verdict(ks.validate)[0] == 0 and _verdict(kb.validate)[0] == 0
    kb.close()
    ks.close()


def test_both_checks_report_a_page_owned_twice():
    """A page table edited from the host so that one head names a page of another: one page is
    then owned twice and one not at all, and both entry points must say so (and agree).  The
    handle is only validated and destroyed afterwards."""
    wl = Workload(name="na_bad", seed=44, n_layers=2, n_q_heads=4, n_kv_heads=2, batch=2, prompt=40,
                  think_steps=8, budget_per_head=64)
    kv = _run(wl, 8)
    assert _verdict(kv.validate)[0] == 0 and _verdict(kv.validate_static) == (0, (0, 0))
    # head (layer 1, seq 1, head 0) owns pages 0..2 of its list (48 entries + the next arrival): its second
    # page is replaced by the id the first head of the sequence holds first
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    victim = 0      # page ids are handed out in ascending order from 0 within a sequence
    assert kv.lib.crystalkv_debug_set_page(kv._h, 1, 1, 0, 1, victim, stream) == 0
    assert kv.lib.crystalkv_debug_set_page(kv._h, 1, 1, 0, 10 ** 6, 0, stream) == -1      # index out of range
    assert kv.lib.crystalkv_debug_set_page(kv._h, 1, 1, 0, 0, 10 ** 9, stream) == -1      # page out of range
    code, _ = _verdict(kv.validate)
    assert code == -5
    assert b"2 pages not owned exactly once" in kv.lib.crystalkv_last_error(kv._h)
    counts = np.full(2, -1, dtype=np.int32)
    rc = kv.lib.crystalkv_validate_static(kv._h, counts.ctypes.data_as(C.c_void_p), stream)
    assert rc == -5 and tuple(counts) == (0, 2)
    kv.close()


def test_static_check_refuses_a_handle_beyond_its_array():
    """2**17 pool pages (16 entries each) is the limit; a handle with more is refused with EINVAL
    and a message that names the limit, and nothing is launched."""
    kv = CrystalKV(Config(n_layers=8, n_q_heads=8, n_kv_heads=8, batch=17, budget_per_head=2047,
                          max_context=64))       # 17 * (8 * 8 * 2049 / 16 + 64) pages > 2**17
    pk = torch.zeros(17, 4, 8, 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(17, 8, 128, dtype=torch.bfloat16, device="cuda")
    for l in range(8):
        kv.prefill(l, pk, pk, q)
    counts = np.full(2, -1, dtype=np.int32)
    rc = kv.lib.crystalkv_validate_static(kv._h, counts.ctypes.data_as(C.c_void_p), None)
    assert rc == -1
    assert b"131072" in kv.lib.crystalkv_last_error(kv._h)
    assert tuple(counts) == (-1, -1)
    assert _verdict(kv.validate)[0] == 0         # the allocating entry point still serves it
    kv.close()


def test_static_check_rejects_bad_arguments_without_a_launch():
    from paper_2601_16986_b200 import load_library
    lib = load_library()
    assert lib.crystalkv_validate_static(None, None, None) == -1
    kv = CrystalKV(Config(n_layers=2, n_q_heads=2, n_kv_heads=1, batch=1, budget_per_head=8, max_context=32))
    with pytest.raises(CrystalKVError) as e:     # before every layer is prefilled
        kv.validate_static()
    assert e.value.code == -2
    kv.close()
