"""GPU <-> oracle parity through the C ABI (needs a B200; run with -m gpu).

Retained sets / CRF bits / tau must be bit-exact except where the oracle logged a tie
(decision within 1e-6 relative of flipping); attention outputs within max-abs 2e-2 of the
fp32 oracle output.  Full-size shapes are run with the whole batch on the GPU and whole
sampled sequences on the oracle.
"""
import os

import numpy as np
import pytest
import torch

from synth import WORKLOADS, Workload
from tests.harness import LockStep

pytestmark = pytest.mark.gpu
SCALE = float(os.environ.get("CRYSTALKV_TEST_SCALE", "1.0"))   # lengthen or shorten the sampled runs


def steps(n):
    return max(8, int(n * SCALE))


def report(name, ls, note=""):
    """One line per run: what was covered.  Printed, and appended to the file named by
    CRYSTALKV_PARITY_REPORT when that is set."""
    r = ls.rep
    line = (f"{name}: sampled seqs {ls.seqs}, steps={r.steps} heads_compared={r.heads_compared} "
            f"ties_logged={r.ties_logged} tie_explained={r.tie_explained} (each verified by a flipped replay; "
            f"{r.replays} replays) unexplained={len(r.unexplained)} budgets_compared={r.budgets_compared} "
            f"max_out_err={r.max_out_err:.3e}{note}")
    print(line)
    path = os.environ.get("CRYSTALKV_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")


def test_cfg1_every_step_of_the_full_run():
    """Config 1 exactly: 256-token prompt, 2048 think steps, budget 512, state compared every step."""
    wl = WORKLOADS["cfg1_gqa4_b512"]
    ls = LockStep(wl, [0])
    ls.prefill()
    ls.compare()
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    report("cfg1_gqa4_b512", ls, " (state compared after every step)")
    ls.assert_clean()
    for h in range(2):
        assert len(ls.gpu.get_retained(0, 0, h)) == 512
    c = ls.gpu.get_counters()
    assert c["evictions"] == 2 * (256 + 2048 - 512)
    ls.close()


@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
def test_every_group_size_with_ragged_tails(G):
    """Budgets and prompts that are not multiples of the 16-key group; prompt above the
    budget (prefill evicts many at once); several tiles per head."""
    wl = Workload(name=f"g{G}", seed=100 + G, n_layers=2, n_q_heads=2 * G, n_kv_heads=2, batch=3,
                  prompt=83, think_steps=70, budget_per_head=53, outlier="flat", outlier_frac=0.05)
    ls = LockStep(wl, [0, 2], max_answer_tokens=40)
    ls.prefill()
    ls.compare()
    for s in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    assert ls.rep.heads_compared > 0 and len(ls.gpu.get_retained(1, 2, 1)) == 53
    ls.close()


class _PairedKeys(Workload):
    """Keys of positions 2i and 2i+1 are identical: exact ties in the group-mean probability."""

    def keys(self, layer, positions, seqs=None, device="cpu"):
        pos = (torch.as_tensor(positions, dtype=torch.int64) // 2) * 2
        return super().keys(layer, pos, seqs, device)


def test_equal_scores_take_the_earlier_position():
    wl = _PairedKeys(name="pairs", seed=5, n_layers=1, n_q_heads=4, n_kv_heads=2, batch=2, prompt=40,
                     think_steps=120, budget_per_head=48, top_p=0.6)
    ls = LockStep(wl, [0, 1])
    ls.prefill()
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


@pytest.mark.parametrize("lam,top_p", [(0.0, 0.9), (1.0, 0.9), (0.6, 1.0), (0.6, 0.5), (0.3, 0.05)])
def test_limits_of_lambda_and_p(lam, top_p):
    """lambda = 0 (LRU), lambda = 1 (LFU), p = 1 (every entry is a hit) and small p."""
    wl = Workload(name="lim", seed=31, n_layers=1, n_q_heads=4, n_kv_heads=1, batch=2, prompt=30,
                  think_steps=150, budget_per_head=64, lam=lam, top_p=top_p)
    ls = LockStep(wl, [0, 1])
    ls.prefill()
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


def test_rebudget_small_with_answer_stage():
    """Adaptive reallocation every 16 steps on a small model, then an answer stage."""
    wl = Workload(name="rb", seed=77, n_layers=3, n_q_heads=8, n_kv_heads=4, batch=3, prompt=64,
                  think_steps=160, answer_steps=12, budget_per_head=64, rebudget_every=16,
                  outlier="perhead", outlier_lo=0.01, outlier_hi=0.3)
    ls = LockStep(wl, [0, 1, 2], max_answer_tokens=16)
    ls.prefill()
    for s in range(wl.think_steps):
        ls.step()
        if (s + 1) % wl.rebudget_every == 0:
            ls.rebudget()
    b = ls.gpu.get_budgets()
    assert (b.reshape(3, -1).sum(axis=1) == 64 * 12).all() and b.min() >= 16 and b.max() <= 256
    assert (b != 64).any()
    ls.set_stage_answer()
    for s in range(wl.answer_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    assert ls.rep.budgets_compared == 30
    ls.close()


@pytest.mark.parametrize("prompt,budget", [(256, 64), (1000, 250), (83, 53)])
def test_prompt_far_longer_than_the_budget_needs_no_reserve(prompt, budget):
    """A prompt of four times the budget with no answer reserve: the prompt is scored from the caller's
    tensors and only the survivors of the one Algorithm 1 pass are stored, so the pool (sized for the
    budget) is never exceeded; state and ownership against the oracle, then decode steps."""
    wl = Workload(name=f"long{prompt}", seed=700 + prompt, n_layers=2, n_q_heads=10, n_kv_heads=2, batch=3,
                  prompt=prompt, think_steps=30, budget_per_head=budget, outlier="flat", outlier_frac=0.05)
    ls = LockStep(wl, [0, 2], max_budget=max(4 * budget, prompt))
    ls.prefill()
    ls.gpu.validate()
    for h in range(2):
        assert len(ls.gpu.get_retained(1, 2, h)) == budget
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


def test_ratio_budgets_follow_the_context():
    """Ratio budgets: the prompt's share at prefill (heads evict down to it), then Algorithm 2 over a
    total that grows with the context at every reallocation; budgets, retained sets and CRF state
    against the oracle."""
    wl = Workload(name="ratio", seed=88, n_layers=3, n_q_heads=8, n_kv_heads=4, batch=3, prompt=96,
                  think_steps=160, budget_per_head=96, rebudget_every=16, outlier="perhead", outlier_lo=0.01, outlier_hi=0.3)
    ls = LockStep(wl, [0, 2], min_budget=4, max_budget=200, max_answer_tokens=80, budget_ratio=0.25)
    ls.prefill()
    assert (ls.gpu.get_budgets() == 24).all() and len(ls.gpu.get_retained(2, 2, 3)) == 24
    totals = []
    for s in range(wl.think_steps):
        ls.step()
        if (s + 1) % wl.rebudget_every == 0:
            ls.rebudget()
            totals.append(int(ls.gpu.get_budgets()[0].sum()))
    assert totals == [min(96, (96 + 16 * (i + 1)) // 4) * 12 for i in range(10)]
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


def test_fullkv_mode_is_plain_decode_attention():
    wl = Workload(name="full", seed=9, n_layers=2, n_q_heads=10, n_kv_heads=2, batch=2, prompt=100,
                  think_steps=60, budget_per_head=16)
    ls = LockStep(wl, [0, 1], mode=1)
    ls.prefill()
    for _ in range(wl.think_steps):
        ls.step(compare_state=False)
    ls.compare()
    ls.gpu.check()
    ls.assert_clean()
    assert len(ls.gpu.get_retained(1, 1, 1)) == 160
    ls.close()


def test_shrinking_one_budget_by_hand():
    """set_budget below the current length evicts many at once and frees their slots."""
    wl = Workload(name="sb", seed=12, n_layers=1, n_q_heads=2, n_kv_heads=2, batch=1, prompt=50,
                  think_steps=30, budget_per_head=60)
    ls = LockStep(wl, [0])
    ls.prefill()
    for _ in range(20):
        ls.step()
    ls.gpu.set_budget(0, 0, 1, 17)
    ls.ora.set_budget(0, 0, 1, 17)
    ls.compare()                   # both sides evict down at once
    assert len(ls.gpu.get_retained(0, 0, 1)) == 17
    ls.step()
    for _ in range(9):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


def _check_plan(kv, layer, lengths, n_kv_heads):
    """Structure of a launch plan against the heads' lengths (entries before the arriving one)."""
    hdr, wrange, desc = kv.debug_plan(layer)
    pieces, groups, warps, append = (int(x) for x in hdr)
    assert append == 1 and warps == wrange.shape[0]
    g = {u: (n + 1 + 15) // 16 for u, n in lengths.items()}
    assert groups == sum(g.values())
    # pieces: head after head, j = 0 .. k - 1
    i = 0
    first = {}
    for u in sorted(g):
        k = int(desc[i, 2])
        assert k >= 1
        first[u] = i
        for j in range(k):
            assert tuple(desc[i + j, :3]) == (u, j, k), (u, j, desc[i + j])
            assert desc[i + j, 3] == desc[i, 3]
        i += k
    assert i == pieces
    # every piece belongs to exactly one warp
    owner = np.full(pieces, -1)
    for w in range(warps):
        a, b = wrange[w]
        assert 0 <= a <= b <= pieces
        assert (owner[a:b] == -1).all()
        owner[a:b] = w
    assert (owner >= 0).all()
    # heads marked `together`: consecutive warps of one CTA, nothing else in those warps (mark 1), or
    # the same for every run of eight pieces and the shorter last run (mark 2)
    together = 0
    for u in g:
        k, i0, mark = int(desc[first[u], 2]), first[u], int(desc[first[u], 3])
        if mark:
            assert (mark == 1) == (k <= 8)
            for r0 in range(0, k, 8):
                ws = owner[i0 + r0:i0 + min(k, r0 + 8)]
                assert (np.diff(ws) == 1).all() and ws[0] // 8 == ws[-1] // 8, (u, ws)
                assert k <= 8 or r0 + 8 > k or ws[0] % 8 == 0
                assert all(wrange[w][1] - wrange[w][0] == 1 for w in ws)
            together += 1
    # with at most one piece per warp, every head of two or more pieces is placed that way
    if pieces <= warps:
        assert together == sum(1 for u in g if desc[first[u], 2] >= 2)
    longest = max(-(-g[u] // int(desc[first[u], 2])) for u in g)
    return pieces, warps, together, longest, groups


def test_launch_plans_keep_each_head_inside_one_cta():
    """Heads of very different lengths in one launch: some need more than the eight warps of a
    CTA (whole CTAs plus a shorter run elsewhere, merged through global memory), most need two to
    eight (all in one CTA, merged in its shared memory), the shortest are one piece.  The plan is
    checked as a structure, the outputs and the cache against the oracle."""
    wl = Workload(name="mixed", seed=31, n_layers=2, n_q_heads=16, n_kv_heads=8, batch=2, prompt=3000,
                  think_steps=12, budget_per_head=3100)
    ls = LockStep(wl, [0, 1])
    ls.prefill()
    new = [3000, 2200, 1400, 840, 600, 340, 200, 128, 100, 66, 34, 1800, 2600, 500, 1040, 150]
    for seq in range(2):
        for h in range(8):
            b = new[seq * 8 + h]
            for layer in range(2):
                ls.gpu.set_budget(layer, seq, h, b)
                ls.ora.set_budget(layer, seq, h, b)
    ls.compare()
    lengths = {seq * 8 + h: len(ls.gpu.get_retained(0, seq, h)) for seq in range(2) for h in range(8)}
    assert sorted(lengths.values()) == sorted(new)
    pieces, warps, together, longest, groups = _check_plan(ls.gpu, 0, lengths, 8)
    assert together >= 6
    assert longest <= max(12, 2 * -(-groups // warps))      # no warp streams much more than its share (a small launch
                                                            # takes pieces of up to 12 groups to keep heads inside a CTA)
    hdr, wrange, desc = ls.gpu.debug_plan(0)
    assert {int(x) for x in desc[:pieces, 3]} == {0, 1, 2}  # one piece, one CTA, runs of eight: all three kinds of head
    for _ in range(12):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


def test_launch_plans_after_reallocations_are_all_inside_ctas():
    """The 14B shape after reallocations: every head of two to eight pieces has them in one CTA."""
    wl = WORKLOADS["cfg4_qwen14b"].scaled(n_layers=2, think_steps=300)
    from paper_2601_16986_b200 import Config, CrystalKV
    dev = torch.device("cuda", 0)
    kv = CrystalKV(Config(n_layers=2, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, batch=wl.batch,
                          budget_per_head=wl.budget_per_head, max_context=wl.prompt + 400, top_p=wl.top_p, lam=wl.lam))
    for l in range(2):
        k, v = wl.prompt_kv(l, device=dev)
        kv.prefill(l, k, v, wl.queries(l, [wl.prompt - 1], device=dev)[:, 0].contiguous())
    out = torch.empty(wl.batch, wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device=dev)
    for s in range(256):
        pos = [wl.prompt + s]
        for l in range(2):
            kv.decode_step(l, wl.queries(l, pos, device=dev)[:, 0].contiguous(), wl.keys(l, pos, device=dev)[:, 0].contiguous(),
                           wl.values(l, pos, device=dev)[:, 0].contiguous(), out)
        if (s + 1) % 128 == 0:
            kv.rebudget()
    kv.check()
    H = wl.n_kv_heads
    for l in range(2):
        lengths = {seq * H + h: len(kv.get_retained(l, seq, h)) for seq in range(wl.batch) for h in range(H)}
        pieces, warps, together, longest, groups = _check_plan(kv, l, lengths, H)
        assert together == len(lengths)          # (budgets of 300 and more: no head is a single piece here)
        assert longest <= -(-groups // warps) * 1.25 + 1
    kv.close()


# ------------------------------------------------------------------ full-size shapes, sampled
def _run_sampled(name, sample, n_steps, cmp_every, answer=0, max_answer=0):
    wl = WORKLOADS[name]
    wl = wl.scaled(think_steps=n_steps, answer_steps=answer)
    ls = LockStep(wl, sample, max_answer_tokens=max_answer)
    ls.prefill()
    ls.compare()
    for s in range(n_steps):
        ls.step(compare_state=((s + 1) % cmp_every == 0))
        if wl.rebudget_every and (s + 1) % wl.rebudget_every == 0:
            ls.rebudget()
    ls.compare()
    if answer:
        ls.set_stage_answer()
        for _ in range(answer):
            ls.step(compare_state=False)
        ls.compare()
    ls.gpu.check()
    report(name, ls, f" (state compared every {cmp_every} steps and around every reallocation)")
    ls.assert_clean()
    return ls


def test_cfg2_qwen7b_shape_sampled():
    """7B shape (28 layers, 28q/4kv, batch 8, budget 1024): 512 steps to fill every head, then
    more than 500 steps in which Algorithm 1 step 4 runs on every head."""
    ls = _run_sampled("cfg2_qwen7b", [7], steps(1056), 32)
    assert len(ls.gpu.get_retained(27, 7, 3)) == 1024
    ls.close()


def test_cfg3_llama8b_shape_sampled():
    """8B shape (32 layers, 32q/8kv, batch 16, B_total = 2048 x heads), reallocation every 128:
    past the point where the cache of a sequence is full (1536 steps after a 512-token prompt), so
    that the last reallocations move slots between full heads and step 4 runs everywhere."""
    ls = _run_sampled("cfg3_llama8b", [15], steps(1728), 32)
    assert ls.rep.budgets_compared >= (13 if SCALE >= 1 else 0)
    b = ls.gpu.get_budgets()
    assert (b.reshape(16, -1).sum(axis=1) == 2048 * 32 * 8).all()
    ls.close()


def test_cfg4_qwen14b_shape_sampled():
    """14B shape (48 layers, 40q/8kv, batch 32, B_total = 1024 x heads), reallocation every 128,
    then answer steps: the configuration the bench times."""
    ls = _run_sampled("cfg4_qwen14b", [31], steps(1024), 32, answer=4, max_answer=8)
    assert ls.rep.budgets_compared >= (8 if SCALE >= 1 else 0)
    b = ls.gpu.get_budgets()
    assert (b.reshape(32, -1).sum(axis=1) == 1024 * 48 * 8).all() and (b != 1024).any()
    ls.close()


def test_cfg5_sweep_cells_sampled():
    """Two cells of the 14B sweep (fewer layers: the layers are independent without
    reallocation): small budget with a long prompt, and a large budget."""
    for batch, budget, prompt, n in [(8, 256, 200, steps(120)), (1, 4096, 4000, steps(150))]:
        wl = WORKLOADS["cfg5_sweep14b"].scaled(n_layers=4, batch=batch, budget_per_head=budget,
                                               prompt=prompt, think_steps=n)
        ls = LockStep(wl, [batch - 1])
        ls.prefill()
        for s in range(n):
            ls.step(compare_state=((s + 1) % 30 == 0))
        ls.compare()
        ls.gpu.check()
        ls.assert_clean()
        assert len(ls.gpu.get_retained(3, batch - 1, 7)) == budget
        ls.close()


def test_more_heads_than_warps_in_the_grid():
    """batch x kv heads above the attention grid's warp count (148 SMs x 8): every warp takes
    several whole heads in turn instead of one piece."""
    wl = Workload(name="wide", seed=61, n_layers=1, n_q_heads=24, n_kv_heads=8, batch=180, prompt=37,
                  think_steps=24, budget_per_head=44, outlier="flat", outlier_frac=0.05)
    ls = LockStep(wl, [0, 97, 179])
    ls.prefill()
    ls.compare()
    for s in range(wl.think_steps):
        ls.step(compare_state=(s % 4 == 3))
    ls.compare()
    ls.gpu.check()
    ls.assert_clean()
    assert len(ls.gpu.get_retained(0, 179, 7)) == 44
    ls.close()


@pytest.mark.parametrize("G", [1, 2, 3, 6, 7, 8])
def test_large_launch_merges_inside_the_cta_for_every_group_size(G):
    """A launch large enough that CTAs take eight pieces at once: three pieces per head, so some
    heads lie inside one CTA (merged through shared memory) and some straddle two (merged through
    global memory), for group sizes other than those of the named shapes."""
    wl = Workload(name=f"big{G}", seed=500 + G, n_layers=1, n_q_heads=8 * G, n_kv_heads=8, batch=40,
                  prompt=600, think_steps=24, budget_per_head=600, outlier="flat", outlier_frac=0.03)
    ls = LockStep(wl, [0, 17, 39])
    ls.prefill()
    ls.compare()
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


def test_window_prefill_and_buffered_cadence_in_a_large_launch():
    """The observation window's causal views and the eviction of several entries per call, in a
    launch large enough that CTAs take eight pieces at once and merge in shared memory."""
    wl = Workload(name="bigwin", seed=611, n_layers=1, n_q_heads=40, n_kv_heads=8, batch=40,
                  prompt=640, think_steps=20, budget_per_head=600, outlier="perhead")
    ls = LockStep(wl, [0, 21, 39], max_answer_tokens=64, evict_every=5)
    ls.prefill_window(6)
    ls.compare()
    ls.gpu.validate()
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    assert len(ls.gpu.get_retained(0, 39, 7)) in range(600, 605)
    ls.close()


def test_very_long_heads_use_the_general_lrfu_path():
    """A head above 17 x 256 entries: the LRFU kernel keeps pbar in global scratch, the attention
    kernel cuts the head into many pieces (merge in several rounds)."""
    wl = Workload(name="long", seed=62, n_layers=1, n_q_heads=4, n_kv_heads=1, batch=2, prompt=4500,
                  think_steps=12, budget_per_head=4504)
    ls = LockStep(wl, [0, 1])
    ls.prefill()
    ls.compare()
    for s in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    assert len(ls.gpu.get_retained(0, 1, 0)) == 4504
    ls.close()


def test_host_buffer_steps_match_device_steps():
    """crystalkv_decode_step_host with pinned buffers (the kernel reads them over PCIe) and with
    pageable buffers (staged copies) gives the outputs and the state of the device-pointer call."""
    import ctypes as C
    from paper_2601_16986_b200 import Config, CrystalKV
    wl = Workload(name="hostio", seed=21, n_layers=2, n_q_heads=10, n_kv_heads=2, batch=3, prompt=50,
                  think_steps=40, budget_per_head=64)
    def make():
        kv = CrystalKV(Config(n_layers=2, n_q_heads=10, n_kv_heads=2, batch=3, budget_per_head=64, max_context=256))
        for l in range(2):
            k, v = wl.prompt_kv(l, device="cuda")
            kv.prefill(l, k, v, wl.queries(l, [wl.prompt - 1], device="cuda")[:, 0].contiguous())
        return kv
    dev, pin, page = make(), make(), make()
    for s in range(40):
        for l in range(2):
            q, k, v = wl.step_inputs(l, wl.prompt + s, device="cuda")
            ref = dev.decode_step(l, q, k, v)
            hq, hk, hv = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
            ho = torch.empty_like(hq).pin_memory()
            pin.decode_step_host(l, hq, hk, hv, ho)
            # pageable: plain tensors through the C ABI
            pq, pk, pv = q.cpu(), k.cpu(), v.cpu()
            po = torch.empty_like(pq)
            P = lambda t: C.c_void_p(t.data_ptr())
            rc = page.lib.crystalkv_decode_step_host(page._h, l, P(pq), P(pk), P(pv), P(po),
                                                     C.c_void_p(torch.cuda.current_stream().cuda_stream))
            assert rc == 0
            pin.join()
            page.join()
            torch.cuda.synchronize()
            assert torch.equal(ho, ref.cpu()) and torch.equal(po, ref.cpu())
    # the same without a host synchronisation between calls: the staging sets are reused several
    # times over while earlier copies may still be in flight
    refs, outs, keep = [], [], []
    for s in range(40, 130):
        for l in range(2):
            q, k, v = wl.step_inputs(l, wl.prompt + s, device="cuda")
            refs.append(dev.decode_step(l, q, k, v))
            hq, hk, hv = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
            ho = torch.empty_like(hq).pin_memory()
            pin.decode_step_host(l, hq, hk, hv, ho)
            keep.append((hq, hk, hv))
            outs.append(ho)
    pin.join()
    torch.cuda.synchronize()
    assert all(torch.equal(o, r.cpu()) for o, r in zip(outs, refs))
    page.close()
    page = pin   # the pageable handle stopped at step 40; the final state is compared for the other two
    for l in range(2):
        for b in range(3):
            for h in range(2):
                a = dev.export_state(l, b, h)
                assert (a == pin.export_state(l, b, h)).all() and (a == page.export_state(l, b, h)).all()
    for kv in (dev, pin):
        kv.check()
        kv.validate()
        kv.close()


def test_a_smaller_handle_created_later_leaves_a_larger_one_working():
    """Function attributes (the attention kernel's shared-memory limit) are per function, not per
    handle: a handle with few heads created after one with many must not lower them."""
    from paper_2601_16986_b200 import Config, CrystalKV
    wl = Workload(name="many", seed=71, n_layers=1, n_q_heads=16, n_kv_heads=8, batch=200, prompt=20,
                  think_steps=12, budget_per_head=24)
    ls = LockStep(wl, [0, 199])
    ls.prefill()
    for _ in range(4):
        ls.step()
    small = CrystalKV(Config(n_layers=1, n_q_heads=2, n_kv_heads=1, batch=1, budget_per_head=8, max_context=64))
    z = torch.zeros(1, 6, 1, 128, dtype=torch.bfloat16, device="cuda")
    small.prefill(0, z, z, torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda"))
    small.decode_step(0, torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda"), z[:, 0], z[:, 0])
    small.check()
    for _ in range(8):
        ls.step()                       # the larger handle still launches
    ls.gpu.check()
    ls.assert_clean()
    small.close()
    ls.close()


def test_a_handle_rebuilt_from_exports_continues_like_the_original():
    """Every head exported (records and K/V rows) after 120 steps with two reallocations, the handle
    destroyed, a fresh handle rebuilt by import alone (no prefill), 60 more steps on both the rebuilt
    handle and an uninterrupted twin: budgets and state bit for bit, outputs within the tolerance, ownership sound."""
    from paper_2601_16986_b200 import Config, CrystalKV, CrystalKVError
    wl = Workload(name="ckpt", seed=123, n_layers=3, n_q_heads=10, n_kv_heads=2, batch=2, prompt=70,
                  think_steps=180, budget_per_head=64, rebudget_every=50, outlier="perhead", outlier_lo=0.01, outlier_hi=0.3)
    cfg = Config(n_layers=3, n_q_heads=10, n_kv_heads=2, batch=2, budget_per_head=64, max_context=300, min_budget=8)

    def fresh(prefill=True):
        kv = CrystalKV(cfg)
        if prefill:
            for l in range(3):
                k, v = wl.prompt_kv(l, device="cuda")
                kv.prefill(l, k, v, wl.queries(l, [wl.prompt - 1], device="cuda")[:, 0].contiguous())
        return kv

    def run(kv, s0, s1):
        outs = []
        for s in range(s0, s1):
            for l in range(3):
                outs.append(kv.decode_step(l, *wl.step_inputs(l, wl.prompt + s, device="cuda")).clone())
            if (s + 1) % wl.rebudget_every == 0:
                kv.rebudget()
        return outs

    a, twin = fresh(), fresh()
    run(a, 0, 120); run(twin, 0, 120)
    budgets = a.get_budgets()
    saved = {}
    for l in range(3):
        for b in range(2):
            for h in range(2):
                rec = a.export_state(l, b, h)
                k, v = a.export_kv(l, b, h)
                pos = rec[:, 0].tolist()
                assert torch.equal(k, wl.keys(l, pos, seqs=[b])[0, :, h]) and torch.equal(v, wl.values(l, pos, seqs=[b])[0, :, h])
                saved[(l, b, h)] = (rec, k.contiguous(), v.contiguous())
    t = a.time(0)
    a.close()
    c = fresh(prefill=False)
    with pytest.raises(CrystalKVError):                       # a record after the layer's time
        rec, k, v = saved[(0, 0, 0)]
        bad = rec.copy(); bad[0, 2] = t + 5
        c.import_state(0, 0, 0, bad, k, v, int(budgets[0, 0, 0]), t)
    for (l, b, h), (rec, k, v) in saved.items():
        perm = np.random.default_rng(l * 7 + b * 3 + h).permutation(len(rec))     # any order is accepted
        c.import_state(l, b, h, rec[perm], k[torch.as_tensor(perm)].contiguous(), v[torch.as_tensor(perm)].contiguous(),
                       int(budgets[b, l, h]), t)
    with pytest.raises(CrystalKVError):                       # the layer is at time t now
        rec, k, v = saved[(1, 1, 1)]
        c.import_state(1, 1, 1, rec, k, v, 0, t + 1)
    c.check(); c.validate()
    assert (c.get_budgets() == budgets).all()
    oc, ot = run(c, 120, 180), run(twin, 120, 180)
    # (the rebuilt heads list their entries in another order, so sums run in another order: outputs
    # agree to the last bf16 digit or so, the state exactly)
    assert max(float((x.float() - y.float()).abs().max()) for x, y in zip(oc, ot)) <= 2e-2
    assert (c.get_budgets() == twin.get_budgets()).all()
    for l in range(3):
        for b in range(2):
            for h in range(2):
                assert (c.export_state(l, b, h) == twin.export_state(l, b, h)).all()
    for kv in (c, twin):
        kv.check(); kv.validate(); kv.close()


# ------------------------------------------------------------------ error paths on a live handle
@pytest.mark.parametrize("W,prompt,budget", [(1, 83, 53), (8, 83, 53), (32, 200, 96), (40, 40, 64), (16, 300, 256)])
def test_observation_window_prefill(W, prompt, budget):
    """Algorithm 1 replayed over the last W prompt queries (causal views, steps 1-3 each, one
    eviction after the last), then think steps; window outputs, state and ownership compared."""
    wl = Workload(name=f"win{W}", seed=300 + W, n_layers=2, n_q_heads=10, n_kv_heads=2, batch=3,
                  prompt=prompt, think_steps=40, budget_per_head=budget, outlier="flat", outlier_frac=0.05)
    ls = LockStep(wl, [0, 2], max_answer_tokens=max(64, prompt - budget + 8))
    ls.prefill_window(W)
    ls.compare()
    ls.gpu.validate()
    for h in range(2):
        assert len(ls.gpu.get_retained(1, 2, h)) == min(prompt, budget)
    for _ in range(wl.think_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    ls.close()


@pytest.mark.parametrize("m,literal,prompt,budget", [(8, 0, 83, 53), (16, 0, 40, 64), (3, 1, 30, 64), (1, 1, 83, 53),
                                                     (64, 0, 300, 256)])
def test_buffered_cadence_and_literal_return(m, literal, prompt, budget):
    """Eviction once a head is m entries over its budget (m leave per call) and Algorithm 1's
    early return as printed; head lengths cycle between B and B + m - 1."""
    wl = Workload(name=f"cad{m}", seed=400 + m, n_layers=2, n_q_heads=8, n_kv_heads=2, batch=3,
                  prompt=prompt, think_steps=3 * m + 60, budget_per_head=budget, outlier="flat", outlier_frac=0.05)
    ls = LockStep(wl, [0, 2], max_answer_tokens=max(40, prompt - budget + 8), evict_every=m, literal_return=literal)
    ls.prefill()
    ls.compare()
    sizes = set()
    for s in range(wl.think_steps):
        ls.step()
        sizes.add(len(ls.gpu.get_retained(0, 0, 0)))
        if s % 7 == 0:
            ls.gpu.validate()
    ls.gpu.check()
    ls.assert_clean()
    assert max(sizes) == budget + m - 1 and budget in sizes
    ls.close()


def test_buffered_cadence_with_reallocation_and_answer_stage():
    """The buffered heads through Algorithm 2 (shrinking releases every spare but one) and into
    the answer stage (which uses up the spares a head still owns before it takes new slots)."""
    wl = Workload(name="cadre", seed=77, n_layers=3, n_q_heads=8, n_kv_heads=2, batch=2, prompt=64,
                  think_steps=100, answer_steps=12, budget_per_head=48, outlier="perhead", outlier_lo=0.01, outlier_hi=0.3)
    ls = LockStep(wl, [0, 1], min_budget=8, max_answer_tokens=16, evict_every=6)
    ls.prefill()
    for s in range(wl.think_steps):
        ls.step()
        if (s + 1) % 25 == 0:
            ls.rebudget()
    ls.set_stage_answer()
    for _ in range(wl.answer_steps):
        ls.step()
    ls.gpu.check()
    ls.assert_clean()
    assert ls.rep.budgets_compared > 0
    ls.close()


def test_call_order_errors():
    from paper_2601_16986_b200 import Config, CrystalKV, CrystalKVError
    kv = CrystalKV(Config(n_layers=2, n_q_heads=4, n_kv_heads=2, batch=1, budget_per_head=32, max_context=64))
    q = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(CrystalKVError) as e:
        kv.decode_step(0, q, k, k)
    assert e.value.code == -2
    pk = torch.zeros(1, 8, 2, 128, dtype=torch.bfloat16, device="cuda")
    kv.prefill(0, pk, pk, q)
    with pytest.raises(CrystalKVError):
        kv.prefill(0, pk, pk, q)              # twice
    with pytest.raises(CrystalKVError):
        kv.rebudget()                         # layer 1 not prefilled: layers out of step
    with pytest.raises(CrystalKVError):
        kv.decode_step(5, q, k, k)            # bad layer
    kv.decode_step(0, q, k, k)
    kv.check()
    kv.close()
