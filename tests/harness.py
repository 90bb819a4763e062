"""Lock-step GPU <-> oracle comparison (test infrastructure).

Both sides get the same seeded inputs.  The GPU library runs the whole batch; the oracle
runs a sample of whole sequences (sequences are independent).  Compared:

* attention outputs, max-abs against the fp32 oracle output (tolerance 2e-2 for bf16);
* the per-entry state (position, CRF bits, tau) of every sampled head, which contains the
  retained position set;
* budgets after every reallocation.

A state mismatch is accepted only when the oracle logged a tie (a decision within 1e-6
relative of flipping) for that head since the last comparison; the oracle is then
re-synchronised from the GPU state.  Anything else is an unexplained mismatch.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from oracle import Oracle, OracleConfig
from paper_2601_16986_b200 import ANSWER, Config, CrystalKV
from synth import Workload

OUT_TOL = 2e-2


@dataclass
class Report:
    steps: int = 0
    heads_compared: int = 0
    tie_explained: int = 0
    unexplained: list = field(default_factory=list)
    max_out_err: float = 0.0
    budgets_compared: int = 0
    ties_logged: int = 0


class LockStep:
    def __init__(self, wl: Workload, sample_seqs, mode=0, min_budget=0, max_budget=0,
                 max_answer_tokens=0, device="cuda", evict_every=1, literal_return=0):
        self.wl, self.seqs, self.dev = wl, list(sample_seqs), device
        ctx = wl.prompt + wl.think_steps + wl.answer_steps + 2
        self.gpu = CrystalKV(Config(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                                    batch=wl.batch, budget_per_head=wl.budget_per_head, max_context=ctx,
                                    min_budget=min_budget, max_budget=max_budget,
                                    max_answer_tokens=max_answer_tokens, top_p=wl.top_p, lam=wl.lam, mode=mode,
                                    evict_every=evict_every, literal_return=literal_return))
        bph = wl.budget_per_head
        self.ora = Oracle(OracleConfig(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                                       batch=len(self.seqs), budget_per_head=bph, max_context=ctx,
                                       min_budget=min_budget or min(bph, max(16, bph // 8)),
                                       max_budget=max_budget or 4 * bph, top_p=wl.top_p, lam=wl.lam, mode=mode,
                                       evict_every=evict_every, literal_return=literal_return))
        self.rep = Report()
        self.t = wl.prompt - 1
        self._tie_seen = 0

    def close(self):
        self.gpu.close()
        self.ora.close()

    # ------------------------------------------------------------------ driving
    def prefill(self):
        wl = self.wl
        for l in range(wl.n_layers):
            k, v = wl.prompt_kv(l, device=self.dev)
            q = wl.queries(l, [wl.prompt - 1], device=self.dev)[:, 0].contiguous()
            self.gpu.prefill(l, k, v, q)
            idx = torch.tensor(self.seqs, device=self.dev)
            self.ora.prefill(l, k[idx].cpu(), v[idx].cpu(), q[idx].cpu())
        self.gpu.check()

    def prefill_window(self, W):
        """Prompt with the last W queries replayed; the window's attention outputs are compared too."""
        wl = self.wl
        idx = torch.tensor(self.seqs, device=self.dev)
        for l in range(wl.n_layers):
            k, v = wl.prompt_kv(l, device=self.dev)
            q = wl.queries(l, list(range(wl.prompt - W, wl.prompt)), device=self.dev).transpose(0, 1).contiguous()
            out = torch.zeros_like(q)
            self.gpu.prefill_window(l, k, v, q, out)
            ref = self.ora.prefill_window(l, k[idx].cpu(), v[idx].cpu(), q[:, idx].cpu())
            err = float(np.abs(out[:, idx].float().cpu().numpy() - ref).max())
            self.rep.max_out_err = max(self.rep.max_out_err, err)
        self.gpu.check()

    def step(self, compare_state=True, layers=None):
        """One token through every layer on both sides."""
        wl = self.wl
        self.t += 1
        idx = torch.tensor(self.seqs, device=self.dev)
        for l in range(wl.n_layers):
            q, k, v = wl.step_inputs(l, self.t, device=self.dev)
            out = self.gpu.decode_step(l, q, k, v)
            ref = self.ora.decode_step(l, q[idx].cpu(), k[idx].cpu(), v[idx].cpu())
            err = float((out[idx].float().cpu().numpy() - ref).__abs__().max())
            self.rep.max_out_err = max(self.rep.max_out_err, err)
        self.rep.steps += 1
        if compare_state:
            self.compare(layers)

    def set_stage_answer(self):
        self.gpu.set_stage(ANSWER)
        self.ora.set_stage(1)

    def rebudget(self):
        self.compare()                 # equal states going in => budgets must be bit-equal
        self.gpu.rebudget()
        self.ora.rebudget()
        g = self.gpu.get_budgets()
        o = self.ora.get_budgets()
        for si, s in enumerate(self.seqs):
            self.rep.budgets_compared += 1
            if not (g[s] == o[si]).all():
                self.rep.unexplained.append(("budgets", s, self.t))
        self.compare()
        self.gpu.check()
        self.gpu.validate()

    # ------------------------------------------------------------------ comparing
    def _new_ties(self):
        ties = self.ora.ties()
        new = ties[self._tie_seen:]
        self._tie_seen = len(ties)
        self.rep.ties_logged = len(ties)
        return {(int(r[0]), int(r[1]), int(r[2])) for r in new}

    def compare(self, layers=None):
        wl = self.wl
        tied = self._new_ties() | getattr(self, "_pending_ties", set())
        pending = set()
        for l in (range(wl.n_layers) if layers is None else layers):
            for si, s in enumerate(self.seqs):
                for h in range(wl.n_kv_heads):
                    g = self.gpu.export_state(l, s, h)
                    o = self.ora.export_state(l, si, h)
                    self.rep.heads_compared += 1
                    if g.shape == o.shape and (g == o).all():
                        continue
                    if (l, si, h) in tied:
                        self.rep.tie_explained += 1
                        pos = g[:, 0].tolist()
                        k = wl.keys(l, pos, seqs=[s])[0, :, h]
                        v = wl.values(l, pos, seqs=[s])[0, :, h]
                        self.ora.import_state(l, si, h, g, k, v)
                    else:
                        self.rep.unexplained.append(("state", l, s, h, self.t))
        if layers is not None:  # ties of layers not compared now stay pending
            pending = {x for x in tied if x[0] not in set(layers)}
        self._pending_ties = pending

    def assert_clean(self):
        self.gpu.validate()          # every slot owned exactly once
        r = self.rep
        assert not r.unexplained, f"unexplained mismatches: {r.unexplained[:8]} (of {len(r.unexplained)})"
        assert r.max_out_err <= OUT_TOL, f"max |out_gpu - out_oracle| = {r.max_out_err}"
