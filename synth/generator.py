"""Counter-based synthetic Q/K/V generator (bit-identical on CPU and CUDA).

Every value is ``table[hash32(seed, stream, seq, layer, head, pos, channel) >> 16]``
where ``table`` holds the 65 536 standard-normal quantiles ``Phi^-1((i + 0.5) / 65536)``
rounded to bf16.  All integer mixing is done on int64 tensors that hold 32-bit
unsigned values, with every product kept below 2**63, so the arithmetic is exact and
device independent.

Structure added on top of the iid N(0,1) draw, for keys only:

* the key at position 0 of every (seq, layer, kv head) is scaled x8 (attention sink);
* "outlier" keys are scaled x3.  A key is an outlier when a separate 32-bit hash of
  (seed, seq, layer, head, pos) falls below ``f * 2**32``; ``f`` is either one flat
  fraction or a per-(layer, head) fraction drawn uniformly from ``[f_lo, f_hi]``.

The recipes for the named workloads stand in for reasoning traces of R1-distilled
models (shapes, think lengths and budgets only; no dataset item or weight is used).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Sequence

import torch

_M32 = 0xFFFFFFFF
# odd multipliers below 2**31 so that (32-bit value) * multiplier < 2**63
_C1 = 0x7FEB352D
_C2 = 0x2C1B3C6D
_C3 = 0x297A2D39
_ADD = 0x632BE5AB

STREAM_Q, STREAM_K, STREAM_V, STREAM_OUTLIER, STREAM_FRAC = 1, 2, 3, 4, 5


def _mix(h: torch.Tensor) -> torch.Tensor:
    """32-bit avalanche on an int64 tensor holding values in [0, 2**32)."""
    h = h ^ (h >> 16)
    h = (h * _C1) & _M32
    h = h ^ (h >> 15)
    h = (h * _C2) & _M32
    h = h ^ (h >> 13)
    h = (h * _C3) & _M32
    h = h ^ (h >> 16)
    return h


def _absorb(h: torch.Tensor, x) -> torch.Tensor:
    """Fold one more counter field into the running hash."""
    return _mix(((h ^ x) + _ADD) & _M32)


_TABLE_CACHE = {}


def normal_table(device="cpu") -> torch.Tensor:
    """65 536 N(0,1) quantiles as bf16; computed once on the host in fp64."""
    key = str(device)
    if key not in _TABLE_CACHE:
        if "cpu" not in _TABLE_CACHE:
            i = torch.arange(65536, dtype=torch.float64)
            z = torch.special.ndtri((i + 0.5) / 65536.0)
            _TABLE_CACHE["cpu"] = z.to(torch.float32).to(torch.bfloat16)
        _TABLE_CACHE[key] = _TABLE_CACHE["cpu"].to(device)
    return _TABLE_CACHE[key]


@dataclass(frozen=True)
class Workload:
    """Shape and structure of one synthetic decode workload."""

    name: str
    seed: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    batch: int
    prompt: int
    think_steps: int
    answer_steps: int = 0
    budget_per_head: int = 1024
    rebudget_every: int = 0            # 0 = static uniform budgets
    head_dim: int = 128
    outlier: str = "none"              # "none" | "flat" | "perhead"
    outlier_frac: float = 0.02         # flat fraction
    outlier_lo: float = 0.005          # per-head fractions ~ U(lo, hi)
    outlier_hi: float = 0.05
    top_p: float = 0.9
    lam: float = 0.6

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def scaled(self, **kw) -> "Workload":
        """A smaller (or otherwise modified) copy; same recipe, other sizes."""
        return replace(self, **kw)

    # ------------------------------------------------------------------ hashing
    def _base(self, stream: int, device) -> torch.Tensor:
        h = torch.tensor([self.seed & _M32], dtype=torch.int64, device=device)
        return _absorb(_mix(h), stream)

    def _field(self, stream, seqs, layer, heads, positions, device):
        """Hash of (seed, stream, seq, layer, head, pos): shape [S, P, Hh]."""
        seqs = torch.as_tensor(seqs, dtype=torch.int64, device=device).view(-1, 1, 1)
        pos = torch.as_tensor(positions, dtype=torch.int64, device=device).view(1, -1, 1)
        hd = torch.arange(heads, dtype=torch.int64, device=device).view(1, 1, -1)
        h = self._base(stream, device)
        h = _absorb(h, seqs)
        h = _absorb(h, int(layer))
        h = _absorb(h, hd)
        h = _absorb(h, pos)
        return h

    def _draw(self, stream, seqs, layer, heads, positions, device) -> torch.Tensor:
        """bf16 tensor [S, P, heads, head_dim] of table-normal values."""
        h = self._field(stream, seqs, layer, heads, positions, device).unsqueeze(-1)
        ch = torch.arange(self.head_dim, dtype=torch.int64, device=device).view(1, 1, 1, -1)
        h = _absorb(h, ch)
        return normal_table(device)[(h >> 16)]

    def outlier_fraction(self, layer: int, device="cpu") -> torch.Tensor:
        """Per-kv-head outlier fraction f_{layer,h} as float64 [H]."""
        H = self.n_kv_heads
        if self.outlier == "none":
            return torch.zeros(H, dtype=torch.float64, device=device)
        if self.outlier == "flat":
            return torch.full((H,), self.outlier_frac, dtype=torch.float64, device=device)
        hd = torch.arange(H, dtype=torch.int64, device=device)
        h = _absorb(_absorb(self._base(STREAM_FRAC, device), int(layer)), hd)
        u = h.to(torch.float64) / 4294967296.0
        return self.outlier_lo + (self.outlier_hi - self.outlier_lo) * u

    # ------------------------------------------------------------------ tensors
    def queries(self, layer: int, positions, seqs: Optional[Sequence[int]] = None,
                device="cpu") -> torch.Tensor:
        """Query states, bf16 [S, P, n_q_heads, head_dim]."""
        seqs = range(self.batch) if seqs is None else seqs
        return self._draw(STREAM_Q, list(seqs), layer, self.n_q_heads, positions, device)

    def values(self, layer: int, positions, seqs=None, device="cpu") -> torch.Tensor:
        """Value rows, bf16 [S, P, n_kv_heads, head_dim]."""
        seqs = range(self.batch) if seqs is None else seqs
        return self._draw(STREAM_V, list(seqs), layer, self.n_kv_heads, positions, device)

    def keys(self, layer: int, positions, seqs=None, device="cpu") -> torch.Tensor:
        """Key rows with the sink and outlier scaling, bf16 [S, P, n_kv_heads, head_dim]."""
        seqs = list(range(self.batch) if seqs is None else seqs)
        H = self.n_kv_heads
        k = self._draw(STREAM_K, seqs, layer, H, positions, device)
        pos = torch.as_tensor(positions, dtype=torch.int64, device=device).view(1, -1, 1)
        scale = torch.ones(k.shape[:3], dtype=torch.float32, device=device)
        if self.outlier != "none":
            ho = self._field(STREAM_OUTLIER, seqs, layer, H, positions, device)
            thr = (self.outlier_fraction(layer, device) * 4294967296.0).to(torch.int64)
            scale = torch.where(ho < thr.view(1, 1, -1), 3.0, 1.0).to(torch.float32)
        scale = torch.where(pos == 0, torch.full_like(scale, 8.0), scale)
        return (k.to(torch.float32) * scale.unsqueeze(-1)).to(torch.bfloat16)

    def is_outlier(self, layer: int, positions, seqs=None, device="cpu") -> torch.Tensor:
        """bool [S, P, n_kv_heads]: which keys carry the x3 outlier scaling."""
        seqs = list(range(self.batch) if seqs is None else seqs)
        H = self.n_kv_heads
        if self.outlier == "none":
            return torch.zeros(len(seqs), len(positions), H, dtype=torch.bool, device=device)
        ho = self._field(STREAM_OUTLIER, seqs, layer, H, positions, device)
        thr = (self.outlier_fraction(layer, device) * 4294967296.0).to(torch.int64)
        return ho < thr.view(1, 1, -1)

    # convenience wrappers with the shapes the library's calls take
    def prompt_kv(self, layer: int, seqs=None, device="cpu"):
        """(k, v), each [S, prompt, H, d]."""
        pos = torch.arange(self.prompt)
        return self.keys(layer, pos, seqs, device), self.values(layer, pos, seqs, device)

    def step_inputs(self, layer: int, pos: int, seqs=None, device="cpu"):
        """(q [S, Hq, d], k_new [S, H, d], v_new [S, H, d]) for the token at ``pos``."""
        q = self.queries(layer, [pos], seqs, device)[:, 0]
        k = self.keys(layer, [pos], seqs, device)[:, 0]
        v = self.values(layer, [pos], seqs, device)[:, 0]
        return q.contiguous(), k.contiguous(), v.contiguous()


def _mk(idx, **kw) -> Workload:
    return Workload(seed=20260116 + idx, **kw)


# The five benchmark configurations (synthetic stand-ins; see the module docstring).
WORKLOADS = {
    "cfg1_gqa4_b512": _mk(1, name="cfg1_gqa4_b512", n_layers=1, n_q_heads=8, n_kv_heads=2,
                          batch=1, prompt=256, think_steps=2048, budget_per_head=512,
                          outlier="none"),
    "cfg2_qwen7b": _mk(2, name="cfg2_qwen7b", n_layers=28, n_q_heads=28, n_kv_heads=4,
                       batch=8, prompt=512, think_steps=8192, budget_per_head=1024,
                       outlier="flat", outlier_frac=0.02),
    "cfg3_llama8b": _mk(3, name="cfg3_llama8b", n_layers=32, n_q_heads=32, n_kv_heads=8,
                        batch=16, prompt=512, think_steps=16384, budget_per_head=2048,
                        rebudget_every=128, outlier="perhead"),
    "cfg4_qwen14b": _mk(4, name="cfg4_qwen14b", n_layers=48, n_q_heads=40, n_kv_heads=8,
                        batch=32, prompt=1024, think_steps=8192, answer_steps=256,
                        budget_per_head=1024, rebudget_every=128, outlier="perhead"),
    "cfg5_sweep14b": _mk(5, name="cfg5_sweep14b", n_layers=48, n_q_heads=40, n_kv_heads=8,
                         batch=32, prompt=1024, think_steps=32768, budget_per_head=1024,
                         outlier="none"),
}
