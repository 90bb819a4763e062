"""ctypes front end of the C oracle (TEST INFRASTRUCTURE; see crystalkv_oracle.c).

Argument marshalling only: every number comes out of the C file.  bf16 tensors cross
as their uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np
import torch

from . import build as _build

THINK, ANSWER = 0, 1
EVICT, FULLKV = 0, 1
TIE_EVICT, TIE_NUCLEUS = 1, 2


class _Cfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("batch", C.c_int32), ("budget_per_head", C.c_int32),
                ("min_budget", C.c_int32), ("max_budget", C.c_int32), ("max_context", C.c_int32),
                ("mode", C.c_int32), ("top_p", C.c_float), ("lam", C.c_float),
                ("sm_scale", C.c_float), ("tie_eps", C.c_double),
                ("evict_every", C.c_int32), ("literal_return", C.c_int32), ("budget_ratio", C.c_float)]


@dataclass
class OracleConfig:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    batch: int
    budget_per_head: int
    max_context: int
    head_dim: int = 128
    min_budget: int = 0
    max_budget: int = 0          # 0 -> budget_per_head * n_layers * n_kv_heads (no cap)
    mode: int = EVICT
    top_p: float = 0.9
    lam: float = 0.6
    sm_scale: float = 0.0        # 0 -> 1/sqrt(head_dim)
    tie_eps: float = 1e-6
    evict_every: int = 1         # m: evict once a head is m entries over its budget
    literal_return: int = 0      # 1: no tracking while a head is below its budget (Algorithm 1, first line)
    budget_ratio: float = 0.0    # r > 0: the average budget per head follows the context, floor(r * tokens)


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(_build.build())
        vp, i32 = C.c_void_p, C.c_int
        lib.okv_create.restype = vp
        lib.okv_create.argtypes = [C.POINTER(_Cfg)]
        lib.okv_destroy.argtypes = [vp]
        lib.okv_set_stage.argtypes = [vp, i32]
        lib.okv_prefill.argtypes = [vp, i32, vp, vp, vp, i32]
        lib.okv_prefill_window.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp]
        lib.okv_decode_step.argtypes = [vp, i32, vp, vp, vp, vp]
        lib.okv_rebudget.argtypes = [vp]
        lib.okv_get_retained.argtypes = [vp, i32, i32, i32, vp, i32]
        lib.okv_get_budgets.argtypes = [vp, vp]
        lib.okv_set_budget.argtypes = [vp, i32, i32, i32, i32]
        lib.okv_time.argtypes = [vp, i32]
        lib.okv_export_state.argtypes = [vp, i32, i32, i32, vp, i32]
        lib.okv_import_state.argtypes = [vp, i32, i32, i32, vp, i32, vp, vp]
        lib.okv_replay_unit.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32]
        lib.okv_ratio_budget.argtypes = [vp, i32]
        lib.okv_tie_count.argtypes = [vp]
        lib.okv_get_ties.argtypes = [vp, vp, i32]
        lib.okv_clear_ties.argtypes = [vp]
        lib.okv_decay.argtypes = [vp, i32]
        lib.okv_decay.restype = C.c_float
        lib.okv_attention.argtypes = [vp, vp, vp, i32, i32, i32, C.c_double, vp, vp]
        lib.okv_hit_mask.argtypes = [vp, vp, i32, C.c_double, vp, C.c_double, vp]
        lib.okv_alg2.argtypes = [vp, vp, i32, i32, C.c_int64, C.c_int32, C.c_int32, vp]
        _lib = lib
    return _lib


def _bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> contiguous uint16 numpy array of its bit patterns."""
    assert t.dtype == torch.bfloat16
    return np.ascontiguousarray(t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


# ---------------------------------------------------------------- free functions
def attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, scale: float):
    """q [G,d], k [n,d], v [n,d] bf16 -> (prob [G,n] f64, y [G,d] f64)."""
    lib = _load()
    G, d = q.shape
    n = k.shape[0]
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    kp = (C.c_void_p * n)(*[kb[i].ctypes.data for i in range(n)])
    vp = (C.c_void_p * n)(*[vb[i].ctypes.data for i in range(n)])
    prob = np.zeros((G, n), dtype=np.float64)
    y = np.zeros((G, d), dtype=np.float64)
    lib.okv_attention(_p(qb), kp, vp, n, G, d, float(scale), _p(prob), _p(y))
    return prob, y


def hit_mask(pbar, pos, top_p: float, rel_eps: float = 1e-6):
    """-> (hit uint8 [n], near_tie bool)."""
    lib = _load()
    pbar = np.ascontiguousarray(pbar, dtype=np.float64)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    hit = np.zeros(len(pbar), dtype=np.uint8)
    near = C.c_int(0)
    lib.okv_hit_mask(_p(pbar), _p(pos), len(pbar), float(top_p), _p(hit), float(rel_eps), C.byref(near))
    return hit, bool(near.value)


def alg2(A, B, B_total: int, min_b: int = 0, max_b: int = 0):
    """A, B [L,H] -> new integer budgets [L,H]."""
    lib = _load()
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.int32)
    L, H = A.shape
    out = np.zeros((L, H), dtype=np.int32)
    lib.okv_alg2(_p(A), _p(B), L, H, int(B_total), int(min_b), int(max_b or B_total), _p(out))
    return out


# ---------------------------------------------------------------- stateful oracle
class Oracle:
    def __init__(self, cfg: OracleConfig):
        lib = _load()
        self.cfg = cfg
        max_b = cfg.max_budget or cfg.budget_per_head * cfg.n_layers * cfg.n_kv_heads
        self._c = _Cfg(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.batch,
                       cfg.budget_per_head, cfg.min_budget, max_b, cfg.max_context, cfg.mode,
                       cfg.top_p, cfg.lam, cfg.sm_scale, cfg.tie_eps, cfg.evict_every, cfg.literal_return,
                       cfg.budget_ratio)
        self._h = lib.okv_create(C.byref(self._c))
        if not self._h:
            raise ValueError("oracle: bad config")
        self._lib = lib

    def close(self):
        if self._h:
            self._lib.okv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stage(self, stage: int):
        self._lib.okv_set_stage(self._h, stage)

    def prefill(self, layer, k, v, q_last):
        """k, v [batch,P,H,d]; q_last [batch,Hq,d] (bf16)."""
        P = k.shape[1]
        kb, vb, qb = _bits(k), _bits(v), _bits(q_last)
        rc = self._lib.okv_prefill(self._h, layer, _p(kb), _p(vb), _p(qb), P)
        if rc:
            raise RuntimeError("oracle prefill failed")

    def prefill_window(self, layer, k, v, q_win) -> np.ndarray:
        """k, v [batch,P,H,d]; q_win [W,batch,Hq,d] (bf16), the queries of the last W prompt
        tokens -> their causal attention outputs [W,batch,Hq,d] float32."""
        P, W = k.shape[1], q_win.shape[0]
        kb, vb, qb = _bits(k), _bits(v), _bits(q_win)
        y = np.zeros(q_win.shape, dtype=np.float32)
        rc = self._lib.okv_prefill_window(self._h, layer, _p(kb), _p(vb), _p(qb), P, W, _p(y))
        if rc:
            raise RuntimeError("oracle prefill_window failed")
        return y

    def decode_step(self, layer, q, k_new, v_new) -> np.ndarray:
        """-> out [batch,Hq,d] float32."""
        qb, kb, vb = _bits(q), _bits(k_new), _bits(v_new)
        out = np.zeros(q.shape, dtype=np.float32)
        rc = self._lib.okv_decode_step(self._h, layer, _p(qb), _p(kb), _p(vb), _p(out))
        if rc:
            raise RuntimeError("oracle decode_step failed")
        return out

    def rebudget(self):
        if self._lib.okv_rebudget(self._h):
            raise RuntimeError("oracle rebudget failed")

    def get_retained(self, layer, seq, head) -> np.ndarray:
        cap = self.cfg.max_context + 2
        buf = np.zeros(cap, dtype=np.int32)
        n = self._lib.okv_get_retained(self._h, layer, seq, head, _p(buf), cap)
        assert n >= 0
        return buf[:n].copy()

    def get_budgets(self) -> np.ndarray:
        c = self.cfg
        out = np.zeros((c.batch, c.n_layers, c.n_kv_heads), dtype=np.int32)
        self._lib.okv_get_budgets(self._h, _p(out))
        return out

    def set_budget(self, layer, seq, head, budget):
        self._lib.okv_set_budget(self._h, layer, seq, head, int(budget))

    def time(self, layer) -> int:
        return self._lib.okv_time(self._h, layer)

    def ratio_budget(self, tokens: int) -> int:
        """Average budget per head after `tokens` tokens under the configured ratio."""
        return int(self._lib.okv_ratio_budget(self._h, int(tokens)))

    def export_state(self, layer, seq, head) -> np.ndarray:
        """-> int32 [n,3] rows (pos, crf bits, tau) sorted by pos."""
        cap = self.cfg.max_context + 2
        buf = np.zeros((cap, 3), dtype=np.int32)
        n = self._lib.okv_export_state(self._h, layer, seq, head, _p(buf), cap)
        assert n >= 0
        return buf[:n].copy()

    def import_state(self, layer, seq, head, rec: np.ndarray, k: torch.Tensor, v: torch.Tensor):
        rec = np.ascontiguousarray(rec, dtype=np.int32)
        kb, vb = _bits(k), _bits(v)
        self._lib.okv_import_state(self._h, layer, seq, head, _p(rec), len(rec), _p(kb), _p(vb))

    def replay_unit(self, rec, k, v, budget, t_first, q, k_new, v_new, flips, append_first=True) -> np.ndarray:
        """One head replayed outside the oracle's state from records rec [n,3] with rows k, v [n,d]:
        len(flips) think steps at times t_first, t_first+1, .. with queries q [steps,G,d] and arriving
        rows [steps,d], flips[s] moving the hit boundary of step s (0 none, 1 one hit more, 2 one
        fewer, 3 swap).  append_first=False: the first step is a prefill's scoring pass (nothing
        arrives).  -> final records [m,3] sorted by position."""
        rec = np.ascontiguousarray(rec, dtype=np.int32)
        flips = np.ascontiguousarray(flips, dtype=np.int32)
        kb, vb, qb, knb, vnb = _bits(k), _bits(v), _bits(q), _bits(k_new), _bits(v_new)
        cap = len(rec) + len(flips) + 1
        out = np.zeros((cap, 3), dtype=np.int32)
        n = self._lib.okv_replay_unit(self._h, _p(rec), _p(kb), _p(vb), len(rec), int(budget), int(t_first), int(bool(append_first)), len(flips),
                                      _p(qb), _p(knb), _p(vnb), _p(flips), _p(out), cap)
        assert n >= 0
        return out[:n].copy()

    def ties(self) -> np.ndarray:
        """-> int32 [m,5] rows (layer, seq, head, t, kind)."""
        m = self._lib.okv_tie_count(self._h)
        buf = np.zeros((max(m, 1), 5), dtype=np.int32)
        m = self._lib.okv_get_ties(self._h, _p(buf), m)
        return buf[:m].copy()

    def clear_ties(self):
        self._lib.okv_clear_ties(self._h)

    def decay(self, D: int) -> float:
        return float(self._lib.okv_decay(self._h, D))
