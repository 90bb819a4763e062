"""ctypes binding of libcrystalkv.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  PyTorch is used for device
memory and streams; a missing library or a missing GPU is an error, never a fallback.
"""
from __future__ import annotations

import ctypes as C
import os
import re
from dataclasses import dataclass

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libcrystalkv.so")
HEADER = os.path.join(os.path.dirname(HERE), "include", "crystalkv.h")

THINK, ANSWER = 0, 1
EVICT, FULLKV = 0, 1
BF16 = 1


class CrystalKVError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"crystalkv error {code}: {text}")
        self.code = code


class _Cfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("batch", C.c_int32), ("dtype", C.c_int32),
                ("budget_per_head", C.c_int32), ("min_budget", C.c_int32), ("max_budget", C.c_int32),
                ("max_answer_tokens", C.c_int32), ("max_context", C.c_int32), ("top_p", C.c_float),
                ("lam", C.c_float), ("sm_scale", C.c_float), ("mode", C.c_int32), ("device", C.c_int32),
                ("evict_every", C.c_int32), ("literal_return", C.c_int32), ("budget_ratio", C.c_float)]


@dataclass
class Config:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    batch: int
    budget_per_head: int
    max_context: int
    head_dim: int = 128
    min_budget: int = 0
    max_budget: int = 0
    max_answer_tokens: int = 0
    top_p: float = 0.9
    lam: float = 0.6
    sm_scale: float = 0.0
    mode: int = EVICT
    device: int = 0
    dtype: int = BF16
    evict_every: int = 1
    literal_return: int = 0
    budget_ratio: float = 0.0


def declared_symbols():
    """Names of the functions include/crystalkv.h declares."""
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(crystalkv_[a-z_]+)\s*\(", text)))


_lib = None


def load_library():
    """Loads the in-tree shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise CrystalKVError(-100, f"{LIB_PATH} is missing: run `python -m paper_2601_16986_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, p32 = C.c_void_p, C.c_int, C.POINTER(C.c_int32)
    lib.crystalkv_create.argtypes = [C.POINTER(_Cfg), C.POINTER(vp)]
    lib.crystalkv_destroy.argtypes = [vp]
    lib.crystalkv_prefill.argtypes = [vp, i32, vp, vp, vp, i32, vp]
    lib.crystalkv_prefill_window.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp, vp]
    lib.crystalkv_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.crystalkv_decode_step_host.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.crystalkv_set_stage.argtypes = [vp, i32]
    lib.crystalkv_join.argtypes = [vp, vp]
    lib.crystalkv_rebudget.argtypes = [vp, vp]
    lib.crystalkv_get_retained.argtypes = [vp, i32, i32, i32, vp, C.c_int32, p32, vp]
    lib.crystalkv_get_budgets.argtypes = [vp, vp, vp]
    lib.crystalkv_export_state.argtypes = [vp, i32, i32, i32, vp, C.c_int32, p32, vp]
    lib.crystalkv_export_kv.argtypes = [vp, i32, i32, i32, vp, vp, C.c_int32, p32, vp]
    lib.crystalkv_import_state.argtypes = [vp, i32, i32, i32, vp, C.c_int32, vp, vp, C.c_int32, C.c_int32, vp]
    lib.crystalkv_set_budget.argtypes = [vp, i32, i32, i32, C.c_int32, vp]
    lib.crystalkv_time.argtypes = [vp, i32]
    lib.crystalkv_get_counters.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), vp]
    lib.crystalkv_check.argtypes = [vp, vp]
    lib.crystalkv_validate.argtypes = [vp, vp]
    lib.crystalkv_validate_static.argtypes = [vp, vp, vp]
    lib.crystalkv_debug_set_page.argtypes = [vp, i32, i32, i32, C.c_int32, C.c_int32, vp]
    lib.crystalkv_debug_get_plan.argtypes = [vp, i32, vp, vp, C.c_int32, vp, C.c_int32, vp]
    lib.crystalkv_debug_ctas_needed.argtypes = [C.c_int32, vp]
    lib.crystalkv_strerror.argtypes = [i32]
    lib.crystalkv_strerror.restype = C.c_char_p
    lib.crystalkv_last_error.argtypes = [vp]
    lib.crystalkv_last_error.restype = C.c_char_p
    _lib = lib
    return lib


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, shape=None):
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise ValueError("expected a contiguous bf16 CUDA tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return C.c_void_p(t.data_ptr())


class CrystalKV:
    """One handle = the compressed KV cache of `batch` sequences on one GPU."""

    def __init__(self, cfg: Config):
        if not torch.cuda.is_available():
            raise CrystalKVError(-101, "no CUDA device: this library has no CPU path")
        self.lib = load_library()
        self.cfg = cfg
        c = _Cfg(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.batch, cfg.dtype,
                 cfg.budget_per_head, cfg.min_budget, cfg.max_budget, cfg.max_answer_tokens,
                 cfg.max_context, cfg.top_p, cfg.lam, cfg.sm_scale, cfg.mode, cfg.device,
                 cfg.evict_every, cfg.literal_return, cfg.budget_ratio)
        h = C.c_void_p()
        rc = self.lib.crystalkv_create(C.byref(c), C.byref(h))
        if rc:
            raise CrystalKVError(rc, self.lib.crystalkv_last_error(None).decode())
        self._h = h
        self._cap = max(cfg.max_context, 4 * cfg.budget_per_head, cfg.max_budget) + cfg.max_answer_tokens + 8

    def _ck(self, rc):
        if rc:
            raise CrystalKVError(rc, self.lib.crystalkv_strerror(rc).decode() + ": " +
                                 self.lib.crystalkv_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self.lib.crystalkv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the calls of the C ABI, same names
    def prefill(self, layer, k, v, q_last):
        c = self.cfg
        P = k.shape[1]
        self._ck(self.lib.crystalkv_prefill(self._h, layer, _dev(k, (c.batch, P, c.n_kv_heads, c.head_dim)),
                                            _dev(v, (c.batch, P, c.n_kv_heads, c.head_dim)),
                                            _dev(q_last, (c.batch, c.n_q_heads, c.head_dim)), P, _stream()))

    def prefill_window(self, layer, k, v, q_window, out_window=None):
        c = self.cfg
        P, W = k.shape[1], q_window.shape[0]
        shape_q = (W, c.batch, c.n_q_heads, c.head_dim)
        self._ck(self.lib.crystalkv_prefill_window(
            self._h, layer, _dev(k, (c.batch, P, c.n_kv_heads, c.head_dim)),
            _dev(v, (c.batch, P, c.n_kv_heads, c.head_dim)), _dev(q_window, shape_q), P, W,
            None if out_window is None else _dev(out_window, shape_q), _stream()))
        return out_window

    def decode_step(self, layer, q, k_new, v_new, out=None):
        c = self.cfg
        if out is None:
            out = torch.empty_like(q)
        self._ck(self.lib.crystalkv_decode_step(
            self._h, layer, _dev(q, (c.batch, c.n_q_heads, c.head_dim)),
            _dev(k_new, (c.batch, c.n_kv_heads, c.head_dim)), _dev(v_new, (c.batch, c.n_kv_heads, c.head_dim)),
            _dev(out, (c.batch, c.n_q_heads, c.head_dim)), _stream()))
        return out

    def decode_step_host(self, layer, q, k_new, v_new, out):
        """Pinned host bf16 tensors in and out; copies are enqueued on the current stream."""
        for t in (q, k_new, v_new, out):
            if t.is_cuda or not t.is_pinned() or t.dtype != torch.bfloat16 or not t.is_contiguous():
                raise ValueError("expected contiguous pinned host bf16 tensors")
        self._ck(self.lib.crystalkv_decode_step_host(self._h, layer, C.c_void_p(q.data_ptr()),
                                                     C.c_void_p(k_new.data_ptr()), C.c_void_p(v_new.data_ptr()),
                                                     C.c_void_p(out.data_ptr()), _stream()))
        return out

    def join(self):
        self._ck(self.lib.crystalkv_join(self._h, _stream()))

    def set_stage(self, stage):
        self._ck(self.lib.crystalkv_set_stage(self._h, stage))

    def rebudget(self):
        self._ck(self.lib.crystalkv_rebudget(self._h, _stream()))

    def get_retained(self, layer, seq, kv_head) -> np.ndarray:
        buf = np.zeros(self._cap, dtype=np.int32)
        n = C.c_int32(0)
        self._ck(self.lib.crystalkv_get_retained(self._h, layer, seq, kv_head, buf.ctypes.data_as(C.c_void_p),
                                                 self._cap, C.byref(n), _stream()))
        return buf[:n.value].copy()

    def get_budgets(self) -> np.ndarray:
        c = self.cfg
        out = np.zeros((c.batch, c.n_layers, c.n_kv_heads), dtype=np.int32)
        self._ck(self.lib.crystalkv_get_budgets(self._h, out.ctypes.data_as(C.c_void_p), _stream()))
        return out

    def export_state(self, layer, seq, kv_head) -> np.ndarray:
        buf = np.zeros((self._cap, 3), dtype=np.int32)
        n = C.c_int32(0)
        self._ck(self.lib.crystalkv_export_state(self._h, layer, seq, kv_head, buf.ctypes.data_as(C.c_void_p),
                                                 self._cap, C.byref(n), _stream()))
        return buf[:n.value].copy()

    def export_kv(self, layer, seq, kv_head):
        """K and V rows of one head in the order of export_state's records: two host bf16 tensors [n, 128]."""
        k = torch.empty(self._cap, self.cfg.head_dim, dtype=torch.bfloat16)
        v = torch.empty(self._cap, self.cfg.head_dim, dtype=torch.bfloat16)
        n = C.c_int32(0)
        self._ck(self.lib.crystalkv_export_kv(self._h, layer, seq, kv_head, C.c_void_p(k.data_ptr()),
                                              C.c_void_p(v.data_ptr()), self._cap, C.byref(n), _stream()))
        return k[:n.value].clone(), v[:n.value].clone()

    def import_state(self, layer, seq, kv_head, rec: np.ndarray, k: torch.Tensor, v: torch.Tensor, budget: int, t: int):
        """Rebuilds one head from records [n, 3] and host bf16 rows k, v [n, 128]; budget 0 keeps the current one."""
        rec = np.ascontiguousarray(rec, dtype=np.int32)
        for x in (k, v):
            if x.is_cuda or x.dtype != torch.bfloat16 or not x.is_contiguous() or tuple(x.shape) != (len(rec), self.cfg.head_dim):
                raise ValueError("expected contiguous host bf16 rows [n, head_dim]")
        self._ck(self.lib.crystalkv_import_state(self._h, layer, seq, kv_head, rec.ctypes.data_as(C.c_void_p), len(rec),
                                                 C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()), int(budget), int(t),
                                                 _stream()))

    def set_budget(self, layer, seq, kv_head, budget):
        self._ck(self.lib.crystalkv_set_budget(self._h, layer, seq, kv_head, int(budget), _stream()))

    def time(self, layer) -> int:
        return self.lib.crystalkv_time(self._h, layer)

    def get_counters(self):
        a, b, c = C.c_uint64(0), C.c_uint64(0), C.c_uint64(0)
        self._ck(self.lib.crystalkv_get_counters(self._h, C.byref(a), C.byref(b), C.byref(c), _stream()))
        return {"entries_attended": a.value, "hits": b.value, "evictions": c.value}

    def check(self):
        self._ck(self.lib.crystalkv_check(self._h, _stream()))

    def validate(self):
        self._ck(self.lib.crystalkv_validate(self._h, _stream()))

    def debug_plan(self, layer: int):
        """Launch plan of the layer's next attention kernel (test hook): hdr int32[4], wrange
        int32[warps, 2], desc int32[warps + heads, 4] as the header describes them."""
        warps = 8 * torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
        heads = self.cfg.batch * self.cfg.n_kv_heads
        hdr = np.zeros(4, dtype=np.int32)
        wrange = np.zeros((warps, 2), dtype=np.int32)
        desc = np.zeros((warps + heads, 4), dtype=np.int32)
        vp = C.c_void_p
        self._ck(self.lib.crystalkv_debug_get_plan(self._h, layer, hdr.ctypes.data_as(vp), wrange.ctypes.data_as(vp), warps,
                                                   desc.ctypes.data_as(vp), warps + heads, _stream()))
        return hdr, wrange, desc

    def validate_static(self) -> np.ndarray:
        """The same check without any device allocation (scratch built into the library; at
        most 2**17 pool pages).  Returns int32[2]: page ids out of range, pages not owned exactly once."""
        counts = np.full(2, -1, dtype=np.int32)
        self._ck(self.lib.crystalkv_validate_static(self._h, counts.ctypes.data_as(C.c_void_p), _stream()))
        return counts
