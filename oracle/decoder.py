"""CPU ORACLE -- test infrastructure, not product code.

ctypes front end of ``decoder.c`` (the plain C decoder forward, with and without a KV
cache).  Only tests, the smoke check and the benchmark's CPU-baseline leg may import this.
The C file is compiled on demand with gcc into ``oracle/_build/``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "decoder.c")
_OUT = os.path.join(_HERE, "_build", "liboracle_decoder.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_OUT) or os.path.getmtime(_OUT) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_OUT), exist_ok=True)
        tmp = _OUT + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _OUT)
    return _OUT


class OrcArch(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab", "max_pos", "norm", "act",
        "pos", "parallel_residual", "has_bias", "tie_lm_head", "dtype", "rotary_dim")] + [
        ("rotary_base", ctypes.c_float), ("norm_eps", ctypes.c_float)]


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, f32p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_float)
        L.orc_set_threads.argtypes = [i32]
        L.orc_get_threads.restype = i32
        L.orc_round_bf16.argtypes = [ctypes.c_float]
        L.orc_round_bf16.restype = ctypes.c_float
        L.orc_gelu.argtypes = [ctypes.c_float]
        L.orc_gelu.restype = ctypes.c_float
        L.orc_silu.argtypes = [ctypes.c_float]
        L.orc_silu.restype = ctypes.c_float
        L.orc_linear.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32]
        L.orc_norm.argtypes = [vp, vp, vp, vp, i32, i32, i32, ctypes.c_float]
        L.orc_rotary.argtypes = [vp, i32, i32, ctypes.c_float]
        L.orc_attend.argtypes = [vp, vp, vp, vp, i32, i32, ctypes.c_size_t]
        L.orc_forward_full.argtypes = [ctypes.POINTER(OrcArch), vp, vp, i32, vp]
        L.orc_forward_full.restype = i32
        L.orc_forward_cached.argtypes = [ctypes.POINTER(OrcArch), vp, vp, i32, i32, vp, i32, vp]
        L.orc_forward_cached.restype = i32
        L.orc_attention_rows.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp]
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


def get_threads() -> int:
    return int(lib().orc_get_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a: np.ndarray, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


# ---- primitives (exposed so each can be pinned on its own) ----
def linear(x, W, b=None, dtype=0):
    x = _c(x, np.float32)
    W = _c(W, np.uint16 if dtype else np.float32)
    M, Kd = x.shape
    N = W.shape[0]
    assert W.shape[1] == Kd
    y = np.empty((M, N), np.float32)
    bb = None if b is None else _c(b, np.float32)
    lib().orc_linear(_ptr(y), _ptr(x), _ptr(W), _ptr(bb), M, N, Kd, dtype)
    return y


def norm(x, g, b, kind, eps):
    x = _c(x, np.float32)
    g = _c(g, np.float32)
    bb = None if b is None else _c(b, np.float32)
    y = np.empty_like(x)
    lib().orc_norm(_ptr(y), _ptr(x), _ptr(g), _ptr(bb), x.shape[0], x.shape[1], kind, eps)
    return y


def gelu(v: float) -> float:
    return float(lib().orc_gelu(v))


def silu(v: float) -> float:
    return float(lib().orc_silu(v))


def round_bf16(v: float) -> float:
    return float(lib().orc_round_bf16(v))


def rotary(vec, rd, pos, base=10000.0):
    v = _c(vec, np.float32).copy()
    lib().orc_rotary(_ptr(v), rd, pos, base)
    return v


def attend(q, keys, vals):
    q = _c(q, np.float32)
    keys = _c(keys, np.float32)
    vals = _c(vals, np.float32)
    n, Dh = keys.shape
    out = np.empty(Dh, np.float32)
    lib().orc_attend(_ptr(out), _ptr(q), _ptr(keys), _ptr(vals), n, Dh, Dh)
    return out


def attention_rows(q, kv_layer, len_, m):
    """q [m, H*Dh] (position-encoded), kv_layer [2, H, S_max, Dh] fp32; row r sees 0..len_+r."""
    q = _c(q, np.float32)
    kv_layer = _c(kv_layer, np.float32)
    _, H, S, Dh = kv_layer.shape
    o = np.empty((m, H * Dh), np.float32)
    lib().orc_attention_rows(_ptr(q), _ptr(kv_layer), H, Dh, S, len_, m, _ptr(o))
    return o


class Model:
    """A model = architecture fields + the tensor list of ``tensor order`` (see decoder.c enums)."""

    def __init__(self, arch, weights: Sequence[Optional[np.ndarray]]):
        fields = {n: getattr(arch, n) for n, _ in OrcArch._fields_}
        self.arch = OrcArch(**fields)
        self.a = arch
        self._keep: List[Optional[np.ndarray]] = []
        for w in weights:
            if w is None:
                self._keep.append(None)
            elif w.ndim == 2:
                self._keep.append(_c(w, np.uint16 if arch.dtype else np.float32))
            else:
                self._keep.append(_c(w, np.float32))
        n = len(self._keep)
        assert n == 2 + 12 * arch.n_layers + 3, n
        self._ptrs = (ctypes.c_void_p * n)(*[None if w is None else w.ctypes.data for w in self._keep])

    def forward_full(self, tokens) -> np.ndarray:
        tok = _c(tokens, np.int32)
        out = np.empty((tok.shape[0], self.a.vocab), np.float32)
        rc = lib().orc_forward_full(ctypes.byref(self.arch), self._ptrs, _ptr(tok), tok.shape[0], _ptr(out))
        assert rc == 0
        return out

    def new_cache(self, s_max: int) -> "Cache":
        return Cache(self, s_max)


class Cache:
    """KV cache of one sequence: [L][2][H][S_max][Dh] fp32 storage and a committed length."""

    def __init__(self, model: Model, s_max: int):
        a = model.a
        self.model = model
        self.s_max = s_max
        self.kv = np.zeros((a.n_layers, 2, a.n_heads, s_max, a.head_dim), np.float32)
        self.len = 0

    def feed(self, tokens, want_logits: bool = True, advance: bool = True) -> Optional[np.ndarray]:
        """Feed tokens at positions len.. ; by default the rows are committed (len advances)."""
        tok = _c(np.atleast_1d(tokens), np.int32)
        m = tok.shape[0]
        out = np.empty((m, self.model.a.vocab), np.float32) if want_logits else None
        rc = lib().orc_forward_cached(ctypes.byref(self.model.arch), self.model._ptrs, _ptr(self.kv),
                                      self.s_max, self.len, _ptr(tok), m, _ptr(out))
        if rc != 0:
            raise ValueError("rows do not fit the cache / position table")
        if advance:
            self.len += m
        return out

    def rollback(self, new_len: int) -> None:
        assert 0 <= new_len <= self.len
        self.len = new_len
