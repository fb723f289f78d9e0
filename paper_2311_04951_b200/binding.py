"""ctypes binding of the C ABI in ``include/ssd.h``: same names, argument marshalling only.

torch supplies device memory and streams; every step of the path runs in the library's own
kernels.  Loading fails loudly when the compiled library is missing: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

_LIB = None

SSD_OK = 0
MAX_ROWS = 64
MAX_ROWS_PER_SEQ = 32


class SsdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class SsdArch(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab", "max_pos", "norm", "act",
        "pos", "parallel_residual", "has_bias", "tie_lm_head", "dtype", "rotary_dim")] + [
        ("rotary_base", ctypes.c_float), ("norm_eps", ctypes.c_float)]


EXPORTS = ["ssd_model_create", "ssd_model_desc_bytes", "ssd_set_persistent", "ssd_set_attention_mode", "ssd_model_share_prefix", "ssd_model_destroy", "ssd_kv_bytes",
           "ssd_workspace_bytes", "kv_init", "kv_destroy", "kv_prefill", "draft_step", "target_verify",
           "kv_commit", "kv_rollback", "spec_advance", "kv_lengths", "ssd_device_status",
           "verify_from_logits", "verify_from_logits_noalloc", "verify_scratch_bytes", "attention_rows", "ssd_last_logits", "ssd_set_trace", "ssd_read_trace", "ssd_launch_count",
           "ssd_gemm_profile", "ssd_gemm_profile_read", "ssd_strerror", "ssd_set_wait_limit", "ssd_wait_probe", "ssd_set_sampling", "draft_steps",
           "ssd_prefill_workspace_bytes", "ssd_set_prefill_mode"]


def lib_path() -> str:
    return _build.LIB


def load():
    """Load the compiled CUDA library.  Raises if it has not been built."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2311_04951_b200.build` "
                           "(there is no non-CUDA fallback)")
    L = ctypes.CDLL(path)
    vp, i32, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t, ctypes.c_float
    pp = ctypes.POINTER(ctypes.c_void_p)
    L.ssd_model_create.argtypes = [ctypes.POINTER(SsdArch), pp, i32, vp, sz, pp]
    L.ssd_model_desc_bytes.argtypes = [ctypes.POINTER(SsdArch)]
    L.ssd_model_desc_bytes.restype = sz
    L.ssd_set_persistent.argtypes = [i32]
    L.ssd_set_attention_mode.argtypes = [i32]
    L.ssd_set_prefill_mode.argtypes = [i32]
    L.ssd_prefill_workspace_bytes.argtypes = [vp, i32, i32]
    L.ssd_prefill_workspace_bytes.restype = sz
    L.ssd_model_share_prefix.argtypes = [vp, i32, pp]
    L.ssd_model_destroy.argtypes = [vp]
    L.ssd_model_destroy.restype = None
    L.ssd_kv_bytes.argtypes = [vp, i32, i32]
    L.ssd_kv_bytes.restype = sz
    L.ssd_workspace_bytes.argtypes = [vp, i32, i32, i32]
    L.ssd_workspace_bytes.restype = sz
    L.kv_init.argtypes = [vp, i32, i32, vp, sz, vp, pp]
    L.kv_destroy.argtypes = [vp]
    L.kv_destroy.restype = None
    L.kv_prefill.argtypes = [vp, vp, vp, vp, i32, vp, sz, vp]
    L.draft_step.argtypes = [vp, vp, vp, i32, i32, vp, f32, vp, i32, vp, i32, vp, sz, vp, sz, vp]
    L.draft_steps.argtypes = [vp, vp, i32, vp, i32, i32, vp, f32, vp, i32, vp, i32, vp, sz, vp, sz, vp]
    L.target_verify.argtypes = [vp, vp, vp, i32, vp, vp, f32, vp, vp, i32, vp, vp, sz, vp]
    L.kv_commit.argtypes = [vp, vp, vp]
    L.kv_rollback.argtypes = [vp, vp, vp]
    L.spec_advance.argtypes = [vp, vp, vp, i32, vp, vp, i32, vp, i32, vp, vp, vp, vp]
    L.kv_lengths.argtypes = [vp, vp, vp]
    L.ssd_device_status.argtypes = [vp, vp, vp]
    L.verify_from_logits.argtypes = [vp, i32, i32, i32, vp, vp, vp, f32, vp, vp, i32, vp, vp, sz, vp]
    L.verify_from_logits_noalloc.argtypes = [vp, i32, i32, i32, vp, vp, vp, f32, vp, vp, i32, vp, vp]
    L.verify_scratch_bytes.argtypes = [i32, i32]
    L.verify_scratch_bytes.restype = sz
    L.attention_rows.argtypes = [vp, vp, i32, vp, i32, vp, vp, sz, vp]
    L.ssd_last_logits.argtypes = [vp, i32, i32, vp, sz, vp, vp]
    L.ssd_set_trace.argtypes = [i32]
    L.ssd_read_trace.argtypes = [vp, i32, i32, vp, sz, vp, i32, ctypes.POINTER(ctypes.c_int), vp]
    L.ssd_launch_count.restype = ctypes.c_uint64
    L.ssd_gemm_profile.argtypes = [i32]
    L.ssd_gemm_profile_read.argtypes = [ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_double), i32]
    L.ssd_set_sampling.argtypes = [i32, f32]
    L.ssd_set_wait_limit.argtypes = [ctypes.c_longlong]
    L.ssd_wait_probe.argtypes = [vp, vp]
    L.ssd_strerror.argtypes = [i32]
    L.ssd_strerror.restype = ctypes.c_char_p
    _LIB = L
    return L


def strerror(code: int) -> str:
    return load().ssd_strerror(int(code)).decode()


def _check(rc: int, where: str) -> None:
    if rc != SSD_OK:
        raise SsdError(rc, where)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def device_buffer(nbytes: int) -> torch.Tensor:
    """Every device block this binding hands to the library (descriptor table, cache slab, workspace) comes
    from here: uint8, 256-byte aligned.  Tests replace it to put guard bands around the blocks."""
    return torch.empty(max(int(nbytes), 1), dtype=torch.uint8, device="cuda")


def arch_struct(arch) -> SsdArch:
    return SsdArch(**{n: getattr(arch, n) for n, _ in SsdArch._fields_})


def upload_weights(arch, weights: Sequence[Optional[np.ndarray]], device="cuda") -> List[Optional[torch.Tensor]]:
    """numpy tensors (bf16 as uint16 bit patterns) -> device tensors in the ABI's tensor order."""
    out = []
    for w in weights:
        if w is None:
            out.append(None)
        elif w.dtype == np.uint16:
            out.append(torch.from_numpy(w.view(np.int16)).to(device).view(torch.bfloat16))
        else:
            out.append(torch.from_numpy(np.ascontiguousarray(w, np.float32)).to(device))
    return out


class Model:
    """ssd_model handle; keeps the device tensors it borrows alive."""

    def __init__(self, arch, tensors: Sequence[Optional[torch.Tensor]], _handle=None, _parent=None):
        self.arch = arch
        self.tensors = list(tensors)
        self._parent = _parent
        if _handle is not None:
            self.h = _handle
            return
        L = load()
        n = len(self.tensors)
        ptrs = (ctypes.c_void_p * n)(*[None if t is None else t.data_ptr() for t in self.tensors])
        h = ctypes.c_void_p()
        a = arch_struct(arch)
        nd = int(L.ssd_model_desc_bytes(ctypes.byref(a)))
        self.desc = device_buffer(nd) if nd else None
        _check(L.ssd_model_create(ctypes.byref(a), ptrs, n, _p(self.desc), nd, ctypes.byref(h)), "ssd_model_create")
        self.h = h

    def share_prefix(self, n_layers: int) -> "Model":
        h = ctypes.c_void_p()
        _check(load().ssd_model_share_prefix(self.h, n_layers, ctypes.byref(h)), "ssd_model_share_prefix")
        keep = 2 + 12 * n_layers
        return Model(self.arch.replace(n_layers=n_layers), self.tensors[:keep] + self.tensors[-3:], _handle=h,
                     _parent=self)

    def kv_bytes(self, batch: int, max_len: int) -> int:
        return int(load().ssd_kv_bytes(self.h, batch, max_len))

    def workspace_bytes(self, batch: int, rows_per_seq: int, max_len: int) -> int:
        return int(load().ssd_workspace_bytes(self.h, batch, rows_per_seq, max_len))

    def prefill_workspace_bytes(self, batch: int, rows_per_seq: int) -> int:
        """Workspace of the many-row prompt pass (0: this model has none)."""
        return int(load().ssd_prefill_workspace_bytes(self.h, batch, rows_per_seq))

    def new_workspace(self, batch: int, rows_per_seq: int, max_len: int) -> torch.Tensor:
        n = self.workspace_bytes(batch, rows_per_seq, max_len)
        if n == 0:
            raise SsdError(-3, "ssd_workspace_bytes")
        return device_buffer(n)

    def __del__(self):
        try:
            if getattr(self, "h", None):
                load().ssd_model_destroy(self.h)
                self.h = None
        except Exception:
            pass


class KV:
    """ssd_kv handle over a torch-owned slab."""

    def __init__(self, model: Model, batch: int, max_len: int):
        self.model, self.batch, self.max_len = model, batch, max_len
        n = model.kv_bytes(batch, max_len)
        self.buf = device_buffer(n)
        h = ctypes.c_void_p()
        _check(load().kv_init(model.h, batch, max_len, _p(self.buf), n, _stream(), ctypes.byref(h)), "kv_init")
        self.h = h

    def cache_view(self) -> torch.Tensor:
        """[L, B, 2, H, S, Dh] view of the cache in the model dtype (for tests and synthetic fills)."""
        a = self.model.arch
        header = (4 * (64 + 2 * self.batch) + 1023) // 1024 * 1024
        dt = torch.bfloat16 if a.dtype else torch.float32
        return self.buf[header:].view(dt).view(a.n_layers, self.batch, 2, a.n_heads, self.max_len, a.head_dim)

    def lengths(self) -> np.ndarray:
        out = np.zeros(self.batch, np.int32)
        _check(load().kv_lengths(self.h, out.ctypes.data_as(ctypes.c_void_p), _stream()), "kv_lengths")
        return out

    def status(self) -> int:
        out = np.zeros(1, np.int32)
        _check(load().ssd_device_status(self.h, out.ctypes.data_as(ctypes.c_void_p), _stream()), "ssd_device_status")
        return int(out[0])

    def __del__(self):
        try:
            if getattr(self, "h", None):
                load().kv_destroy(self.h)
                self.h = None
        except Exception:
            pass


def kv_prefill(model: Model, kv: KV, tokens: torch.Tensor, n_tokens: torch.Tensor, ws: torch.Tensor) -> None:
    assert tokens.dtype == torch.int32 and tokens.dim() == 2 and tokens.is_contiguous()
    _check(load().kv_prefill(model.h, kv.h, _p(tokens), _p(n_tokens), tokens.shape[1], _p(ws), ws.numel(), _stream()),
           "kv_prefill")


def draft_step(draft: Model, dkv: KV, tokens_in: torch.Tensor, tokens_stride: int, rows_in: int,
               n_in: Optional[torch.Tensor], temperature: float, u: torch.Tensor, u_stride: int,
               token_out: torch.Tensor, token_out_stride: int, q_out: torch.Tensor, q_stride: int,
               ws: torch.Tensor) -> None:
    _check(load().draft_step(draft.h, dkv.h, _p(tokens_in), tokens_stride, rows_in, _p(n_in), temperature, _p(u),
                             u_stride, _p(token_out), token_out_stride, _p(q_out), q_stride, _p(ws), ws.numel(),
                             _stream()), "draft_step")


def draft_steps(draft: Model, dkv: KV, n_steps: int, tokens_in: torch.Tensor, tokens_stride: int, rows_in: int,
                n_in: Optional[torch.Tensor], temperature: float, u: torch.Tensor, u_stride: int,
                tokens_out: torch.Tensor, token_out_stride: int, q_out: torch.Tensor, q_stride: int,
                ws: torch.Tensor) -> None:
    """n_steps draft steps in one call (one launch for bf16 models): step s draws with u[b * u_stride + s] and
    writes tokens_out[b * token_out_stride + s] and the q row at q_out + b * q_stride + s * vocab."""
    _check(load().draft_steps(draft.h, dkv.h, n_steps, _p(tokens_in), tokens_stride, rows_in, _p(n_in), temperature,
                              _p(u), u_stride, _p(tokens_out), token_out_stride, _p(q_out), q_stride, _p(ws),
                              ws.numel(), _stream()), "draft_steps")


def target_verify(target: Model, tkv: KV, rows: torch.Tensor, K: int, q: Optional[torch.Tensor], u: torch.Tensor,
                  temperature: float, n_accepted: torch.Tensor, next_token: torch.Tensor, next_token_stride: int,
                  p_debug: Optional[torch.Tensor], ws: torch.Tensor) -> None:
    _check(load().target_verify(target.h, tkv.h, _p(rows), K, _p(q), _p(u), temperature, _p(n_accepted),
                                _p(next_token), next_token_stride, _p(p_debug), _p(ws), ws.numel(), _stream()),
           "target_verify")


def kv_commit(kv: KV, n_keep: Optional[torch.Tensor] = None) -> None:
    _check(load().kv_commit(kv.h, _p(n_keep), _stream()), "kv_commit")


def kv_rollback(kv: KV, new_len: torch.Tensor) -> None:
    _check(load().kv_rollback(kv.h, _p(new_len), _stream()), "kv_rollback")


def spec_advance(tkv: KV, dkv: Optional[KV], rows: torch.Tensor, K: int, n_accepted: torch.Tensor,
                 next_token: torch.Tensor, next_token_stride: int, out_tokens: Optional[torch.Tensor], out_cap: int,
                 out_count: Optional[torch.Tensor], draft_in: Optional[torch.Tensor],
                 draft_n_in: Optional[torch.Tensor]) -> None:
    _check(load().spec_advance(tkv.h, None if dkv is None else dkv.h, _p(rows), K, _p(n_accepted), _p(next_token),
                               next_token_stride, _p(out_tokens), out_cap, _p(out_count), _p(draft_in),
                               _p(draft_n_in), _stream()), "spec_advance")


def verify_scratch_bytes(batch: int, K: int) -> int:
    return int(load().verify_scratch_bytes(batch, K))


def verify_from_logits(logits: torch.Tensor, K: int, rows: torch.Tensor, q: Optional[torch.Tensor], u: torch.Tensor,
                       temperature: float, n_accepted: torch.Tensor, next_token: torch.Tensor,
                       next_token_stride: int, p_debug: Optional[torch.Tensor], scratch: torch.Tensor) -> None:
    B, M, V = logits.shape
    assert M == K + 1 and logits.is_contiguous() and logits.dtype == torch.float32
    _check(load().verify_from_logits(_p(logits), B, K, V, _p(rows), _p(q), _p(u), temperature, _p(n_accepted),
                                     _p(next_token), next_token_stride, _p(p_debug), _p(scratch), scratch.numel(),
                                     _stream()), "verify_from_logits")


NOALLOC_MAX_ROWS = 4096


def verify_from_logits_noalloc(logits: torch.Tensor, K: int, rows: torch.Tensor, q: Optional[torch.Tensor],
                               u: torch.Tensor, temperature: float, n_accepted: torch.Tensor,
                               next_token: torch.Tensor, next_token_stride: int,
                               p_debug: Optional[torch.Tensor]) -> None:
    """The tail of a verification on supplied logits, for callers that may not allocate on the device:
    same arguments as verify_from_logits minus the scratch buffer (the library keeps a fixed 64 KB
    array for it, shared by all calls on a device; at most NOALLOC_MAX_ROWS logits rows per call;
    calls that overlap on the GPU must be ordered by the caller)."""
    Bn, M, V = logits.shape
    assert M == K + 1 and logits.is_contiguous() and logits.dtype == torch.float32
    _check(load().verify_from_logits_noalloc(_p(logits), Bn, K, V, _p(rows), _p(q), _p(u), temperature,
                                             _p(n_accepted), _p(next_token), next_token_stride, _p(p_debug),
                                             _stream()), "verify_from_logits_noalloc")


def attention_rows(model: Model, kv: KV, layer: int, q: torch.Tensor, rows: int, out: torch.Tensor,
                   ws: torch.Tensor) -> None:
    _check(load().attention_rows(model.h, kv.h, layer, _p(q), rows, _p(out), _p(ws), ws.numel(), _stream()),
           "attention_rows")


def last_logits(model: Model, batch: int, rows_per_seq: int, ws: torch.Tensor) -> torch.Tensor:
    out = torch.empty(batch, rows_per_seq, model.arch.vocab, dtype=torch.float32, device="cuda")
    _check(load().ssd_last_logits(model.h, batch, rows_per_seq, _p(ws), ws.numel(), _p(out), _stream()),
           "ssd_last_logits")
    return out


def set_persistent(enable: bool) -> None:
    _check(load().ssd_set_persistent(1 if enable else 0), "ssd_set_persistent")


def set_attention_mode(mode: int) -> None:
    """0: per pass (default); 1: warp-MMA items over 16-row tiles; 2: tensor-core items wherever they apply;
    3: the hi-and-lo-in-one-tile MMA items for passes of at most eight rows, the first form otherwise."""
    _check(load().ssd_set_attention_mode(int(mode)), "ssd_set_attention_mode")


def set_prefill_mode(mode: int) -> None:
    """0: many-row prompt pass from 256 rows per pass (default); 1: never; 2: wherever it applies."""
    _check(load().ssd_set_prefill_mode(int(mode)), "ssd_set_prefill_mode")


def set_trace(enable: bool) -> None:
    _check(load().ssd_set_trace(1 if enable else 0), "ssd_set_trace")


def read_trace(model: Model, batch: int, rows_per_seq: int, ws: torch.Tensor) -> np.ndarray:
    """Nanosecond stamps of the last single-kernel forward on this workspace (start, after every
    grid barrier, end)."""
    out = np.zeros(1024, np.uint64)
    n = ctypes.c_int()
    _check(load().ssd_read_trace(model.h, batch, rows_per_seq, _p(ws), ws.numel(), out.ctypes.data_as(ctypes.c_void_p),
                                 1024, ctypes.byref(n), _stream()), "ssd_read_trace")
    return out[:n.value]


def set_sampling(top_k: int = 0, top_p: float = 1.0) -> None:
    """Restrict both models' distributions to the top_k most probable tokens and / or the top_p nucleus
    (0 and 1.0 switch the restriction off)."""
    _check(load().ssd_set_sampling(int(top_k), float(top_p)), "ssd_set_sampling")


def set_wait_limit(cycles: int) -> None:
    """Bound (GPU clock cycles) of every device-side wait that takes work; 0 restores the default (~2 s)."""
    _check(load().ssd_set_wait_limit(int(cycles)), "ssd_set_wait_limit")


def wait_probe(kv: KV) -> None:
    """Queue the failure-detection probe: a wait on a barrier nobody arrives at; it runs out after the
    configured bound and leaves SSD_E_TIMEOUT in the cache's status word."""
    _check(load().ssd_wait_probe(kv.h, _stream()), "ssd_wait_probe")


def launch_count() -> int:
    return int(load().ssd_launch_count())


def gemm_profile(enable: bool) -> None:
    _check(load().ssd_gemm_profile(1 if enable else 0), "ssd_gemm_profile")


def gemm_profile_read(reset: bool = True):
    n, ms = ctypes.c_uint64(), ctypes.c_double()
    _check(load().ssd_gemm_profile_read(ctypes.byref(n), ctypes.byref(ms), 1 if reset else 0), "ssd_gemm_profile_read")
    return int(n.value), float(ms.value)
