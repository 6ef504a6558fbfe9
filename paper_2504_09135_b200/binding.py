"""Thin Python binding of the C ABI in include/disc.h.

Argument marshalling only: every function here checks tensor types, hands raw pointers to the
CUDA library and returns the output tensors.  torch is used for device memory and streams.  There
is no CPU fallback: without the compiled library (or without a CUDA device for the calls that need
one) these functions raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

from . import build as _build

DISC_F32, DISC_BF16 = 0, 1
ROW_DEAD, ROW_NOMASS, ROW_NONFINITE, ROW_DONE, ROW_FAULT = 1, 2, 4, 8, 16
MAX_DEPTH = 64

ERRORS = {-1: "DISC_ERR_ARG", -2: "DISC_ERR_EMPTY", -3: "DISC_ERR_TOKEN", -4: "DISC_ERR_PREFIX",
          -5: "DISC_ERR_OOM", -6: "DISC_ERR_CUDA", -7: "DISC_ERR_UNSUPPORTED"}

EXPORTS = ["disc_build_set", "disc_build_set_eok", "disc_free_set", "disc_set_info", "disc_set_rows", "disc_state_init",
           "disc_mask", "disc_mask_static", "disc_verify", "disc_step", "disc_project_step", "disc_project_scratch_bytes",
           "disc_project_error", "disc_topm", "disc_step_topm", "disc_step_topm_scratch_bytes", "disc_resample", "disc_accept", "disc_accept_resample",
           "disc_sampling_uniforms",
           "disc_error_string", "disc_last_cuda_error"]


class DiscError(RuntimeError):
    def __init__(self, code: int, where: str):
        name = ERRORS.get(code, str(code))
        extra = ""
        if code == -6:
            extra = f" (cudaError {lib().disc_last_cuda_error()})"
        super().__init__(f"{where} failed: {name}{extra}")
        self.code = code


class _SetInfo(C.Structure):
    _fields_ = [("n_members", C.c_int64), ("n_entries", C.c_int64), ("n_nodes", C.c_int64),
                ("vocab_size", C.c_int32), ("mask_words", C.c_int32), ("l_max", C.c_int32),
                ("n_heavy", C.c_int32), ("device_bytes", C.c_int64), ("build_seconds", C.c_double),
                ("level_nodes", C.c_int64 * MAX_DEPTH)]


_lib = None


def lib():
    """Load (building first if needed) the CUDA library.  Raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB if _build.is_fresh() else _build.build()
    L = C.CDLL(path)
    vp, i32, i64, u32, u64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_float
    L.disc_build_set.argtypes = [vp, vp, i64, i32, u32, vp, C.POINTER(vp)]
    L.disc_build_set_eok.argtypes = [vp, vp, i64, i32, i32, vp, C.POINTER(vp)]
    L.disc_free_set.argtypes = [vp]
    L.disc_free_set.restype = None
    L.disc_set_info.argtypes = [vp, C.POINTER(_SetInfo)]
    L.disc_set_rows.argtypes = [vp, vp, vp]
    L.disc_state_init.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp, vp]
    L.disc_mask.argtypes = [vp, vp, i32, vp, i64, vp, vp, vp, vp, vp, vp]
    L.disc_mask_static.argtypes = [vp, vp, i32, vp, i64, vp, vp, vp, vp, vp, vp]
    L.disc_verify.argtypes = [vp, vp, i32, vp, i64, vp, i32, vp, vp, vp, vp, vp, vp]
    L.disc_step.argtypes = [vp, vp, C.c_int, i64, i64, f32, u64, u32, i64, vp, vp, vp, vp, vp, vp,
                            vp, vp, i32, vp, vp, vp, vp, vp]
    L.disc_project_step.argtypes = [vp, vp, i64, vp, i64, i32, i64, f32, u64, u32, i64, vp, vp, vp, vp, vp, vp,
                                    vp, vp, i32, vp, vp, vp, vp, i64, i32, vp, i64, vp]
    L.disc_topm.argtypes = [vp, C.c_int, i64, i64, i32, i32, f32, vp, vp, vp, vp]
    L.disc_step_topm_scratch_bytes.argtypes = [i64, i32]
    L.disc_step_topm.argtypes = [vp, vp, C.c_int, i64, i64, i32, f32, u64, u32, i64, vp, vp, vp, vp, vp, vp,
                                 vp, vp, i32, vp, vp, vp, vp, vp, vp, i64, vp]
    L.disc_project_scratch_bytes.argtypes = [vp, i64]
    L.disc_project_error.argtypes = [vp, vp]
    L.disc_resample.argtypes = [vp, i32, i32, u64, i64, vp, vp, vp, i32, vp, vp, vp]
    L.disc_accept.argtypes = [vp, i32, i32, u64, i64, vp, vp]
    L.disc_accept_resample.argtypes = [vp, i32, i32, u64, i64, vp, vp, vp, vp, i32, vp, vp, vp]
    L.disc_sampling_uniforms.argtypes = [u64, u32, u32, i32, i32, vp, vp]
    L.disc_error_string.argtypes = [C.c_int]
    L.disc_error_string.restype = C.c_char_p
    L.disc_last_cuda_error.argtypes = []
    for name in EXPORTS:
        if name in ("disc_project_scratch_bytes", "disc_step_topm_scratch_bytes"):
            getattr(L, name).restype = C.c_int64
        elif name not in ("disc_free_set", "disc_error_string"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(rc: int, where: str):
    if rc != 0:
        raise DiscError(rc, where)


def _stream_ptr(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if t is None:
        return 0
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


class DiscSet:
    """Handle of a built constraint set (owns device memory; free with .close())."""

    def __init__(self, handle, info: _SetInfo):
        self._h = handle
        self.N = int(info.n_members)
        self.E = int(info.n_entries)
        self.n_nodes = int(info.n_nodes)
        self.V = int(info.vocab_size)
        self.W = int(info.mask_words)
        self.l_max = int(info.l_max)
        self.n_heavy = int(info.n_heavy)
        self.device_bytes = int(info.device_bytes)
        self.build_seconds = float(info.build_seconds)
        self.level_nodes = [int(info.level_nodes[d]) for d in range(self.l_max)]

    @property
    def handle(self):
        if not self._h:
            raise RuntimeError("constraint set already freed")
        return self._h

    def close(self):
        if getattr(self, "_h", None):
            lib().disc_free_set(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def disc_build_set(tokens, row_offsets, vocab_size: int, stream=None) -> DiscSet:
    """tokens int32[E], row_offsets int64[n+1] on the host (numpy or CPU tensors)."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    row_offsets = np.ascontiguousarray(row_offsets, dtype=np.int64)
    if row_offsets.ndim != 1 or row_offsets.shape[0] < 1:
        raise DiscError(-1, "disc_build_set")
    if not torch.cuda.is_available():
        raise RuntimeError("disc_build_set needs a CUDA device; there is no CPU path")
    h = C.c_void_p()
    rc = lib().disc_build_set(tokens.ctypes.data, row_offsets.ctypes.data, row_offsets.shape[0] - 1,
                              int(vocab_size), 0, _stream_ptr(stream), C.byref(h))
    _check(rc, "disc_build_set")
    info = _SetInfo()
    _check(lib().disc_set_info(h, C.byref(info)), "disc_set_info")
    return DiscSet(h, info)


def disc_build_set_eok(tokens, row_offsets, vocab_size: int, eok_token: int, stream=None) -> DiscSet:
    """Like disc_build_set for sets in which a member may be a prefix of another: every member is
    closed by `eok_token` (Section 2.1's end-of-keyword token) before the build."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    row_offsets = np.ascontiguousarray(row_offsets, dtype=np.int64)
    if row_offsets.ndim != 1 or row_offsets.shape[0] < 1:
        raise DiscError(-1, "disc_build_set_eok")
    if not torch.cuda.is_available():
        raise RuntimeError("disc_build_set_eok needs a CUDA device; there is no CPU path")
    h = C.c_void_p()
    rc = lib().disc_build_set_eok(tokens.ctypes.data, row_offsets.ctypes.data, row_offsets.shape[0] - 1,
                                  int(vocab_size), int(eok_token), _stream_ptr(stream), C.byref(h))
    _check(rc, "disc_build_set_eok")
    info = _SetInfo()
    _check(lib().disc_set_info(h, C.byref(info)), "disc_set_info")
    return DiscSet(h, info)


def disc_set_rows(s: DiscSet):
    tok = np.empty(s.E, dtype=np.int32)
    off = np.empty(s.N + 1, dtype=np.int64)
    _check(lib().disc_set_rows(s.handle, tok.ctypes.data, off.ctypes.data), "disc_set_rows")
    return tok, off


@dataclass
class DiscState:
    """Per-candidate cursor and importance log-weight, all device tensors of n entries."""
    node: torch.Tensor
    lo: torch.Tensor
    hi: torch.Tensor
    depth: torch.Tensor
    logw: torch.Tensor
    done: torch.Tensor

    @property
    def n(self) -> int:
        return self.node.shape[0]

    @staticmethod
    def empty(n: int, device) -> "DiscState":
        i32 = dict(dtype=torch.int32, device=device)
        return DiscState(torch.empty(n, **i32), torch.empty(n, **i32), torch.empty(n, **i32),
                         torch.empty(n, **i32), torch.empty(n, dtype=torch.float32, device=device),
                         torch.empty(n, dtype=torch.uint8, device=device))

    def clone(self) -> "DiscState":
        return DiscState(*(t.clone() for t in (self.node, self.lo, self.hi, self.depth, self.logw, self.done)))


def disc_state_init(s: DiscSet, n: int, device="cuda", state: DiscState | None = None, stream=None) -> DiscState:
    st = DiscState.empty(n, device) if state is None else state
    rc = lib().disc_state_init(s.handle, n, _dev(st.node, torch.int32, "node"), _dev(st.lo, torch.int32, "lo"),
                               _dev(st.hi, torch.int32, "hi"), _dev(st.depth, torch.int32, "depth"),
                               _dev(st.logw, torch.float32, "logw"), _dev(st.done, torch.uint8, "done"),
                               _stream_ptr(stream))
    _check(rc, "disc_state_init")
    return st


def disc_mask(s: DiscSet, prefix: torch.Tensor, prefix_len: torch.Tensor, *, want_mask=True, out=None, stream=None):
    """prefix int32[n, ld], prefix_len int32[n] on the device -> dict(mask, lo, hi, node, status)."""
    n = prefix_len.shape[0]
    dev = prefix_len.device
    ld = prefix.shape[1] if prefix.ndim == 2 else 0
    if out is None:
        out = {"mask": torch.empty((n, s.W), dtype=torch.int32, device=dev) if want_mask else None,
               "lo": torch.empty(n, dtype=torch.int32, device=dev),
               "hi": torch.empty(n, dtype=torch.int32, device=dev),
               "node": torch.empty(n, dtype=torch.int32, device=dev),
               "status": torch.empty(n, dtype=torch.uint8, device=dev)}
    rc = lib().disc_mask(s.handle, _dev(prefix, torch.int32, "prefix") if ld > 0 else 0, ld,
                         _dev(prefix_len, torch.int32, "prefix_len"), n,
                         _dev(out["mask"], torch.int32, "mask"), _dev(out["lo"], torch.int32, "lo"),
                         _dev(out["hi"], torch.int32, "hi"), _dev(out["node"], torch.int32, "node"),
                         _dev(out["status"], torch.uint8, "status"), _stream_ptr(stream))
    _check(rc, "disc_mask")
    return out


def disc_verify(s: DiscSet, prefix: torch.Tensor, prefix_len: torch.Tensor, cand: torch.Tensor, *, want_rows=True,
                want_mask=False, out=None, stream=None):
    """Algorithm 2, lines 4-6: prefix int32[n, ld], prefix_len int32[n], cand int32[n, M] on the
    device -> dict(valid uint8[n, M], rows int32[n, M] or None, mask or None, lo, hi)."""
    n = prefix_len.shape[0]
    dev = prefix_len.device
    ld = prefix.shape[1] if prefix.ndim == 2 else 0
    M = cand.shape[1] if cand.ndim == 2 else 0
    if out is None:
        out = {"valid": torch.empty((n, M), dtype=torch.uint8, device=dev),
               "rows": torch.empty((n, M), dtype=torch.int32, device=dev) if want_rows else None,
               "mask": torch.empty((n, s.W), dtype=torch.int32, device=dev) if want_mask else None,
               "lo": torch.empty(n, dtype=torch.int32, device=dev),
               "hi": torch.empty(n, dtype=torch.int32, device=dev)}
    rc = lib().disc_verify(s.handle, _dev(prefix, torch.int32, "prefix") if ld > 0 else 0, ld,
                           _dev(prefix_len, torch.int32, "prefix_len"), n,
                           _dev(cand, torch.int32, "cand") if M > 0 else 0, M,
                           _dev(out["valid"], torch.uint8, "valid") if M > 0 else 0,
                           _dev(out["rows"], torch.int32, "rows"), _dev(out["mask"], torch.int32, "mask"),
                           _dev(out["lo"], torch.int32, "lo"), _dev(out["hi"], torch.int32, "hi"), _stream_ptr(stream))
    _check(rc, "disc_verify")
    return out


MASK_STATIC_MAX_ROWS = 1 << 30


def disc_mask_static(s: DiscSet, prefix: torch.Tensor, prefix_len: torch.Tensor, *, want_mask=True, out=None,
                     stream=None):
    """disc_mask through the entry point that keeps its row counter in a fixed word block of the
    library instead of allocated device memory (same arguments and results)."""
    n = prefix_len.shape[0]
    if n > MASK_STATIC_MAX_ROWS:
        raise ValueError(f"disc_mask_static: {n} prefixes exceed the limit of {MASK_STATIC_MAX_ROWS} per call")
    dev = prefix_len.device
    ld = prefix.shape[1] if prefix.ndim == 2 else 0
    if out is None:
        out = {"mask": torch.empty((n, s.W), dtype=torch.int32, device=dev) if want_mask else None,
               "lo": torch.empty(n, dtype=torch.int32, device=dev),
               "hi": torch.empty(n, dtype=torch.int32, device=dev),
               "node": torch.empty(n, dtype=torch.int32, device=dev),
               "status": torch.empty(n, dtype=torch.uint8, device=dev)}
    rc = lib().disc_mask_static(s.handle, _dev(prefix, torch.int32, "prefix") if ld > 0 else 0, ld,
                                _dev(prefix_len, torch.int32, "prefix_len"), n,
                                _dev(out["mask"], torch.int32, "mask"), _dev(out["lo"], torch.int32, "lo"),
                                _dev(out["hi"], torch.int32, "hi"), _dev(out["node"], torch.int32, "node"),
                                _dev(out["status"], torch.uint8, "status"), _stream_ptr(stream))
    _check(rc, "disc_mask_static")
    return out


@dataclass
class StepOutputs:
    token: torch.Tensor
    status: torch.Tensor
    logq: torch.Tensor | None = None
    logp: torch.Tensor | None = None
    mask: torch.Tensor | None = None

    @staticmethod
    def empty(n: int, device, *, logq=True, logp=True, mask_words: int = 0) -> "StepOutputs":
        f = dict(dtype=torch.float32, device=device)
        return StepOutputs(torch.empty(n, dtype=torch.int32, device=device),
                           torch.empty(n, dtype=torch.uint8, device=device),
                           torch.empty(n, **f) if logq else None, torch.empty(n, **f) if logp else None,
                           torch.empty((n, mask_words), dtype=torch.int32, device=device) if mask_words else None)


def disc_step(s: DiscSet, logits: torch.Tensor, state: DiscState, *, inv_temperature=1.0, seed=0, step=0,
              row_base=0, seq_tokens: torch.Tensor | None = None, out: StepOutputs | None = None,
              stream=None) -> StepOutputs:
    """logits [n, ld] float32 or bfloat16 (row stride ld >= V, unit element stride): a device tensor,
    or a pinned host tensor, which the kernel then reads in place over PCIe (only the rows that are
    still live are read)."""
    n = state.n
    if logits.dtype == torch.float32:
        dt = DISC_F32
    elif logits.dtype == torch.bfloat16:
        dt = DISC_BF16
    else:
        raise DiscError(-7, "disc_step")
    if not ((logits.is_cuda or logits.is_pinned()) and logits.ndim == 2 and logits.shape[0] == n
            and logits.stride(1) == 1):
        raise TypeError("logits: expected a CUDA (or pinned host) tensor [n, >=V] with unit inner stride")
    ld = logits.stride(0) if n > 1 else max(logits.shape[1], logits.stride(0))
    if out is None:
        out = StepOutputs.empty(n, state.node.device)
    seq_ld = 0
    if seq_tokens is not None:
        seq_ld = seq_tokens.shape[-1]
    rc = lib().disc_step(s.handle, logits.data_ptr(), dt, ld, n, float(inv_temperature), int(seed), int(step),
                         int(row_base), _dev(state.node, torch.int32, "node"), _dev(state.lo, torch.int32, "lo"),
                         _dev(state.hi, torch.int32, "hi"), _dev(state.depth, torch.int32, "depth"),
                         _dev(state.logw, torch.float32, "logw"), _dev(state.done, torch.uint8, "done"),
                         _dev(out.token, torch.int32, "token"), _dev(seq_tokens, torch.int32, "seq_tokens"),
                         seq_ld, _dev(out.logq, torch.float32, "logq"), _dev(out.logp, torch.float32, "logp"),
                         _dev(out.mask, torch.int32, "mask"), _dev(out.status, torch.uint8, "status"),
                         _stream_ptr(stream))
    _check(rc, "disc_step")
    return out


def _logits_args(logits: torch.Tensor, n: int, where: str):
    if logits.dtype == torch.float32:
        dt = DISC_F32
    elif logits.dtype == torch.bfloat16:
        dt = DISC_BF16
    else:
        raise DiscError(-7, where)
    if not (logits.is_cuda and logits.ndim == 2 and logits.shape[0] == n and logits.stride(1) == 1):
        raise TypeError("logits: expected a CUDA tensor [n, >=V] with unit inner stride")
    return dt, (logits.stride(0) if n > 1 else max(logits.shape[1], logits.stride(0)))


def disc_topm(logits: torch.Tensor, V: int, M: int, *, inv_temperature=1.0, done: torch.Tensor | None = None,
              want_lse=False, stream=None):
    """The M largest logits of every row as token ids in ascending order: int32[n, M]; with want_lse
    also float32[n, 2], the pair (m, s) with sum_v 2^(z_v log2e / T) = 2^m * s."""
    n = logits.shape[0]
    dt, ld = _logits_args(logits, n, "disc_topm")
    cand = torch.empty((n, M), dtype=torch.int32, device=logits.device)
    lse = torch.empty((n, 2), dtype=torch.float32, device=logits.device) if want_lse else None
    rc = lib().disc_topm(logits.data_ptr(), dt, ld, n, int(V), int(M), float(inv_temperature),
                         _dev(done, torch.uint8, "done"), cand.data_ptr(), _dev(lse, torch.float32, "lse"),
                         _stream_ptr(stream))
    _check(rc, "disc_topm")
    return (cand, lse) if want_lse else cand


def disc_step_topm(s: DiscSet, logits: torch.Tensor, state: DiscState, M: int, seq_tokens: torch.Tensor, *,
                   inv_temperature=1.0, seed=0, step=0, row_base=0, out: StepOutputs | None = None,
                   cand: torch.Tensor | None = None, scratch: torch.Tensor | None = None, stream=None):
    """One step in the paper's top-M mode.  Returns (StepOutputs, cand int32[n, M])."""
    n = state.n
    dt, ld = _logits_args(logits, n, "disc_step_topm")
    dev = state.node.device
    if out is None:
        out = StepOutputs.empty(n, dev)
    if cand is None:
        cand = torch.empty((n, M), dtype=torch.int32, device=dev)
    need = lib().disc_step_topm_scratch_bytes(n, int(M))
    if need < 0:
        raise DiscError(int(need), "disc_step_topm_scratch_bytes")
    if scratch is None:
        scratch = torch.empty(int(need), dtype=torch.uint8, device=dev)
    rc = lib().disc_step_topm(s.handle, logits.data_ptr(), dt, ld, n, int(M), float(inv_temperature), int(seed),
                              int(step), int(row_base), _dev(state.node, torch.int32, "node"),
                              _dev(state.lo, torch.int32, "lo"), _dev(state.hi, torch.int32, "hi"),
                              _dev(state.depth, torch.int32, "depth"), _dev(state.logw, torch.float32, "logw"),
                              _dev(state.done, torch.uint8, "done"), _dev(out.token, torch.int32, "token"),
                              _dev(seq_tokens, torch.int32, "seq_tokens"), seq_tokens.shape[-1],
                              _dev(out.logq, torch.float32, "logq"), _dev(out.logp, torch.float32, "logp"),
                              _dev(out.mask, torch.int32, "mask"), _dev(out.status, torch.uint8, "status"),
                              _dev(cand, torch.int32, "cand"), _dev(scratch, torch.uint8, "scratch"), scratch.numel(),
                              _stream_ptr(stream))
    _check(rc, "disc_step_topm")
    return out, cand


def disc_project_scratch(s: DiscSet, n: int, device) -> torch.Tensor:
    """Scratch buffer disc_project_step needs for n rows (caller-owned device memory)."""
    nbytes = lib().disc_project_scratch_bytes(s.handle, int(n))
    if nbytes < 0:
        raise DiscError(int(nbytes), "disc_project_scratch_bytes")
    return torch.empty(int(nbytes), dtype=torch.uint8, device=device)


def disc_project_step(s: DiscSet, hidden: torch.Tensor, wt: torch.Tensor, state: DiscState, logits_buf: torch.Tensor,
                      scratch: torch.Tensor, *, inv_temperature=1.0, seed=0, step=0, row_base=0,
                      seq_tokens: torch.Tensor | None = None, out: StepOutputs | None = None, store_all=False,
                      stream=None) -> StepOutputs:
    """One step with the last projection fused in: hidden bf16[n, d], wt bf16[V, d] (one vocabulary entry
    per row), logits_buf bf16[n, >=V] (receives the pieces of the logits the step reads; everything
    with store_all), scratch from disc_project_scratch."""
    n = state.n
    for name, t in (("hidden", hidden), ("wt", wt), ("logits_buf", logits_buf)):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.ndim == 2 and t.stride(1) == 1):
            raise TypeError(f"{name}: expected a CUDA bfloat16 matrix with unit inner stride")
    if hidden.shape[0] != n or wt.shape[1] != hidden.shape[1] or logits_buf.shape[0] != n:
        raise TypeError("disc_project_step: shapes do not fit")
    if out is None:
        out = StepOutputs.empty(n, state.node.device)
    seq_ld = 0 if seq_tokens is None else seq_tokens.shape[-1]
    rc = lib().disc_project_step(s.handle, hidden.data_ptr(), hidden.stride(0), wt.data_ptr(), wt.stride(0),
                                 hidden.shape[1], n, float(inv_temperature), int(seed), int(step), int(row_base),
                                 _dev(state.node, torch.int32, "node"), _dev(state.lo, torch.int32, "lo"),
                                 _dev(state.hi, torch.int32, "hi"), _dev(state.depth, torch.int32, "depth"),
                                 _dev(state.logw, torch.float32, "logw"), _dev(state.done, torch.uint8, "done"),
                                 _dev(out.token, torch.int32, "token"), _dev(seq_tokens, torch.int32, "seq_tokens"),
                                 seq_ld, _dev(out.logq, torch.float32, "logq"), _dev(out.logp, torch.float32, "logp"),
                                 _dev(out.status, torch.uint8, "status"), logits_buf.data_ptr(),
                                 logits_buf.stride(0) if n > 1 else max(logits_buf.shape[1], logits_buf.stride(0)),
                                 1 if store_all else 0, _dev(scratch, torch.uint8, "scratch"), scratch.numel(),
                                 _stream_ptr(stream))
    _check(rc, "disc_project_step")
    return out


def disc_project_check(scratch: torch.Tensor, stream=None) -> None:
    """Synchronises the stream and raises if the projection kernel gave up on one of its waits."""
    _check(lib().disc_project_error(_dev(scratch, torch.uint8, "scratch"), _stream_ptr(stream)), "disc_project_error")


def disc_resample(logw: torch.Tensor, *, seed=0, query_base=0, seq_tokens: torch.Tensor | None = None,
                  out=None, stream=None):
    """logw float32[B, K] on the device -> dict(idx, logz, status, tokens)."""
    B, K = logw.shape
    dev = logw.device
    seq_ld = 0 if seq_tokens is None else seq_tokens.shape[-1]
    if out is None:
        out = {"idx": torch.empty(B, dtype=torch.int32, device=dev),
               "logz": torch.empty(B, dtype=torch.float32, device=dev),
               "status": torch.empty(B, dtype=torch.uint8, device=dev),
               "tokens": None if seq_tokens is None else torch.empty((B, seq_ld), dtype=torch.int32, device=dev)}
    rc = lib().disc_resample(_dev(logw, torch.float32, "logw"), B, K, int(seed), int(query_base),
                             _dev(out["idx"], torch.int32, "idx"), _dev(out["logz"], torch.float32, "logz"),
                             _dev(seq_tokens, torch.int32, "seq_tokens"), seq_ld,
                             _dev(out["tokens"], torch.int32, "tokens"), _dev(out["status"], torch.uint8, "status"),
                             _stream_ptr(stream))
    _check(rc, "disc_resample")
    return out


def disc_accept(logw: torch.Tensor, *, seed=0, query_base=0, out=None, stream=None) -> torch.Tensor:
    B, K = logw.shape
    if out is None:
        out = torch.empty(B, dtype=torch.int32, device=logw.device)
    rc = lib().disc_accept(_dev(logw, torch.float32, "logw"), B, K, int(seed), int(query_base),
                           _dev(out, torch.int32, "first"), _stream_ptr(stream))
    _check(rc, "disc_accept")
    return out


def disc_accept_resample(logw: torch.Tensor, *, seed=0, query_base=0, seq_tokens: torch.Tensor | None = None,
                         out=None, stream=None):
    """logw float32[B, 2K] on the device (first K columns: accept test in order; last K: fresh
    candidates of the K-way draw) -> dict(choice, first, logz, status, tokens)."""
    B, K2 = logw.shape
    if K2 % 2 or K2 == 0:
        raise DiscError(-1, "disc_accept_resample")
    dev = logw.device
    seq_ld = 0 if seq_tokens is None else seq_tokens.shape[-1]
    if out is None:
        out = {"choice": torch.empty(B, dtype=torch.int32, device=dev),
               "first": torch.empty(B, dtype=torch.int32, device=dev),
               "logz": torch.empty(B, dtype=torch.float32, device=dev),
               "status": torch.empty(B, dtype=torch.uint8, device=dev),
               "tokens": None if seq_tokens is None else torch.empty((B, seq_ld), dtype=torch.int32, device=dev)}
    rc = lib().disc_accept_resample(_dev(logw, torch.float32, "logw"), B, K2 // 2, int(seed), int(query_base),
                                    _dev(out["choice"], torch.int32, "choice"), _dev(out["first"], torch.int32, "first"),
                                    _dev(out["logz"], torch.float32, "logz"),
                                    _dev(seq_tokens, torch.int32, "seq_tokens"), seq_ld,
                                    _dev(out["tokens"], torch.int32, "tokens"),
                                    _dev(out["status"], torch.uint8, "status"), _stream_ptr(stream))
    _check(rc, "disc_accept_resample")
    return out


def disc_sampling_uniforms(seed: int, step: int, row: int, v0: int, n: int, device="cuda", stream=None):
    out = torch.empty(n, dtype=torch.float32, device=device)
    rc = lib().disc_sampling_uniforms(int(seed), int(step), int(row), int(v0), int(n), out.data_ptr(),
                                      _stream_ptr(stream))
    _check(rc, "disc_sampling_uniforms")
    return out
