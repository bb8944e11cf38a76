"""Thin ctypes binding of the C ABI in include/dgc.h: argument marshalling only.

Every step of the path runs in the CUDA library; there is no CPU fallback.
Importing this module without the built library raises ImportError.
PyTorch supplies device memory and streams: tensors are passed as raw device
pointers, `stream` arguments default to torch's current stream.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdgc.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_1712_01887_b200.build` "
        "(there is no CPU fallback)")

_lib = ctypes.CDLL(LIB_PATH)

OK, EINVAL, ENOMEM, ECAPACITY, ECUDA, ESTATE = 0, -1, -2, -3, -4, -5
FLAG_NONFINITE_NORM, FLAG_FULL_SELECT, FLAG_CAND_OVERFLOW, FLAG_CAND_SHORT = 1, 2, 4, 8
FLAG_TIE_FILL = 16
ARENA_ALIGN = 512
MAX_DECODE_WORKERS = 64


class Config(ctypes.Structure):
    _fields_ = [("num_tensors", ctypes.c_int32), ("num_workers", ctypes.c_int32),
                ("tensor_numel", ctypes.POINTER(ctypes.c_int64)), ("momentum", ctypes.c_float),
                ("clip_threshold", ctypes.c_float), ("sparsity", ctypes.c_double),
                ("sample_ratio", ctypes.c_double), ("seed", ctypes.c_uint64),
                ("device", ctypes.c_int32), ("debug_sample_rank", ctypes.c_int32),
                ("nesterov", ctypes.c_int32), ("select_mode", ctypes.c_int32),
                ("clip_scope", ctypes.c_int32)]


class Status(ctypes.Structure):
    _fields_ = [("grad_norm", ctypes.c_double), ("clip_coef", ctypes.c_float),
                ("flags", ctypes.c_int32), ("iterations", ctypes.c_int64),
                ("full_select_last", ctypes.c_int64), ("candidates_last", ctypes.c_int64)]


_vp = ctypes.c_void_p
_i64p = ctypes.POINTER(ctypes.c_int64)
_sigs = {
    "dgc_state_create": (ctypes.c_int32, [ctypes.POINTER(Config), ctypes.POINTER(_vp)]),
    "dgc_state_destroy": (ctypes.c_int32, [_vp]),
    "dgc_set_sparsity": (ctypes.c_int32, [_vp, ctypes.c_double]),
    "dgc_warmup_sparsity": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(ctypes.c_double)]),
    "dgc_max_nnz": (ctypes.c_int64, [_vp]),
    "dgc_layout": (ctypes.c_int32, [_vp, _i64p, _i64p, _i64p, _i64p]),
    "dgc_compress": (ctypes.c_int32, [_vp, _vp, _vp, _vp, ctypes.c_int64, _vp]),
    "dgc_compress_batch": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(_vp),
                                            ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                            ctypes.POINTER(_vp), _i64p, _vp]),
    "dgc_compress_host": (ctypes.c_int32, [_vp, _vp, _vp, _vp, ctypes.c_int64, _vp]),
    "dgc_compress_host_batch": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(_vp),
                                                 ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                                 ctypes.POINTER(_vp), _i64p, _vp]),
    "dgc_decode_accumulate": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(_vp),
                                               ctypes.POINTER(_vp), _i64p, _vp, ctypes.c_int64,
                                               _vp, ctypes.c_int64, _vp]),
    "dgc_decode_workspace_bytes": (ctypes.c_int64, [ctypes.c_int32, ctypes.c_int64]),
    "dgc_decode_accumulate_static": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(_vp),
                                                      ctypes.POINTER(_vp), _i64p, _vp,
                                                      ctypes.c_int64, _vp]),
    "dgc_decode_rejected": (ctypes.c_int32, [ctypes.c_int32, ctypes.c_int64, _vp, _vp, _i64p]),
    "dgc_apply_sgd": (ctypes.c_int32, [_vp, _vp, ctypes.c_int64, ctypes.c_float, _vp]),
    "dgc_decode_accumulate_sgd": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(_vp),
                                                   ctypes.POINTER(_vp), _i64p, _vp, _vp,
                                                   ctypes.c_int64, ctypes.c_float, _vp,
                                                   ctypes.c_int64, _vp]),
    "dgc_decode_apply_sgd": (ctypes.c_int32, [ctypes.c_int32, ctypes.POINTER(_vp),
                                              ctypes.POINTER(_vp), _i64p, _vp, ctypes.c_int64,
                                              ctypes.c_float, _vp, ctypes.c_int64, _vp]),
    "dgc_encode_runlength": (ctypes.c_int32, [_vp, _vp, ctypes.c_int64, _vp, _vp, ctypes.c_int64,
                                              _vp, _vp, ctypes.c_int64, _vp]),
    "dgc_decode_runlength": (ctypes.c_int32, [_vp, _vp, ctypes.c_int64, _vp, _vp, _vp, _vp,
                                              ctypes.c_int64, _vp]),
    "dgc_runlength_max_entries": (ctypes.c_int64, [ctypes.c_int64, ctypes.c_int64]),
    "dgc_runlength_workspace_bytes": (ctypes.c_int64, [ctypes.c_int64]),
    "dgc_get_nnz": (ctypes.c_int32, [_vp, _vp, _i64p, _i64p]),
    "dgc_get_status": (ctypes.c_int32, [_vp, _vp, ctypes.POINTER(Status)]),
    "dgc_get_thresholds": (ctypes.c_int32, [_vp, _vp, _vp, _vp]),
    "dgc_get_clip": (ctypes.c_int32, [_vp, _vp, _vp, _vp]),
    "dgc_state_read": (ctypes.c_int32, [_vp, _vp, _vp, _vp]),
    "dgc_state_write": (ctypes.c_int32, [_vp, _vp, _vp, _vp]),
    "dgc_state_set_iterations": (ctypes.c_int32, [_vp, ctypes.c_int64, _vp]),
    "dgc_timeline_enable": (ctypes.c_int32, [_vp, ctypes.c_int32]),
    "dgc_timeline_read": (ctypes.c_int32, [_vp, _vp, _vp]),
    "dgc_profile_enable": (ctypes.c_int32, [_vp, ctypes.c_int32]),
    "dgc_profile_read": (ctypes.c_int32, [_vp, _vp, ctypes.c_int32,
                                          ctypes.POINTER(ctypes.c_int32)]),
    "dgc_launch_count": (ctypes.c_uint64, []),
    "dgc_error_string": (ctypes.c_char_p, [ctypes.c_int32]),
}
for _name, (_res, _args) in _sigs.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args

EXPORTED = tuple(_sigs)


class DgcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__(f"{where}: {_lib.dgc_error_string(int(code)).decode()} ({code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise DgcError(code, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream
    return int(stream)


def _dev(t: torch.Tensor, dtype) -> int:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError(f"expected a contiguous CUDA {dtype} tensor")
    return t.data_ptr()


def warmup_sparsity(stage: int) -> float:
    s = ctypes.c_double()
    _check(_lib.dgc_warmup_sparsity(int(stage), ctypes.byref(s)), "dgc_warmup_sparsity")
    return s.value


def launch_count() -> int:
    return int(_lib.dgc_launch_count())


class State:
    """One worker of Algorithm 4: owns u and v on the device."""

    def __init__(self, tensor_numel: Sequence[int], num_workers: int, momentum: float,
                 clip_threshold: float, sparsity: float, sample_ratio: float = 0.01,
                 seed: int = 0, device: int = 0, debug_sample_rank: int = 0,
                 nesterov: bool = False, select_mode: int = 0, clip_scope: int = 0):
        numel = (ctypes.c_int64 * len(tensor_numel))(*[int(n) for n in tensor_numel])
        cfg = Config(len(tensor_numel), int(num_workers), numel, float(momentum),
                     float(clip_threshold), float(sparsity), float(sample_ratio), int(seed),
                     int(device), int(debug_sample_rank), int(bool(nesterov)), int(select_mode),
                     int(clip_scope))
        self._h = _vp()
        self.num_tensors = len(tensor_numel)
        self.device = int(device)
        _check(_lib.dgc_state_create(ctypes.byref(cfg), ctypes.byref(self._h)), "dgc_state_create")
        self._refresh_layout()

    def _refresh_layout(self) -> None:
        T = self.num_tensors
        off = np.zeros(T, np.int64)
        k = np.zeros(T, np.int64)
        out = np.zeros(T + 1, np.int64)
        alen = ctypes.c_int64()
        _check(_lib.dgc_layout(self._h, off.ctypes.data_as(_i64p), k.ctypes.data_as(_i64p),
                               out.ctypes.data_as(_i64p), ctypes.byref(alen)), "dgc_layout")
        self.arena_offset, self.k, self.out_offset, self.arena_len = off, k, out, int(alen.value)
        self.max_nnz = int(_lib.dgc_max_nnz(self._h))

    def close(self) -> None:
        if self._h:
            _check(_lib.dgc_state_destroy(self._h), "dgc_state_destroy")
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_sparsity(self, sparsity: float) -> None:
        _check(_lib.dgc_set_sparsity(self._h, float(sparsity)), "dgc_set_sparsity")
        self._refresh_layout()

    def compress(self, grad: torch.Tensor, out_idx: torch.Tensor, out_val: torch.Tensor,
                 stream=None) -> None:
        if grad.numel() != self.arena_len:
            raise ValueError("gradient arena has the wrong length")
        cap = min(out_idx.numel(), out_val.numel())
        _check(_lib.dgc_compress(self._h, _dev(grad, torch.float32), _dev(out_idx, torch.int32),
                                 _dev(out_val, torch.float32), cap, _stream(stream)),
               "dgc_compress")

    def compress_host(self, grad: torch.Tensor, out_idx: torch.Tensor, out_val: torch.Tensor,
                      stream=None) -> None:
        for t, dt in ((grad, torch.float32), (out_idx, torch.int32), (out_val, torch.float32)):
            if t.is_cuda or t.dtype != dt or not t.is_contiguous():
                raise ValueError("expected contiguous host tensors")
        if grad.numel() != self.arena_len:
            raise ValueError("gradient arena has the wrong length")
        cap = min(out_idx.numel(), out_val.numel())
        _check(_lib.dgc_compress_host(self._h, grad.data_ptr(), out_idx.data_ptr(),
                                      out_val.data_ptr(), cap, _stream(stream)),
               "dgc_compress_host")

    def status(self, stream=None) -> Status:
        s = Status()
        _check(_lib.dgc_get_status(self._h, _stream(stream), ctypes.byref(s)), "dgc_get_status")
        return s

    def nnz(self, stream=None):
        """(total, per-tensor) entries written by the last compress call."""
        total = ctypes.c_int64()
        per = np.zeros(self.num_tensors, np.int64)
        _check(_lib.dgc_get_nnz(self._h, _stream(stream), ctypes.byref(total),
                                per.ctypes.data_as(_i64p)), "dgc_get_nnz")
        return int(total.value), per

    def thresholds(self, stream=None):
        kth = np.zeros(self.num_tensors, np.uint32)
        cand = np.zeros(self.num_tensors, np.int32)
        _check(_lib.dgc_get_thresholds(self._h, _stream(stream), kth.ctypes.data, cand.ctypes.data),
               "dgc_get_thresholds")
        return kth, cand

    def clip(self, stream=None):
        """(norms float64[T], coefficients float32[T]) of the last compress call's clipping."""
        norms = np.zeros(self.num_tensors, np.float64)
        coefs = np.ones(self.num_tensors, np.float32)
        _check(_lib.dgc_get_clip(self._h, _stream(stream), norms.ctypes.data, coefs.ctypes.data),
               "dgc_get_clip")
        return norms, coefs

    def profile_enable(self, max_calls: int) -> None:
        _check(_lib.dgc_profile_enable(self._h, int(max_calls)), "dgc_profile_enable")

    def profile_read(self, capacity: int) -> np.ndarray:
        """[calls, 5] stage durations in ms: norm, sample, streaming pass, select, emit."""
        ms = np.zeros((max(int(capacity), 1), 5), np.float32)
        n = ctypes.c_int32()
        _check(_lib.dgc_profile_read(self._h, ms.ctypes.data, int(capacity), ctypes.byref(n)),
               "dgc_profile_read")
        return ms[:n.value].copy()

    def read(self, stream=None):
        u = np.empty(self.arena_len, np.float32)
        v = np.empty(self.arena_len, np.float32)
        _check(_lib.dgc_state_read(self._h, u.ctypes.data, v.ctypes.data, _stream(stream)),
               "dgc_state_read")
        return u, v

    def write(self, u: Optional[np.ndarray], v: Optional[np.ndarray], stream=None) -> None:
        for a in (u, v):
            if a is not None and (a.dtype != np.float32 or a.size != self.arena_len
                                  or not a.flags["C_CONTIGUOUS"]):
                raise ValueError("expected contiguous float32 arrays of arena_len")
        _check(_lib.dgc_state_write(self._h, None if u is None else u.ctypes.data,
                                    None if v is None else v.ctypes.data, _stream(stream)),
               "dgc_state_write")

    def timeline_enable(self, on: bool = True) -> None:
        _check(_lib.dgc_timeline_enable(self._h, int(bool(on))), "dgc_timeline_enable")

    def timeline_read(self, stream=None) -> np.ndarray:
        """[4 kernels][first block start, last block start] in ns of the GPU timer."""
        out = np.zeros(8, np.uint64)
        _check(_lib.dgc_timeline_read(self._h, _stream(stream), out.ctypes.data),
               "dgc_timeline_read")
        return out.reshape(4, 2)

    def set_iterations(self, iterations: int, stream=None) -> None:
        _check(_lib.dgc_state_set_iterations(self._h, int(iterations), _stream(stream)),
               "dgc_state_set_iterations")


def compress_batch(states: Sequence["State"], grads: Sequence[torch.Tensor],
                   out_idx: Sequence[torch.Tensor], out_val: Sequence[torch.Tensor],
                   stream=None) -> None:
    """dgc_compress for several workers on one GPU with overlapped kernels (same results)."""
    n = len(states)
    sp = (_vp * n)(*[st._h for st in states])
    gp = (_vp * n)(*[_dev(g, torch.float32) for g in grads])
    ip = (_vp * n)(*[_dev(t, torch.int32) for t in out_idx])
    vp = (_vp * n)(*[_dev(t, torch.float32) for t in out_val])
    cap = (ctypes.c_int64 * n)(*[min(a.numel(), b.numel()) for a, b in zip(out_idx, out_val)])
    for st, g in zip(states, grads):
        if g.numel() != st.arena_len:
            raise ValueError("gradient arena has the wrong length")
    _check(_lib.dgc_compress_batch(n, sp, gp, ip, vp, cap, _stream(stream)), "dgc_compress_batch")


def compress_host_batch(states: Sequence["State"], grads: Sequence[torch.Tensor],
                        out_idx: Sequence[torch.Tensor], out_val: Sequence[torch.Tensor],
                        stream=None) -> None:
    """dgc_compress_host for several workers on one GPU: host gradients in, host lists out,
    the workers' copies and kernels overlapped; the lists are valid on return."""
    n = len(states)
    for st, g, a, b in zip(states, grads, out_idx, out_val):
        for t, dt in ((g, torch.float32), (a, torch.int32), (b, torch.float32)):
            if t.is_cuda or t.dtype != dt or not t.is_contiguous():
                raise ValueError("expected contiguous host tensors")
        if g.numel() != st.arena_len:
            raise ValueError("gradient arena has the wrong length")
    sp = (_vp * n)(*[st._h for st in states])
    gp = (_vp * n)(*[g.data_ptr() for g in grads])
    ip = (_vp * n)(*[t.data_ptr() for t in out_idx])
    vp = (_vp * n)(*[t.data_ptr() for t in out_val])
    cap = (ctypes.c_int64 * n)(*[min(a.numel(), b.numel()) for a, b in zip(out_idx, out_val)])
    _check(_lib.dgc_compress_host_batch(n, sp, gp, ip, vp, cap, _stream(stream)),
           "dgc_compress_host_batch")


def decode_workspace_bytes(num_workers: int, dense_len: int) -> int:
    return int(_lib.dgc_decode_workspace_bytes(int(num_workers), int(dense_len)))


def decode_accumulate(idx_lists: Sequence[torch.Tensor], val_lists: Sequence[torch.Tensor],
                      dense_out: torch.Tensor, workspace: torch.Tensor, stream=None,
                      nnz: Optional[Sequence[int]] = None) -> None:
    n = len(idx_lists)
    ip = (_vp * n)(*[_dev(t, torch.int32) for t in idx_lists])
    vp = (_vp * n)(*[_dev(t, torch.float32) for t in val_lists])
    cnt = (ctypes.c_int64 * n)(*[int(c) for c in (nnz if nnz is not None
                                                  else [t.numel() for t in idx_lists])])
    _check(_lib.dgc_decode_accumulate(n, ip, vp, cnt, _dev(dense_out, torch.float32),
                                      dense_out.numel(), workspace.data_ptr(),
                                      workspace.numel() * workspace.element_size(),
                                      _stream(stream)), "dgc_decode_accumulate")


def decode_rejected(num_workers: int, dense_len: int, workspace: Optional[torch.Tensor] = None,
                    stream=None) -> int:
    """Pairs the last decode call on `workspace` (None: the built-in scratch of the static
    variant) skipped or flagged because their index was out of range or out of order."""
    out = ctypes.c_int64()
    _check(_lib.dgc_decode_rejected(int(num_workers), int(dense_len),
                                    None if workspace is None else workspace.data_ptr(),
                                    _stream(stream), ctypes.byref(out)), "dgc_decode_rejected")
    return int(out.value)


def decode_accumulate_sgd(idx_lists: Sequence[torch.Tensor], val_lists: Sequence[torch.Tensor],
                          dense_out: torch.Tensor, w: torch.Tensor, lr: float,
                          workspace: torch.Tensor, stream=None,
                          nnz: Optional[Sequence[int]] = None) -> None:
    """dense_out <- sum of the workers' lists and w <- w - lr * dense_out in one pass."""
    n = len(idx_lists)
    ip = (_vp * n)(*[_dev(t, torch.int32) for t in idx_lists])
    vp = (_vp * n)(*[_dev(t, torch.float32) for t in val_lists])
    cnt = (ctypes.c_int64 * n)(*[int(c) for c in (nnz if nnz is not None
                                                  else [t.numel() for t in idx_lists])])
    if w.numel() != dense_out.numel():
        raise ValueError("length mismatch")
    _check(_lib.dgc_decode_accumulate_sgd(n, ip, vp, cnt, _dev(dense_out, torch.float32),
                                          _dev(w, torch.float32), w.numel(), float(lr),
                                          workspace.data_ptr(),
                                          workspace.numel() * workspace.element_size(),
                                          _stream(stream)), "dgc_decode_accumulate_sgd")


def decode_apply_sgd(idx_lists: Sequence[torch.Tensor], val_lists: Sequence[torch.Tensor],
                     w: torch.Tensor, lr: float, workspace: torch.Tensor, stream=None,
                     nnz: Optional[Sequence[int]] = None) -> None:
    """w <- w - lr * (sum of the workers' sparse lists), touching only the listed entries."""
    n = len(idx_lists)
    ip = (_vp * n)(*[_dev(t, torch.int32) for t in idx_lists])
    vp = (_vp * n)(*[_dev(t, torch.float32) for t in val_lists])
    cnt = (ctypes.c_int64 * n)(*[int(c) for c in (nnz if nnz is not None
                                                  else [t.numel() for t in idx_lists])])
    _check(_lib.dgc_decode_apply_sgd(n, ip, vp, cnt, _dev(w, torch.float32), w.numel(), float(lr),
                                     workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(),
                                     _stream(stream)), "dgc_decode_apply_sgd")


def runlength_max_entries(nnz: int, dense_len: int) -> int:
    return int(_lib.dgc_runlength_max_entries(int(nnz), int(dense_len)))


def encode_runlength(idx: torch.Tensor, val: torch.Tensor, dense_len: int, stream=None):
    """Sec. 3.1 encode(): returns (runs uint16, values float32) device tensors trimmed to the
    encoded length (synchronises to read the count)."""
    nnz = idx.numel()
    cap = runlength_max_entries(nnz, dense_len)
    runs = torch.empty(cap, dtype=torch.uint16, device=idx.device)
    values = torch.empty(cap, dtype=torch.float32, device=idx.device)
    count = torch.zeros(1, dtype=torch.int64, device=idx.device)
    ws = torch.empty(max(int(_lib.dgc_runlength_workspace_bytes(nnz)), 8), dtype=torch.uint8,
                     device=idx.device)
    _check(_lib.dgc_encode_runlength(_dev(idx, torch.int32) if nnz else None,
                                     _dev(val, torch.float32) if nnz else None, nnz,
                                     runs.data_ptr(), values.data_ptr(), cap, count.data_ptr(),
                                     ws.data_ptr(), ws.numel(), _stream(stream)),
           "dgc_encode_runlength")
    n = int(count.item())
    return runs[:n], values[:n]


def decode_runlength(runs: torch.Tensor, values: torch.Tensor, stream=None):
    """Inverse of encode_runlength: (idx int32, val float32, dense position after the last entry)."""
    n = runs.numel()
    idx = torch.empty(n, dtype=torch.int32, device=runs.device)
    val = torch.empty(n, dtype=torch.float32, device=runs.device)
    end = torch.zeros(1, dtype=torch.int64, device=runs.device)
    ws = torch.empty(max(int(_lib.dgc_runlength_workspace_bytes(n)), 8), dtype=torch.uint8,
                     device=runs.device)
    if not (runs.is_cuda and runs.dtype == torch.uint16 and runs.is_contiguous()):
        raise ValueError("expected a contiguous CUDA uint16 tensor")
    _check(_lib.dgc_decode_runlength(runs.data_ptr() if n else None,
                                     _dev(values, torch.float32) if n else None, n,
                                     idx.data_ptr(), val.data_ptr(), end.data_ptr(), ws.data_ptr(),
                                     ws.numel(), _stream(stream)), "dgc_decode_runlength")
    return idx, val, int(end.item())


STATIC_DECODE_WORDS = 1 << 18


def decode_accumulate_static(idx_lists: Sequence[torch.Tensor], val_lists: Sequence[torch.Tensor],
                             dense_out: torch.Tensor, stream=None,
                             nnz: Optional[Sequence[int]] = None) -> None:
    """dgc_decode_accumulate without a workspace argument, for callers that may not allocate
    device memory: the scratch is a fixed 1 MiB array inside the library.  Raises DgcError
    (ECAPACITY) when workers x (tiles + 1025) exceeds STATIC_DECODE_WORDS.  Calls on one device
    share that scratch, so do not let two of them overlap on the GPU."""
    n = len(idx_lists)
    ip = (_vp * n)(*[_dev(t, torch.int32) for t in idx_lists])
    vp = (_vp * n)(*[_dev(t, torch.float32) for t in val_lists])
    cnt = (ctypes.c_int64 * n)(*[int(c) for c in (nnz if nnz is not None
                                                  else [t.numel() for t in idx_lists])])
    _check(_lib.dgc_decode_accumulate_static(n, ip, vp, cnt, _dev(dense_out, torch.float32),
                                             dense_out.numel(), _stream(stream)),
           "dgc_decode_accumulate_static")


def apply_sgd(w: torch.Tensor, dense_grad: torch.Tensor, lr: float, stream=None) -> None:
    if w.numel() != dense_grad.numel():
        raise ValueError("length mismatch")
    _check(_lib.dgc_apply_sgd(_dev(w, torch.float32), _dev(dense_grad, torch.float32), w.numel(),
                              float(lr), _stream(stream)), "dgc_apply_sgd")
