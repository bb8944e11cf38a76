"""ctypes access to the CPU oracle (oracle/dgc_oracle.cpp).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline may import this module; the CUDA library and its Python binding must
not.  It marshals numpy arrays to the C functions and holds no arithmetic of
the method itself.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dgc_oracle.cpp")
_LIB = os.path.join(_HERE, "libdgc_oracle.so")

_i64p = ctypes.POINTER(ctypes.c_int64)
_i32p = ctypes.POINTER(ctypes.c_int32)
_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (single thread, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.dgc_oracle_topk_count.restype = ctypes.c_int64
        L.dgc_oracle_topk_count.argtypes = [ctypes.c_int64, ctypes.c_double]
        L.dgc_oracle_warmup_sparsity.restype = ctypes.c_double
        L.dgc_oracle_warmup_sparsity.argtypes = [ctypes.c_int32]
        L.dgc_oracle_clip_coef.restype = None
        L.dgc_oracle_clip_coef.argtypes = [ctypes.c_int32, _i64p, _i64p, _f32p, ctypes.c_double,
                                           ctypes.c_int32, _f64p, _f32p]
        L.dgc_oracle_momentum_correction.restype = None
        L.dgc_oracle_momentum_correction.argtypes = [ctypes.c_int32, _i64p, _i64p, _f32p, _f32p,
                                                     _f32p, ctypes.c_float, ctypes.c_float,
                                                     ctypes.c_int32]
        L.dgc_oracle_select_topk.restype = None
        L.dgc_oracle_select_topk.argtypes = [ctypes.c_int64, _f32p, ctypes.c_int64, _i64p,
                                             ctypes.c_int32]
        L.dgc_oracle_compress.restype = None
        L.dgc_oracle_compress.argtypes = [ctypes.c_int32, _i64p, _i64p, _i64p, _i64p, _f32p, _f32p,
                                          _f32p, ctypes.c_float, ctypes.c_double, ctypes.c_int32,
                                          ctypes.c_int32, ctypes.c_float, ctypes.c_int32,
                                          ctypes.c_int32, _i32p, _f32p, _f64p, _f32p]
        L.dgc_oracle_compress_clip_per_tensor.restype = None
        L.dgc_oracle_compress_clip_per_tensor.argtypes = [
            ctypes.c_int32, _i64p, _i64p, _i64p, _i64p, _f32p, _f32p, _f32p, ctypes.c_float,
            ctypes.c_double, ctypes.c_int32, _f32p, ctypes.c_int32, ctypes.c_int32, _i32p, _f32p,
            _f64p, _f32p]
        L.dgc_oracle_decode_accumulate.restype = None
        L.dgc_oracle_decode_accumulate.argtypes = [ctypes.c_int32, ctypes.POINTER(_i32p),
                                                   ctypes.POINTER(_f32p), _i64p, _f32p,
                                                   ctypes.c_int64]
        L.dgc_oracle_apply_sgd.restype = None
        L.dgc_oracle_apply_sgd.argtypes = [_f32p, _f32p, ctypes.c_int64, ctypes.c_float]
        L.dgc_oracle_sample_count.restype = ctypes.c_int64
        L.dgc_oracle_sample_count.argtypes = [ctypes.c_int64, ctypes.c_double]
        L.dgc_oracle_mix64.restype = ctypes.c_uint64
        L.dgc_oracle_mix64.argtypes = [ctypes.c_uint64]
        L.dgc_oracle_sample_positions.restype = None
        L.dgc_oracle_sample_positions.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_uint64,
                                                  ctypes.c_int32, _i64p]
        L.dgc_oracle_select_from_sample.restype = ctypes.c_int64
        L.dgc_oracle_select_from_sample.argtypes = [ctypes.c_int64, _f32p, _i64p, ctypes.c_int64,
                                                    ctypes.c_int64, ctypes.c_double, _i64p,
                                                    ctypes.POINTER(ctypes.c_uint32)]
        L.dgc_oracle_compress_sampled.restype = ctypes.c_int64
        L.dgc_oracle_compress_sampled.argtypes = [
            ctypes.c_int32, _i64p, _i64p, _i64p, _f32p, _f32p, _f32p, ctypes.c_float,
            ctypes.c_double, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_int32,
            ctypes.c_double, ctypes.c_double, ctypes.c_uint64, ctypes.c_int64, _i32p, _f32p,
            _i64p, _f64p, _f32p]
        L.dgc_oracle_encode_runlength.restype = ctypes.c_int64
        L.dgc_oracle_encode_runlength.argtypes = [_i32p, _f32p, ctypes.c_int64,
                                                  ctypes.POINTER(ctypes.c_uint16), _f32p,
                                                  ctypes.c_int64]
        L.dgc_oracle_decode_runlength.restype = ctypes.c_int64
        L.dgc_oracle_decode_runlength.argtypes = [ctypes.POINTER(ctypes.c_uint16), _f32p,
                                                  ctypes.c_int64, _i32p, _f32p]
        _lib = L
    return _lib


def _p(a: np.ndarray, typ):
    return a.ctypes.data_as(typ)


def _chk(a: np.ndarray, dtype) -> np.ndarray:
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a


def topk_count(n: int, sparsity: float) -> int:
    return int(lib().dgc_oracle_topk_count(int(n), float(sparsity)))


def warmup_sparsity(stage: int) -> float:
    return float(lib().dgc_oracle_warmup_sparsity(int(stage)))


def clip_coef(offset, numel, g, clip_threshold: float, num_workers: int):
    offset = np.ascontiguousarray(offset, dtype=np.int64)
    numel = np.ascontiguousarray(numel, dtype=np.int64)
    norm = ctypes.c_double()
    coef = ctypes.c_float()
    lib().dgc_oracle_clip_coef(len(numel), _p(offset, _i64p), _p(numel, _i64p),
                               _p(_chk(g, np.float32), _f32p), float(clip_threshold),
                               int(num_workers), ctypes.byref(norm), ctypes.byref(coef))
    return norm.value, np.float32(coef.value)


def momentum_correction(offset, numel, u, v, g, momentum: float, coef: float,
                        nesterov: bool = False) -> None:
    offset = np.ascontiguousarray(offset, dtype=np.int64)
    numel = np.ascontiguousarray(numel, dtype=np.int64)
    lib().dgc_oracle_momentum_correction(len(numel), _p(offset, _i64p), _p(numel, _i64p),
                                         _p(_chk(u, np.float32), _f32p),
                                         _p(_chk(v, np.float32), _f32p),
                                         _p(_chk(g, np.float32), _f32p),
                                         ctypes.c_float(momentum), ctypes.c_float(coef),
                                         int(nesterov))


def select_topk(v: np.ndarray, k: int, brute_force: bool = False) -> np.ndarray:
    v = _chk(v, np.float32)
    sel = np.empty(k, dtype=np.int64)
    lib().dgc_oracle_select_topk(v.size, _p(v, _f32p), int(k), _p(sel, _i64p), int(brute_force))
    return sel


@dataclass
class CompressResult:
    idx: np.ndarray      # int32, index into the arena, ascending per tensor
    val: np.ndarray      # float32
    norm: float          # L2 norm of the whole gradient set (fp64)
    coef: np.float32     # clip coefficient that was applied


class Worker:
    """State of one worker (u, v) plus the segment table of its gradient set."""

    def __init__(self, offset, numel, arena_len: int, num_workers: int, momentum: float,
                 clip_threshold: float, sparsity: float, nesterov: bool = False):
        self.offset = np.ascontiguousarray(offset, dtype=np.int64)
        self.numel = np.ascontiguousarray(numel, dtype=np.int64)
        self.arena_len = int(arena_len)
        self.num_workers = int(num_workers)
        self.momentum = float(momentum)
        self.clip_threshold = float(clip_threshold)
        self.nesterov = bool(nesterov)
        self.u = np.zeros(self.arena_len, dtype=np.float32)   # Algorithm 4: U <- 0
        self.v = np.zeros(self.arena_len, dtype=np.float32)   # Algorithm 4: V <- 0
        self.set_sparsity(sparsity)

    def set_sparsity(self, sparsity: float) -> None:
        self.sparsity = float(sparsity)
        self.k = np.array([topk_count(n, sparsity) for n in self.numel], dtype=np.int64)
        self.out_offset = np.zeros(len(self.k) + 1, dtype=np.int64)
        np.cumsum(self.k, out=self.out_offset[1:])

    @property
    def nnz(self) -> int:
        return int(self.out_offset[-1])

    def compress(self, g: np.ndarray, coef_override=None, brute_force: bool = False) -> CompressResult:
        g = _chk(g, np.float32)
        assert g.size == self.arena_len
        idx = np.empty(self.nnz, dtype=np.int32)
        val = np.empty(self.nnz, dtype=np.float32)
        norm = ctypes.c_double()
        coef = ctypes.c_float()
        lib().dgc_oracle_compress(
            len(self.numel), _p(self.offset, _i64p), _p(self.numel, _i64p), _p(self.k, _i64p),
            _p(self.out_offset, _i64p), _p(self.u, _f32p), _p(self.v, _f32p), _p(g, _f32p),
            ctypes.c_float(self.momentum), self.clip_threshold, self.num_workers,
            int(coef_override is not None),
            ctypes.c_float(0.0 if coef_override is None else float(coef_override)),
            int(brute_force), int(self.nesterov), _p(idx, _i32p), _p(val, _f32p),
            ctypes.byref(norm),
            ctypes.byref(coef))
        return CompressResult(idx, val, norm.value, np.float32(coef.value))

    def compress_clip_per_tensor(self, g: np.ndarray, coef_override=None,
                                 brute_force: bool = False):
        """One iteration with every tensor clipped by its own L2 norm: returns
        (CompressResult with norm = per-tensor norms, coef = per-tensor coefficients)."""
        g = _chk(g, np.float32)
        assert g.size == self.arena_len
        T = len(self.numel)
        idx = np.empty(self.nnz, dtype=np.int32)
        val = np.empty(self.nnz, dtype=np.float32)
        norms = np.zeros(T, dtype=np.float64)
        coefs = np.ones(T, dtype=np.float32)
        ov = None
        if coef_override is not None:
            ov = _chk(np.ascontiguousarray(coef_override, dtype=np.float32), np.float32)
            assert ov.size == T
        lib().dgc_oracle_compress_clip_per_tensor(
            T, _p(self.offset, _i64p), _p(self.numel, _i64p), _p(self.k, _i64p),
            _p(self.out_offset, _i64p), _p(self.u, _f32p), _p(self.v, _f32p), _p(g, _f32p),
            ctypes.c_float(self.momentum), self.clip_threshold, self.num_workers,
            None if ov is None else _p(ov, _f32p), int(brute_force), int(self.nesterov),
            _p(idx, _i32p), _p(val, _f32p), _p(norms, _f64p), _p(coefs, _f32p))
        return CompressResult(idx, val, norms, coefs)


def sample_count(n: int, sample_ratio: float = 0.01) -> int:
    """Sec. 5: size of the sample of a tensor of n elements, ceil(ratio * n)."""
    return int(lib().dgc_oracle_sample_count(int(n), float(sample_ratio)))


def mix64(x: int) -> int:
    return int(lib().dgc_oracle_mix64(ctypes.c_uint64(int(x) & 0xFFFFFFFFFFFFFFFF)))


def call_seed(seed: int, iteration: int) -> int:
    """Seed of the sample positions of one call (state seed, calls completed before it)."""
    return mix64((int(seed) * 0x9E3779B97F4A7C15 + int(iteration)) & 0xFFFFFFFFFFFFFFFF)


def sample_positions(n: int, count: int, seed: int, tensor_index: int) -> np.ndarray:
    """The `count` sample positions of tensor `tensor_index` for the call seed `seed`."""
    pos = np.empty(int(count), dtype=np.int64)
    lib().dgc_oracle_sample_positions(int(n), int(count), ctypes.c_uint64(int(seed)),
                                      int(tensor_index), _p(pos, _i64p))
    return pos


def select_from_sample(v: np.ndarray, positions: np.ndarray, k: int, sparsity: float):
    """Sec. 5 selection of one tensor from an explicit sample: (chosen indices ascending,
    bit pattern of the threshold)."""
    v = _chk(v, np.float32)
    positions = _chk(np.ascontiguousarray(positions), np.int64)
    assert positions.size >= 1 and positions.min() >= 0 and positions.max() < v.size
    sel = np.empty(min(v.size, 2 * int(k)), dtype=np.int64)
    thr = ctypes.c_uint32()
    c = lib().dgc_oracle_select_from_sample(v.size, _p(v, _f32p), _p(positions, _i64p),
                                            positions.size, int(k), float(sparsity),
                                            _p(sel, _i64p), ctypes.byref(thr))
    return sel[:c].copy(), int(thr.value)


def compress_sampled(worker: "Worker", g: np.ndarray, seed: int, iteration: int,
                     sample_ratio: float = 0.01, coef_override=None):
    """Paper-literal sampled selection (Sec. 5) on a Worker's state: returns
    (CompressResult with the packed lists, nnz per tensor)."""
    g = _chk(g, np.float32)
    cap = int(np.minimum(worker.numel, 2 * worker.k).sum())
    idx = np.empty(cap, dtype=np.int32)
    val = np.empty(cap, dtype=np.float32)
    nnz = np.zeros(len(worker.numel), dtype=np.int64)
    norm = ctypes.c_double()
    coef = ctypes.c_float()
    n = lib().dgc_oracle_compress_sampled(
        len(worker.numel), _p(worker.offset, _i64p), _p(worker.numel, _i64p), _p(worker.k, _i64p),
        _p(worker.u, _f32p), _p(worker.v, _f32p), _p(g, _f32p), ctypes.c_float(worker.momentum),
        worker.clip_threshold, worker.num_workers, int(coef_override is not None),
        ctypes.c_float(0.0 if coef_override is None else float(coef_override)),
        int(worker.nesterov), worker.sparsity, float(sample_ratio), int(seed), int(iteration),
        _p(idx, _i32p), _p(val, _f32p), _p(nnz, _i64p), ctypes.byref(norm), ctypes.byref(coef))
    return CompressResult(idx[:n].copy(), val[:n].copy(), norm.value, np.float32(coef.value)), nnz


def decode_accumulate(idx_lists, val_lists, dense_len: int) -> np.ndarray:
    n = len(idx_lists)
    idx_lists = [_chk(np.ascontiguousarray(a), np.int32) for a in idx_lists]
    val_lists = [_chk(np.ascontiguousarray(a), np.float32) for a in val_lists]
    ip = (_i32p * n)(*[_p(a, _i32p) for a in idx_lists])
    vp = (_f32p * n)(*[_p(a, _f32p) for a in val_lists])
    nnz = np.array([a.size for a in idx_lists], dtype=np.int64)
    dense = np.empty(int(dense_len), dtype=np.float32)
    lib().dgc_oracle_decode_accumulate(n, ip, vp, _p(nnz, _i64p), _p(dense, _f32p), int(dense_len))
    return dense


def apply_sgd(w: np.ndarray, dense_grad: np.ndarray, lr: float) -> None:
    w = _chk(w, np.float32)
    dense_grad = _chk(dense_grad, np.float32)
    assert w.size == dense_grad.size
    lib().dgc_oracle_apply_sgd(_p(w, _f32p), _p(dense_grad, _f32p), w.size, ctypes.c_float(lr))


def encode_runlength(idx: np.ndarray, val: np.ndarray, capacity: int):
    """Sec. 3.1 encode(): (uint16 zero run lengths, float32 values); raises if capacity is short."""
    idx = _chk(np.ascontiguousarray(idx), np.int32)
    val = _chk(np.ascontiguousarray(val), np.float32)
    runs = np.empty(capacity, dtype=np.uint16)
    values = np.empty(capacity, dtype=np.float32)
    n = lib().dgc_oracle_encode_runlength(_p(idx, _i32p), _p(val, _f32p), idx.size,
                                          runs.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)),
                                          _p(values, _f32p), int(capacity))
    if n < 0:
        raise ValueError("capacity too small")
    return runs[:n].copy(), values[:n].copy()


def decode_runlength(runs: np.ndarray, values: np.ndarray):
    runs = _chk(np.ascontiguousarray(runs), np.uint16)
    values = _chk(np.ascontiguousarray(values), np.float32)
    idx = np.empty(runs.size, dtype=np.int32)
    val = np.empty(runs.size, dtype=np.float32)
    lib().dgc_oracle_decode_runlength(runs.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)),
                                      _p(values, _f32p), runs.size, _p(idx, _i32p), _p(val, _f32p))
    return idx, val
