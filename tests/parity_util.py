"""Shared driver for the GPU-vs-oracle parity tests: runs the CUDA library
(through the C ABI binding) and the CPU oracle on the same seeded gradients and
compares element by element."""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np
import torch

from oracle import dgc_oracle as O
from paper_1712_01887_b200 import binding as B

NORM_RTOL = 1e-6          # clipping norm: relative tolerance (fp64 sums in different orders)


@dataclass
class ParityReport:
    worker_iterations: int = 0
    coef_overrides: int = 0          # oracle re-run with the GPU's clip coefficient
    full_select: int = 0             # tensors that took the full-selection path on the GPU
    max_norm_rel_err: float = 0.0
    notes: List[str] = field(default_factory=list)


def _assert_bits(a: np.ndarray, b: np.ndarray, what: str) -> None:
    """Bit for bit -- except that a NaN matches any NaN at the same place: IEEE 754 leaves sign
    and payload of a NaN that an operation produces (Inf - Inf) to the hardware, and x86 and the
    GPU choose differently."""
    if a.tobytes() != b.tobytes():
        na, nb = np.isnan(a), np.isnan(b)
        if na.any() and np.array_equal(na, nb):
            a, b = np.where(na, np.float32(0), a), np.where(nb, np.float32(0), b)
            if a.tobytes() == b.tobytes():
                return
        bad = np.flatnonzero(a.view(np.uint32) != b.view(np.uint32))
        raise AssertionError(f"{what}: {bad.size} of {a.size} differ, first at {bad[:5]}: "
                             f"{a[bad[:5]]} vs {b[bad[:5]]}")


class Pair:
    """One worker on both sides."""

    def __init__(self, numel: Sequence[int], num_workers: int, momentum: float, clip: float,
                 sparsity: float, seed: int = 0, sample_ratio: float = 0.01,
                 debug_sample_rank: int = 0, nesterov: bool = False):
        self.gpu = B.State(numel, num_workers, momentum, clip, sparsity, sample_ratio=sample_ratio,
                           seed=seed, debug_sample_rank=debug_sample_rank, nesterov=nesterov)
        self.cpu = O.Worker(self.gpu.arena_offset, numel, self.gpu.arena_len, num_workers,
                            momentum, clip, sparsity, nesterov=nesterov)
        self.clip = clip
        self.numel = list(numel)
        self._alloc_out()

    def _alloc_out(self):
        n = max(self.gpu.max_nnz, 1)
        self.out_idx = torch.empty(n, dtype=torch.int32, device="cuda")
        self.out_val = torch.empty(n, dtype=torch.float32, device="cuda")

    def set_sparsity(self, s: float):
        self.gpu.set_sparsity(s)
        self.cpu.set_sparsity(s)
        assert np.array_equal(self.gpu.k, self.cpu.k)
        assert np.array_equal(self.gpu.out_offset, self.cpu.out_offset)
        self._alloc_out()

    def step(self, g: np.ndarray, rep: ParityReport, check_state: bool = True):
        assert np.array_equal(self.gpu.k, self.cpu.k)
        assert self.gpu.max_nnz == self.cpu.nnz
        gd = torch.from_numpy(g).cuda()
        self.out_idx.fill_(-7)
        self.gpu.compress(gd, self.out_idx, self.out_val)
        st = self.gpu.status()
        nnz = self.gpu.max_nnz
        gi = self.out_idx[:nnz].cpu().numpy()
        gv = self.out_val[:nnz].cpu().numpy()
        # the gradient must not be modified
        assert torch.equal(gd.view(torch.int32), torch.from_numpy(g).cuda().view(torch.int32))
        snap = (self.cpu.u.copy(), self.cpu.v.copy()) if self.clip > 0 else None
        r = self.cpu.compress(g)
        if self.clip > 0:
            rel = abs(st.grad_norm - r.norm) / max(r.norm, 1e-300)
            rep.max_norm_rel_err = max(rep.max_norm_rel_err, rel)
            assert rel <= NORM_RTOL, (st.grad_norm, r.norm)
            if np.float32(st.clip_coef).tobytes() != np.float32(r.coef).tobytes():
                # the two fp64 sums rounded to different fp32 coefficients: follow the GPU's
                self.cpu.u[:], self.cpu.v[:] = snap
                r = self.cpu.compress(g, coef_override=st.clip_coef)
                rep.coef_overrides += 1
        else:
            assert st.clip_coef == 1.0
        rep.worker_iterations += 1
        rep.full_select += int(st.full_select_last)
        if gi.tobytes() != r.idx.tobytes():
            # With equal clip coefficients (ensured above) the selected set is unique: any
            # difference is an error, however close the entries are to the threshold.
            diff = np.setxor1d(gi, r.idx)
            raise AssertionError(f"selected sets differ at {diff.size} entries, first {diff[:8]}")
        _assert_bits(gv, r.val, "sent values")
        if check_state:
            u, v = self.gpu.read()
            _assert_bits(u, self.cpu.u, "u")
            _assert_bits(v, self.cpu.v, "v")
        return gi, gv, st

    def close(self):
        self.gpu.close()


def arena_with_padding_poison(arena_len: int, offsets, numel) -> np.ndarray:
    """A gradient arena whose padding slots hold NaN: neither side may read them."""
    a = np.full(arena_len, np.float32(np.nan))
    for o, n in zip(offsets, numel):
        a[o:o + n] = 0.0
    return a


def receive_side(idx_lists, val_lists, dense_len: int, w_init: np.ndarray, lr: float):
    """Decode + SGD on both sides; returns the dense gradient and the new weights (GPU's,
    after they were checked bit-exact against the oracle's)."""
    n = len(idx_lists)
    di = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in idx_lists]
    dv = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in val_lists]
    dense = torch.full((dense_len,), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(B.decode_workspace_bytes(n, dense_len), 4), dtype=torch.uint8,
                     device="cuda")
    B.decode_accumulate(di, dv, dense, ws)
    ref = O.decode_accumulate(idx_lists, val_lists, dense_len)
    _assert_bits(dense.cpu().numpy(), ref, "decoded dense gradient")
    wd = torch.from_numpy(w_init.copy()).cuda()
    B.apply_sgd(wd, dense, lr)
    wref = w_init.copy()
    O.apply_sgd(wref, ref, lr)
    _assert_bits(wd.cpu().numpy(), wref, "weights after SGD")
    # the fused form (Eq. 5 third term applied to the listed entries only) must give the same bits
    wf = torch.from_numpy(w_init.copy()).cuda()
    B.decode_apply_sgd(di, dv, wf, lr, ws)
    _assert_bits(wf.cpu().numpy(), wref, "weights after fused sparse decode + SGD")
    # and the one-pass dense form: same dense gradient, same weights
    wg = torch.from_numpy(w_init.copy()).cuda()
    dense2 = torch.full((dense_len,), float("nan"), dtype=torch.float32, device="cuda")
    B.decode_accumulate_sgd(di, dv, dense2, wg, lr, ws)
    _assert_bits(dense2.cpu().numpy(), ref, "dense gradient of the one-pass decode + SGD")
    _assert_bits(wg.cpu().numpy(), wref, "weights after the one-pass decode + SGD")
    return ref, wref
