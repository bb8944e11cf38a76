"""The allocation-free decode entry point (dgc_decode_accumulate_static), called through the
C ABI, must give bit for bit what dgc_decode_accumulate gives.  Its scratch is one fixed array
inside the library that every call on the device reuses, so the check is made on two calls in a
row with different list contents and a different dense length: the second call must not be
disturbed by what the first one left behind.  This file sorts last on purpose, so that a run
that stops at the first failure has already been through every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _lists(rng, dense_len, workers, density):
    idx, val = [], []
    for w in range(workers):
        k = int(dense_len * density * (1.0 + 0.5 * (w % 3)))
        i = np.sort(rng.choice(dense_len, size=min(k, dense_len), replace=False)).astype(np.int32)
        idx.append(torch.from_numpy(i).cuda())
        val.append(torch.from_numpy(rng.standard_normal(i.size).astype(np.float32)).cuda())
    return idx, val


def test_static_decode_matches_workspace_decode_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests need a B200")
    from paper_1712_01887_b200 import binding as B
    rng = np.random.default_rng(20241125)
    # second call: fewer workers, shorter output, sparser lists than the first
    for dense_len, workers, density in ((3_000_001, 8, 0.002), (70_003, 3, 0.0005)):
        idx, val = _lists(rng, dense_len, workers, density)
        ref = torch.full((dense_len,), float("nan"), dtype=torch.float32, device="cuda")
        ws = torch.empty(B.decode_workspace_bytes(workers, dense_len), dtype=torch.uint8,
                         device="cuda")
        B.decode_accumulate(idx, val, ref, ws)
        out = torch.full((dense_len,), float("nan"), dtype=torch.float32, device="cuda")
        B.decode_accumulate_static(idx, val, out)
        torch.cuda.synchronize()
        # same tolerance as the other decode tests: none (bit-exact)
        assert torch.equal(out.view(torch.int32), ref.view(torch.int32))
        assert not torch.isnan(out).any()
        assert B.decode_rejected(workers, dense_len) == 0     # the built-in scratch's input check
        # what the entry point is for: once the first call on the device has looked the scratch
        # up, a call takes no device memory, neither from the driver nor from torch's allocator
        free0, _ = torch.cuda.mem_get_info()
        held0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        B.decode_accumulate_static(idx, val, out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (held0, reserved0)
        assert torch.equal(out.view(torch.int32), ref.view(torch.int32))


def test_static_decode_rejects_problems_beyond_its_fixed_scratch():
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests need a B200")
    from paper_1712_01887_b200 import binding as B
    workers = 64
    # per worker: one boundary word per tile of 4096 elements, one more, and 1024 check words
    tiles_allowed = B.STATIC_DECODE_WORDS // workers - 1 - 1024
    too_long = (tiles_allowed + 1) * 4096
    empty_i = [torch.zeros(0, dtype=torch.int32, device="cuda") for _ in range(workers)]
    empty_v = [torch.zeros(0, dtype=torch.float32, device="cuda") for _ in range(workers)]
    dense = torch.empty(too_long, dtype=torch.float32, device="cuda")
    with pytest.raises(B.DgcError) as e:
        B.decode_accumulate_static(empty_i, empty_v, dense)
    assert e.value.code == B.ECAPACITY
    # the largest length that fits is accepted and decodes to all zeros
    ok = torch.full((tiles_allowed * 4096,), 1.0, dtype=torch.float32, device="cuda")
    B.decode_accumulate_static(empty_i, empty_v, ok)
    torch.cuda.synchronize()
    assert not ok.any()
