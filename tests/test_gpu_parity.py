"""GPU parity: the CUDA library (called through the C ABI) against the CPU
oracle on the same seeded inputs.  Bit-exact for indices, sent values, u, v,
decoded sums and weights; clipping norm within 1e-6 relative."""
import numpy as np
import pytest
import torch

from paper_1712_01887_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: the gpu tests need a B200")
    import parity_util
    return parity_util


def _run_workload(P, wl, iterations, workers=None, seed=0, receive=True, schedule=None,
                  check_state=True, nesterov=False):
    N = workers or wl.num_workers
    pairs = [P.Pair(wl.numel, wl.num_workers, wl.momentum, wl.clip_threshold, wl.sparsity,
                    seed=seed + w, sample_ratio=wl.sample_ratio, nesterov=nesterov)
             for w in range(N)]
    rep = P.ParityReport()
    off, L = pairs[0].gpu.arena_offset, pairs[0].gpu.arena_len
    rng = np.random.default_rng(99)
    w_host = rng.standard_normal(L).astype(np.float32)
    for t in range(iterations):
        if schedule is not None:
            s = schedule(t)
            if s != pairs[0].cpu.sparsity:
                for p in pairs:
                    p.set_sparsity(s)
        lists_i, lists_v = [], []
        for w, p in enumerate(pairs):
            g = P.arena_with_padding_poison(L, off, wl.numel)
            I.fill(wl, g, off, worker=w, iteration=t)
            gi, gv, _ = p.step(g, rep, check_state=check_state)
            lists_i.append(gi)
            lists_v.append(gv)
        if receive:
            _, w_host = P.receive_side(lists_i, lists_v, L, w_host, lr=0.1)
    for p in pairs:
        p.close()
    return rep


def test_cfg1_outlier_tensor_5_iterations(P):
    wl = I.workload("cfg1")
    rep = _run_workload(P, wl, wl.iterations)
    assert rep.worker_iterations == 20
    assert rep.full_select == 0


def test_resnet50_shapes_two_workers(P):
    wl = I.workload("resnet50")
    rep = _run_workload(P, wl, 3, workers=2)
    assert rep.full_select == 0


def test_resnet50_shapes_with_clipping(P):
    wl = I.workload("resnet50")
    wl.clip_threshold = 1.0
    _run_workload(P, wl, 2, workers=1, receive=False)


def test_lstm_small_row_sparse_embedding(P):
    wl = I.workload("lstm_small")
    _run_workload(P, wl, 4)


def test_deepspeech_small_warmup_schedule(P):
    wl = I.workload("deepspeech_small")
    stages = [0.75, 0.9375, 0.984375, 0.996, 0.999]
    _run_workload(P, wl, 10, workers=2, schedule=lambda t: stages[min(t // 2, 4)])


def test_nesterov_variant_deepspeech_small(P):
    """Algorithm 5 (the paper trains its speech model with Nesterov momentum and clipping)."""
    wl = I.workload("deepspeech_small")
    wl.sparsity = 0.999
    _run_workload(P, wl, 4, workers=2, nesterov=True)


def test_nesterov_variant_resnet50_no_clip(P):
    wl = I.workload("resnet50")
    _run_workload(P, wl, 2, workers=1, receive=False, nesterov=True)


def test_lstm_full_size_all_workers_with_receive_side(P):
    """The 66,034,000-value LSTM-shaped set at full size (15 M-element tensors, 58 parts each;
    a row-sparse embedding gradient whose zeros tie in masses): all 4 workers, 3 iterations,
    clipping on; every index, value and state word against the oracle, then the decoded sum
    of the 4 lists and the weights after the SGD step."""
    wl = I.workload("lstm")
    rep = _run_workload(P, wl, 3)
    assert rep.worker_iterations == 12
    assert rep.full_select == 0


def test_deepspeech_full_size_every_warmup_stage(P):
    """The 122,096,829-value DeepSpeech-shaped set at full size through the whole warm-up
    schedule of Sec. 4.1 (75 %, 93.75 %, 98.4375 %, 99.6 %, 99.9 %: 30.5 M down to 122 K
    entries sent), dgc_set_sparsity between the stages; two iterations at 75 % so that the
    deferred masking of the emission-from-v' path is applied by a following call of the same
    stage, one in each later stage; receive side included."""
    wl = I.workload("deepspeech")
    stages = [0.75, 0.75, 0.9375, 0.984375, 0.996, 0.999]
    rep = _run_workload(P, wl, len(stages), workers=1, schedule=lambda t: stages[t])
    assert rep.worker_iterations == 6
    assert rep.full_select == 0


@pytest.mark.parametrize("n", [1 << 16, 1 << 18, 1 << 20, 1 << 22, 1 << 24])
@pytest.mark.parametrize("sparsity", [0.99, 0.999, 0.9999])
def test_sweep_single_tensor(P, n, sparsity):
    wl = I.workload("sweep", n=n, sparsity=sparsity)
    rep = _run_workload(P, wl, 2, workers=1)
    assert rep.full_select == 0


@pytest.mark.parametrize("n", [1 << 26, 1 << 28])
@pytest.mark.parametrize("sparsity", [0.99, 0.999, 0.9999])
def test_sweep_largest_tensors(P, n, sparsity):
    """The two largest sizes of the single-tensor sweep at all three sparsities (2 iterations
    at 2^26, 1 at 2^28 where one oracle iteration takes several seconds)."""
    wl = I.workload("sweep", n=n, sparsity=sparsity)
    rep = _run_workload(P, wl, 1 if n == 1 << 28 else 2, workers=1, receive=False)
    assert rep.full_select == 0


@pytest.mark.parametrize("sparsity", [0.999, 0.99, 0.75, 0.0])
def test_edge_sizes(P, sparsity):
    numel = [1, 3, 4, 5, 31, 32, 33, 511, 512, 513, 4095, 4096, 4097, 8192, 8193, 70001,
             524288, 524289]
    wl = I.Workload("edge", [(n,) for n in numel], 4, 0.9, 1.0, sparsity, 3, "normal")
    _run_workload(P, wl, 3, workers=1)


def test_heavy_ties_and_zeros(P):
    """Quantised values: thousands of exact ties at the threshold; ties go to the lower index."""
    numel = [100000, 5000, 300000]
    pair = P.Pair(numel, 2, 0.5, 0.0, 0.99, seed=3)
    rep = P.ParityReport()
    rng = np.random.default_rng(5)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    for t in range(4):
        g = P.arena_with_padding_poison(L, off, numel)
        for o, n in zip(off, numel):
            g[o:o + n] = rng.integers(-3, 4, size=n).astype(np.float32) * np.float32(0.25)
        pair.step(g, rep)
    pair.close()


def test_all_zero_gradient_is_zero_filled_with_lowest_indices(P):
    numel = [20000, 100]
    pair = P.Pair(numel, 1, 0.9, 0.0, 0.999, seed=1)
    rep = P.ParityReport()
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    g = P.arena_with_padding_poison(L, off, numel)
    gi, gv, st = pair.step(g, rep)
    assert gi.tolist() == list(range(20)) + [int(off[1])]
    assert not gv.any()
    # no selection at all: the sampled tensor's list is completed with zeros (flag 16), the
    # small one is its own sample; nothing takes the slow full-selection path
    assert st.flags & 16 and not st.flags & 2 and st.full_select_last == 0
    pair.close()


@pytest.mark.parametrize("sparsity", [0.999, 0.99, 0.75])
def test_fewer_nonzeros_than_k_zero_fill_matches_oracle(P, sparsity):
    """Tensors with fewer non-zero entries than k (an almost unused embedding, a frozen layer):
    all non-zeros plus the lowest-index zeros, over several iterations with momentum so that u
    is non-zero where v was sent.  Covers one-part, multi-part and (at 99 %) multi-block-selected
    tensors, a ragged last segment, immediate (99.9 %) and deferred (99 %) masking, emission
    from v' itself (75 %), and zeros of either sign."""
    numel = [700001, 1 << 22, 40000, 300, 1 << 19]
    pair = P.Pair(numel, 1, 0.9, 0.0, sparsity, seed=4)
    rep = P.ParityReport()
    rng = np.random.default_rng(21)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    # start from negative zeros in part of the state: they must be sent as they are
    u0 = np.zeros(L, np.float32)
    v0 = np.zeros(L, np.float32)
    v0[off[0]:off[0] + 1000] = np.float32(-0.0)
    u0[off[0]:off[0] + 1000] = np.float32(-0.0)
    pair.gpu.write(u0, v0)
    pair.cpu.u[:], pair.cpu.v[:] = u0, v0
    nonzeros = [0, 37, 5, 0, 300]            # per tensor and iteration: all below k
    for t in range(4):
        g = P.arena_with_padding_poison(L, off, numel)
        for j, (o, n) in enumerate(zip(off, numel)):
            if j == 0 and t < 2:
                g[o:o + 1000] = np.float32(-0.0)
            pos = rng.choice(n, size=nonzeros[j], replace=False)
            g[o + pos] = rng.standard_normal(nonzeros[j]).astype(np.float32)
        if t == 3:
            g[off[2]:off[2] + numel[2]] = rng.standard_normal(numel[2]).astype(np.float32)
        gi, gv, st = pair.step(g, rep)
        assert st.flags & 16 and st.full_select_last == 0, (t, st.flags, st.full_select_last)
        if t == 0:
            # tensor 0: nothing non-zero, so its k lowest indices, the first 1000 of them -0.0
            k0 = int(pair.gpu.k[0])
            assert gi[:k0].tolist() == list(range(int(off[0]), int(off[0]) + k0))
            assert (gv[:min(k0, 1000)].view(np.uint32) == 0x80000000).all()
    pair.close()


@pytest.mark.parametrize("sparsity", [0.999, 0.99, 0.75])
def test_few_distinct_magnitudes_tie_fill_matches_oracle(P, sparsity):
    """Sign-like gradients: every entry of a tensor has one of a handful of magnitudes, so the
    k-th largest |v| is shared by far more than k entries.  Those ties are counted, not listed
    as candidates, and the lowest indices complete the list; no tensor may take the slow
    full-selection path."""
    numel = [700001, 1 << 22, 40000, 5000]
    pair = P.Pair(numel, 1, 0.5, 0.0, sparsity, seed=9)
    rep = P.ParityReport()
    rng = np.random.default_rng(33)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    for t in range(4):
        g = P.arena_with_padding_poison(L, off, numel)
        for j, (o, n) in enumerate(zip(off, numel)):
            sign = rng.integers(0, 2, size=n).astype(np.float32) * 2 - 1
            if j == 1:
                sign *= rng.integers(0, 3, size=n).astype(np.float32)     # magnitudes 0, 1, 2
            g[o:o + n] = sign * np.float32(0.25)
        gi, gv, st = pair.step(g, rep)
        assert st.full_select_last == 0 and not st.flags & 2, (t, st.flags)
        if t == 0:
            assert st.flags & 16
            k0 = int(pair.gpu.k[0])
            assert gi[:k0].tolist() == list(range(int(off[0]), int(off[0]) + k0))
    pair.close()


def test_nonzeros_concentrated_in_one_sampling_block(P):
    """A large tensor whose non-zero entries all lie in its first twentieth: the sampling block
    of that region holds every one of the sample's largest keys, far more than the shortened
    list it keeps for the merge, so the merge must notice that the lists do not add up and
    select from the whole sample instead.  Bit for bit against the oracle, no full selection."""
    numel = [3_000_000, 70001]
    pair = P.Pair(numel, 1, 0.9, 0.0, 0.999, seed=21)
    rep = P.ParityReport()
    rng = np.random.default_rng(77)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    for t in range(3):
        g = P.arena_with_padding_poison(L, off, numel)
        g[off[0]:off[0] + 150_000] = rng.standard_normal(150_000).astype(np.float32)
        g[off[1]:off[1] + numel[1]] = rng.standard_normal(numel[1]).astype(np.float32)
        _, _, st = pair.step(g, rep)
        assert st.full_select_last == 0 and not st.flags & 2, (t, st.flags)
    pair.close()


def test_forced_full_selection_path_matches(P):
    """debug_sample_rank = 1 proposes the sample maximum: too few pass, every sampled tensor
    falls back to selecting from the whole of v; the result must not change."""
    numel = [50000, 9000, 1200000, 64]
    pair = P.Pair(numel, 1, 0.9, 0.0, 0.99, seed=2, debug_sample_rank=1)
    rep = P.ParityReport()
    rng = np.random.default_rng(8)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    for t in range(3):
        g = P.arena_with_padding_poison(L, off, numel)
        for o, n in zip(off, numel):
            g[o:o + n] = rng.standard_normal(n).astype(np.float32)
        _, _, st = pair.step(g, rep)
        # at 99% sparsity k_j exceeds n_j / sample size for all three sampled tensors
        assert st.full_select_last == 3 and st.flags & 8
    pair.close()


def test_result_independent_of_sampling_seed_and_ratio(P):
    numel = [300000, 40000]
    rng = np.random.default_rng(12)
    grads = []
    outs = []
    for seed, ratio in ((1, 0.01), (2, 0.001), (3, 0.005)):
        pair = P.Pair(numel, 1, 0.9, 0.0, 0.999, seed=seed, sample_ratio=ratio)
        off, L = pair.gpu.arena_offset, pair.gpu.arena_len
        if not grads:
            for t in range(3):
                g = P.arena_with_padding_poison(L, off, numel)
                for o, n in zip(off, numel):
                    g[o:o + n] = rng.standard_t(3, n).astype(np.float32)
                grads.append(g)
        rep = P.ParityReport()
        res = [pair.step(g, rep)[0].copy() for g in grads]
        outs.append(res)
        pair.close()
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert np.array_equal(a, b)


def test_special_values_inf_and_nan_are_selected_first(P):
    numel = [10000]
    pair = P.Pair(numel, 1, 0.9, 0.0, 0.999, seed=4)     # k = 10
    rep = P.ParityReport()
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    rng = np.random.default_rng(1)
    g = P.arena_with_padding_poison(L, off, numel)
    g[:10000] = rng.standard_normal(10000).astype(np.float32)
    g[5000] = np.inf
    g[5001] = -np.inf
    gi, gv, _ = pair.step(g, rep)
    assert {5000, 5001} <= set(gi.tolist())
    # NaN: its payload may differ between CPU and GPU arithmetic, so only the GPU's choice
    # is checked here: the NaN entry has the largest key and is sent
    g[:10000] = rng.standard_normal(10000).astype(np.float32)
    g[77] = np.nan
    pair.gpu.compress(torch.from_numpy(g).cuda(), pair.out_idx, pair.out_val)
    sel = pair.out_idx.cpu().numpy()
    assert 77 in sel.tolist() and np.isnan(pair.out_val.cpu().numpy()[sel.tolist().index(77)])
    pair.close()


def test_deterministic_across_runs(P):
    wl = I.workload("sweep", n=1 << 21)
    outs = []
    for _ in range(2):
        pair = P.Pair(wl.numel, 1, 0.9, 0.5, 0.999, seed=9)
        off, L = pair.gpu.arena_offset, pair.gpu.arena_len
        res = []
        for t in range(3):
            g = np.zeros(L, np.float32)
            I.fill(wl, g, off, 0, t)
            gd = torch.from_numpy(g).cuda()
            pair.gpu.compress(gd, pair.out_idx, pair.out_val)
            u, v = pair.gpu.read()
            res.append((pair.out_idx.cpu().numpy().copy(), pair.out_val.cpu().numpy().copy(), u, v,
                        pair.gpu.status().grad_norm))
        outs.append(res)
        pair.close()
    for a, b in zip(*outs):
        for x, y in zip(a[:4], b[:4]):
            assert x.tobytes() == y.tobytes()
        assert a[4] == b[4]


def test_checkpoint_resume_is_bit_identical(P):
    from paper_1712_01887_b200 import binding as B
    numel = [100000, 777]
    rng = np.random.default_rng(3)
    a = B.State(numel, 1, 0.9, 0.0, 0.999, seed=5)
    L = a.arena_len
    gs = [torch.from_numpy(rng.standard_normal(L).astype(np.float32)).cuda() for _ in range(3)]
    oi = torch.empty(a.max_nnz, dtype=torch.int32, device="cuda")
    ov = torch.empty(a.max_nnz, dtype=torch.float32, device="cuda")
    a.compress(gs[0], oi, ov)
    a.compress(gs[1], oi, ov)
    u, v = a.read()
    b = B.State(numel, 1, 0.9, 0.0, 0.999, seed=5)
    b.write(u, v)
    a.compress(gs[2], oi, ov)
    oi2, ov2 = torch.empty_like(oi), torch.empty_like(ov)
    b.compress(gs[2], oi2, ov2)
    assert torch.equal(oi, oi2) and torch.equal(ov.view(torch.int32), ov2.view(torch.int32))
    ua, va = a.read()
    ub, vb = b.read()
    assert ua.tobytes() == ub.tobytes() and va.tobytes() == vb.tobytes()
    a.close()
    b.close()


@pytest.mark.parametrize("workload,nesterov", [("lstm_small", False), ("resnet50", True)])
def test_clipping_per_tensor_matches_oracle(P, workload, nesterov):
    """dgc_config.clip_scope = 1: every tensor clipped by its own L2 norm (the oracle's
    compress_clip_per_tensor).  Norms within 1e-6, coefficients bit for bit (the oracle is re-run
    with the GPU's coefficients should a last bit differ), then indices, values and state bit
    for bit; the gradients are scaled so that some tensors exceed the threshold and some do not."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    wl = I.workload(workload)
    clip, N = 1.0, 4
    st = B.State(wl.numel, N, wl.momentum, clip, wl.sparsity, seed=11, nesterov=nesterov,
                 clip_scope=1)
    L, off = st.arena_len, st.arena_offset
    cpu = O.Worker(off, wl.numel, L, N, wl.momentum, clip, wl.sparsity, nesterov=nesterov)
    oi = torch.empty(st.max_nnz, dtype=torch.int32, device="cuda")
    ov = torch.empty(st.max_nnz, dtype=torch.float32, device="cuda")
    scale = np.float32(40.0 if workload == "resnet50" else 3.0)
    overrides, clipped, kept = 0, 0, 0
    for t in range(3):
        g = P.arena_with_padding_poison(L, off, wl.numel)
        I.fill(wl, g, off, worker=2, iteration=t)
        for o, n in zip(off, wl.numel):
            g[o:o + n] *= scale
        st.compress(torch.from_numpy(g).cuda(), oi, ov)
        norms, coefs = st.clip()
        status = st.status()
        snap = (cpu.u.copy(), cpu.v.copy())
        r = cpu.compress_clip_per_tensor(g)
        assert np.all(np.abs(norms - r.norm) <= 1e-6 * np.maximum(r.norm, 1e-300))
        if coefs.tobytes() != r.coef.tobytes():
            cpu.u[:], cpu.v[:] = snap
            r = cpu.compress_clip_per_tensor(g, coef_override=coefs)
            overrides += 1
        assert oi.cpu().numpy().tobytes() == r.idx.tobytes(), t
        assert ov.cpu().numpy().tobytes() == r.val.tobytes(), t
        u, v = st.read()
        assert u.tobytes() == cpu.u.tobytes() and v.tobytes() == cpu.v.tobytes()
        assert abs(status.grad_norm - np.sqrt((norms ** 2).sum())) <= 1e-9 * status.grad_norm
        assert status.clip_coef == coefs.min()
        clipped += int((coefs < 1).sum())
        kept += int((coefs == 1).sum())
    assert clipped > 0 and kept > 0 and overrides <= 1
    st.close()
    with pytest.raises(B.DgcError):
        B.State([100], 1, 0.9, 1.0, 0.9, clip_scope=2)


def test_get_clip_reports_the_whole_set_norm_when_clipping_by_it(P):
    """dgc_get_clip with the default scope: every tensor reports the one norm and coefficient
    of the whole set (what dgc_get_status reports); with clipping off, 0 and 1."""
    from paper_1712_01887_b200 import binding as B
    numel = [5000, 70001, 64]
    rng = np.random.default_rng(4)
    for clip in (1.0, 0.0):
        st = B.State(numel, 4, 0.9, clip, 0.99, seed=1)
        L = st.arena_len
        oi = torch.empty(st.max_nnz, dtype=torch.int32, device="cuda")
        ov = torch.empty(st.max_nnz, dtype=torch.float32, device="cuda")
        st.compress(torch.from_numpy(rng.standard_normal(L).astype(np.float32)).cuda(), oi, ov)
        norms, coefs = st.clip()
        status = st.status()
        if clip > 0:
            assert status.grad_norm > 0.5 and status.clip_coef < 1.0
            assert (norms == status.grad_norm).all() and (coefs == status.clip_coef).all()
        else:
            assert not norms.any() and (coefs == 1.0).all()
        st.close()


def test_compress_host_matches_device_path(P):
    from paper_1712_01887_b200 import binding as B
    numel = [200000, 3000]
    rng = np.random.default_rng(6)
    a = B.State(numel, 4, 0.9, 1.0, 0.999, seed=5)
    b = B.State(numel, 4, 0.9, 1.0, 0.999, seed=5)
    L = a.arena_len
    for t in range(2):
        gh = torch.from_numpy(rng.standard_normal(L).astype(np.float32)).pin_memory()
        oi = torch.empty(a.max_nnz, dtype=torch.int32, device="cuda")
        ov = torch.empty(a.max_nnz, dtype=torch.float32, device="cuda")
        a.compress(gh.cuda(), oi, ov)
        hi = torch.empty(a.max_nnz, dtype=torch.int32).pin_memory()
        hv = torch.empty(a.max_nnz, dtype=torch.float32).pin_memory()
        b.compress_host(gh, hi, hv)
        assert torch.equal(oi.cpu(), hi) and torch.equal(ov.cpu().view(torch.int32), hv.view(torch.int32))
    a.close()
    b.close()


def test_compress_host_batch_matches_per_worker_calls(P):
    """dgc_compress_host_batch (what the benchmark's end-to-end leg calls): host gradients of
    several workers in, host lists out, bit for bit what dgc_compress gives each worker on the
    device, over three iterations (state carried); more workers than internal streams."""
    from paper_1712_01887_b200 import binding as B
    numel = [300000, 70001, 64, 9000]
    NW = 10
    rng = np.random.default_rng(16)
    dev_states = [B.State(numel, NW, 0.9, 1.0, 0.999, seed=w) for w in range(NW)]
    host_states = [B.State(numel, NW, 0.9, 1.0, 0.999, seed=w) for w in range(NW)]
    L, nnz = dev_states[0].arena_len, dev_states[0].max_nnz
    hi = [torch.empty(nnz, dtype=torch.int32).pin_memory() for _ in range(NW)]
    hv = [torch.empty(nnz, dtype=torch.float32).pin_memory() for _ in range(NW)]
    for t in range(3):
        gh = [torch.from_numpy(rng.standard_normal(L).astype(np.float32)).pin_memory()
              for _ in range(NW)]
        B.compress_host_batch(host_states, gh, hi, hv)
        for w in range(NW):
            oi = torch.empty(nnz, dtype=torch.int32, device="cuda")
            ov = torch.empty(nnz, dtype=torch.float32, device="cuda")
            dev_states[w].compress(gh[w].cuda(), oi, ov)
            assert torch.equal(oi.cpu(), hi[w]), (t, w)
            assert torch.equal(ov.cpu().view(torch.int32), hv[w].view(torch.int32)), (t, w)
    ua, va = dev_states[3].read()
    ub, vb = host_states[3].read()
    assert ua.tobytes() == ub.tobytes() and va.tobytes() == vb.tobytes()
    with pytest.raises(B.DgcError):                      # the same state twice
        B.compress_host_batch([host_states[0], host_states[0]], gh[:2], hi[:2], hv[:2])
    for st in dev_states + host_states:
        st.close()


def test_abi_errors(P):
    from paper_1712_01887_b200 import binding as B
    with pytest.raises(B.DgcError) as e:
        B.State([0], 1, 0.9, 0.0, 0.999)
    assert e.value.code == B.EINVAL
    with pytest.raises(B.DgcError):
        B.State([10], 1, 0.9, 0.0, 1.0)
    st = B.State([5000], 1, 0.9, 0.0, 0.99)
    g = torch.zeros(st.arena_len, device="cuda")
    small_i = torch.empty(st.max_nnz - 1, dtype=torch.int32, device="cuda")
    small_v = torch.empty(st.max_nnz - 1, dtype=torch.float32, device="cuda")
    with pytest.raises(B.DgcError) as e:
        st.compress(g, small_i, small_v)
    assert e.value.code == B.ECAPACITY
    with pytest.raises(B.DgcError) as e:
        st.set_sparsity(1.5)
    assert e.value.code == B.EINVAL
    st.close()
    with pytest.raises(B.DgcError) as e:
        st.set_sparsity(0.5)
    assert e.value.code == B.ESTATE


def test_decode_edge_cases(P):
    rng = np.random.default_rng(17)
    for L, N, density in ((1, 1, 1.0), (4095, 3, 0.01), (4096, 2, 0.5), (4097, 5, 0.001),
                          (1 << 20, 8, 0.001), (100003, 64, 0.01), (50000, 4, 1.0), (9000, 2, 0.0)):
        idx, val = [], []
        for w in range(N):
            k = int(round(L * density)) if w % 2 == 0 else int(L * density / 2)
            i = np.sort(rng.choice(L, size=min(k, L), replace=False)).astype(np.int32)
            idx.append(i)
            val.append(rng.standard_normal(i.size).astype(np.float32))
        w0 = rng.standard_normal(L).astype(np.float32)
        P.receive_side(idx, val, L, w0, lr=0.05)


def test_decode_skips_and_reports_indices_that_break_the_precondition(P):
    """A list with an index outside [0, dense_len), a repeated one or one out of order must
    not make the receive side write outside its output or workspace.  The buffers are
    allocated with slack beyond the dense_len that is passed, the bad indices point into that
    slack, so the test cannot fault whatever the kernels do (negative and huge indices take
    the same guards: tile numbers are clamped, tile offsets compared as unsigned); the slack must stay untouched, the good
    entries must still be summed, and dgc_decode_rejected must count the bad pairs."""
    from paper_1712_01887_b200 import binding as B
    dense_len, slack = 3 * 4096 + 100, 4 * 4096
    N = 3
    good = [np.array([5, 4096, 4097, 9000, dense_len - 1], np.int32),
            np.array([5, 100, 9000], np.int32),
            np.array([0, 12000], np.int32)]
    vals = [np.arange(1, a.size + 1, dtype=np.float32) * (w + 1) for w, a in enumerate(good)]
    ref = np.zeros(dense_len, np.float32)
    for a, v in zip(good, vals):
        np.add.at(ref, a, v)

    def run(lists_i, lists_v, fn):
        di = [torch.from_numpy(a).cuda() for a in lists_i]
        dv = [torch.from_numpy(v).cuda() for v in lists_v]
        out = torch.full((dense_len + slack,), 7.0, dtype=torch.float32, device="cuda")
        ws_bytes = B.decode_workspace_bytes(N, dense_len)
        ws = torch.full((ws_bytes + 4096,), 0x5A, dtype=torch.uint8, device="cuda")
        fn(di, dv, out[:dense_len], ws[:ws_bytes])
        torch.cuda.synchronize()
        assert bool((out[dense_len:] == 7.0).all()), "wrote past dense_len"
        assert bool((ws[ws_bytes:] == 0x5A).all()), "wrote past the workspace"
        return out[:dense_len].cpu().numpy(), B.decode_rejected(N, dense_len, ws[:ws_bytes])

    dense = lambda di, dv, out, ws: B.decode_accumulate(di, dv, out, ws)      # noqa: E731
    got, rej = run(good, vals, dense)
    assert got.tobytes() == ref.tobytes() and rej == 0
    # (a) indices beyond dense_len at the end of a list (ascending, so the rest is intact)
    bad_i = [np.concatenate([good[0], [dense_len, dense_len + 5000]]).astype(np.int32), good[1],
             good[2]]
    bad_v = [np.concatenate([vals[0], [99.0, 98.0]]).astype(np.float32), vals[1], vals[2]]
    got, rej = run(bad_i, bad_v, dense)
    assert got.tobytes() == ref.tobytes() and rej == 2
    # (b) an index listed twice by one worker: reported (which of the two values lands first is
    #     unspecified, so only the other entries are compared)
    bad_i = [good[0], np.array([5, 100, 100, 9000], np.int32), good[2]]
    bad_v = [vals[0], np.array([1.0, 2.0, 2.5, 3.0], np.float32) * 2, vals[2]]
    got, rej = run(bad_i, bad_v, dense)
    keep = np.ones(dense_len, bool)
    keep[100] = False
    assert got[keep].tobytes() == ref[keep].tobytes() and rej == 1
    # (c) out of order (an unwritten slot in the middle): no fault, no stray write, reported;
    #     the sums of the affected list are unspecified, the other workers' entries are intact
    bad_i = [good[0], good[1], np.array([12000, 0, 7], np.int32)]
    bad_v = [vals[0], vals[1], np.array([1.0, 2.0, 3.0], np.float32)]
    got, rej = run(bad_i, bad_v, dense)
    assert rej >= 1
    only01 = np.zeros(dense_len, np.float32)
    for a, v in zip(good[:2], vals[:2]):
        np.add.at(only01, a, v)
    untouched = np.ones(dense_len, bool)
    untouched[[12000, 0, 7]] = False
    assert got[untouched].tobytes() == only01[untouched].tobytes()
    # the fused forms take the same guarded path
    w0 = np.linspace(-1, 1, dense_len + slack).astype(np.float32)

    def sparse_sgd(di, dv, out, ws):
        out.copy_(torch.from_numpy(w0[:dense_len]).cuda())
        B.decode_apply_sgd(di, dv, out, 0.5, ws)
    bad_i = [np.concatenate([good[0], [dense_len + 1]]).astype(np.int32), good[1], good[2]]
    bad_v = [np.concatenate([vals[0], [99.0]]).astype(np.float32), vals[1], vals[2]]
    got, rej = run(bad_i, bad_v, sparse_sgd)
    assert rej == 1
    assert got.tobytes() == (w0[:dense_len] - np.float32(0.5) * ref).astype(np.float32).tobytes()


def test_runlength_wire_format_matches_oracle(P):
    """Sec. 3.1 encode(): values + 16-bit zero run lengths, against the oracle bit for bit;
    then back through decode and the dense sum."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    rng = np.random.default_rng(31)
    cases = [(1000, 0), (1000, 1000), (70000, 2), (5_000_000, 5000), (300_000_000, 9),
             (40_000_000, 3_000_000)]
    for L, k in cases:
        if k == 0:
            idx = np.zeros(0, np.int32)
        elif k < 100:
            idx = np.sort(rng.choice(L, size=k, replace=False)).astype(np.int32)
        else:
            idx = np.sort(rng.choice(L, size=k, replace=False)).astype(np.int32)
        val = rng.standard_normal(idx.size).astype(np.float32)
        cap = B.runlength_max_entries(idx.size, L)
        ref_runs, ref_vals = O.encode_runlength(idx, val, cap)
        di, dv = torch.from_numpy(idx).cuda(), torch.from_numpy(val).cuda()
        runs, values = B.encode_runlength(di, dv, L)
        assert runs.cpu().numpy().tobytes() == ref_runs.tobytes(), (L, k)
        assert values.cpu().numpy().tobytes() == ref_vals.tobytes(), (L, k)
        ridx, rval = O.decode_runlength(ref_runs, ref_vals)
        gi, gv, end = B.decode_runlength(runs, values)
        assert gi.cpu().numpy().tobytes() == ridx.tobytes()
        assert gv.cpu().numpy().tobytes() == rval.tobytes()
        assert end == (int(idx[-1]) + 1 if idx.size else 0)


def test_runlength_of_compressed_resnet50_gradient(P):
    """The lists dgc_compress emits, encoded: size against the paper's Table 3 context
    (ResNet-50: 97.49 MB -> 0.35 MB, 277x) and decoded back into the same dense sum."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    wl = I.workload("resnet50")
    st = B.State(wl.numel, 8, 0.9, 0.0, 0.999, seed=1)
    L, off = st.arena_len, st.arena_offset
    g = np.zeros(L, np.float32)
    I.fill(wl, g, off, 0, 0)
    oi = torch.empty(st.max_nnz, dtype=torch.int32, device="cuda")
    ov = torch.empty(st.max_nnz, dtype=torch.float32, device="cuda")
    st.compress(torch.from_numpy(g).cuda(), oi, ov)
    runs, values = B.encode_runlength(oi, ov, L)
    ref_runs, ref_vals = O.encode_runlength(oi.cpu().numpy(), ov.cpu().numpy(),
                                            B.runlength_max_entries(st.max_nnz, L))
    assert runs.cpu().numpy().tobytes() == ref_runs.tobytes()
    assert values.cpu().numpy().tobytes() == ref_vals.tobytes()
    ratio = wl.total * 4 / (runs.numel() * 6)
    assert 600 < ratio < 667          # 25,670 entries of 6 bytes for 102 MB: about 664x
    gi, gv, _ = B.decode_runlength(runs, values)
    dense_a = torch.empty(L, dtype=torch.float32, device="cuda")
    dense_b = torch.empty(L, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.decode_workspace_bytes(1, L), dtype=torch.uint8, device="cuda")
    B.decode_accumulate([oi], [ov], dense_a, ws)
    B.decode_accumulate([gi], [gv], dense_b, ws)
    assert torch.equal(dense_a.view(torch.int32), dense_b.view(torch.int32))
    st.close()


def test_workers_on_their_own_streams_like_the_benchmark(P):
    """bench.py issues the simulated workers' compress calls on one CUDA stream per worker
    and joins them before the decode.  Same launch configuration here, on the ResNet-50-shaped
    set with all 8 workers: every worker must still match its oracle bit for bit."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    wl = I.workload("resnet50")
    NW, NS, T = 8, 8, 2
    states = [B.State(wl.numel, wl.num_workers, wl.momentum, wl.clip_threshold, wl.sparsity,
                      seed=I.BASE_SEED + w) for w in range(NW)]
    L, off = states[0].arena_len, states[0].arena_offset
    oracles = [O.Worker(off, wl.numel, L, wl.num_workers, wl.momentum, wl.clip_threshold,
                        wl.sparsity) for _ in range(NW)]
    nnz = states[0].max_nnz
    main = torch.cuda.current_stream()
    side = [torch.cuda.Stream() for _ in range(NS)]
    out_i = [torch.empty(nnz, dtype=torch.int32, device="cuda") for _ in range(NW)]
    out_v = [torch.empty(nnz, dtype=torch.float32, device="cuda") for _ in range(NW)]
    dense = torch.empty(L, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.decode_workspace_bytes(NW, L), dtype=torch.uint8, device="cuda")
    weights = torch.zeros(L, dtype=torch.float32, device="cuda")
    w_ref = np.zeros(L, np.float32)
    for t in range(T):
        hosts = []
        for w in range(NW):
            g = np.zeros(L, np.float32)
            I.fill(wl, g, off, worker=w, iteration=t)
            hosts.append(g)
        dev = [torch.from_numpy(g).cuda() for g in hosts]
        torch.cuda.synchronize()
        fork = torch.cuda.Event()
        fork.record(main)
        for s_ in side:
            s_.wait_event(fork)
        for w in range(NW):
            states[w].compress(dev[w], out_i[w], out_v[w], stream=side[w % NS])
        for s_ in side:
            e = torch.cuda.Event()
            e.record(s_)
            main.wait_event(e)
        B.decode_accumulate(out_i, out_v, dense, ws)
        B.apply_sgd(weights, dense, 0.1)
        torch.cuda.synchronize()
        res = [oracles[w].compress(hosts[w]) for w in range(NW)]
        for w in range(NW):
            assert out_i[w].cpu().numpy().tobytes() == res[w].idx.tobytes(), (t, w)
            assert out_v[w].cpu().numpy().tobytes() == res[w].val.tobytes(), (t, w)
        ref = O.decode_accumulate([r.idx for r in res], [r.val for r in res], L)
        O.apply_sgd(w_ref, ref, 0.1)
        assert dense.cpu().numpy().tobytes() == ref.tobytes()
        assert weights.cpu().numpy().tobytes() == w_ref.tobytes()
    for w in (0, NW - 1):
        u, v = states[w].read()
        assert u.tobytes() == oracles[w].u.tobytes() and v.tobytes() == oracles[w].v.tobytes()
    for st in states:
        st.close()


@pytest.mark.parametrize("sparsity", [0.75, 0.9375, 0.99])
def test_deferred_masking_without_reading_state_between_iterations(P, sparsity):
    """Below 99.8 % sparsity the library does not zero u and v at the sent entries right away:
    it records them as bits and the next call's kernels zero them in registers.  Reading the
    state flushes that, so here nothing is read until the end: five iterations compared on
    indices and values only (with exact ties in the data), then the final state."""
    numel = [300000, 70001, 513, 1 << 20]
    pair = P.Pair(numel, 2, 0.9, 1.0, sparsity, seed=11)
    rep = P.ParityReport()
    rng = np.random.default_rng(23)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    for t in range(5):
        g = P.arena_with_padding_poison(L, off, numel)
        for j, (o, n) in enumerate(zip(off, numel)):
            if j == 1:      # quantised: many ties at the threshold
                g[o:o + n] = rng.integers(-3, 4, size=n).astype(np.float32) * np.float32(0.125)
            else:
                g[o:o + n] = rng.standard_normal(n).astype(np.float32)
        pair.step(g, rep, check_state=False)
    u, v = pair.gpu.read()
    assert u.tobytes() == pair.cpu.u.tobytes() and v.tobytes() == pair.cpu.v.tobytes()
    # and once more after the flush: the next call must start from the flushed state
    g = P.arena_with_padding_poison(L, off, numel)
    for o, n in zip(off, numel):
        g[o:o + n] = rng.standard_normal(n).astype(np.float32)
    pair.step(g, rep, check_state=True)
    pair.close()


@pytest.mark.parametrize("sparsity,numel,iters,ratio", [
    (0.999, [100000, 8192, 64, 70001, 600000, 1 << 21, 1, 3], 12, 0.01),
    (0.99, [1 << 22, 300000, 5000, 9000], 4, 0.01),     # the 2^22 tensor takes the multi-block path
    (0.75, [200000, 1000], 3, 0.01),
    (0.999, [(1 << 23) + 5, 70001], 3, 0.01),           # 83,887 draws: more than 32 sampling blocks
    (0.99, [1 << 23, 513], 2, 0.01),                    # the same with sample rank 839 (> one block)
    (0.999, [1 << 22, 100000, 2000], 4, 0.001),         # the paper's smallest sample: 0.1 %
])
def test_paper_literal_sampled_selection_matches_oracle(P, sparsity, numel, iters, ratio):
    """select_mode = 1: Sec. 5 as stated (ceil(ratio n) uniform draws per tensor, threshold =
    the sample's ceil(S (1 - s))-th largest |v|, strict compare, exact top-k only when more
    than 2k pass; variable count).  The oracle takes the positions from the same counter-based
    generator; indices, values, per-tensor counts and state must agree bit for bit, over
    several iterations and all outcomes (fewer than k, more than k, more than 2k)."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    seed = 77
    st = B.State(numel, 4, 0.9, 1.0, sparsity, seed=seed, select_mode=1, sample_ratio=ratio)
    L, off = st.arena_len, st.arena_offset
    cpu = O.Worker(off, numel, L, 4, 0.9, 1.0, sparsity)
    assert st.max_nnz == int(np.minimum(np.asarray(numel), 2 * cpu.k).sum())
    oi = torch.empty(st.max_nnz, dtype=torch.int32, device="cuda")
    ov = torch.empty(st.max_nnz, dtype=torch.float32, device="cuda")
    rng = np.random.default_rng(3)
    kinds = set()
    for t in range(iters):
        g = P.arena_with_padding_poison(L, off, numel)
        for o, n in zip(off, numel):
            g[o:o + n] = rng.standard_normal(n).astype(np.float32)
        st.compress(torch.from_numpy(g).cuda(), oi, ov)
        status = st.status()
        total, per = st.nnz()
        snap = (cpu.u.copy(), cpu.v.copy())
        r, nnz = O.compress_sampled(cpu, g, seed=seed, iteration=t, sample_ratio=ratio)
        if np.float32(status.clip_coef).tobytes() != np.float32(r.coef).tobytes():
            cpu.u[:], cpu.v[:] = snap
            r, nnz = O.compress_sampled(cpu, g, seed=seed, iteration=t, sample_ratio=ratio,
                                        coef_override=status.clip_coef)
        assert per.tolist() == nnz.tolist(), (t, per, nnz)
        assert total == r.idx.size
        assert oi[:total].cpu().numpy().tobytes() == r.idx.tobytes()
        assert ov[:total].cpu().numpy().tobytes() == r.val.tobytes()
        u, v = st.read()
        assert u.tobytes() == cpu.u.tobytes() and v.tobytes() == cpu.v.tobytes()
        for c, k in zip(nnz, cpu.k):
            kinds.add("k" if c == k else ("fewer" if c < k else "more"))
    if sparsity == 0.999 and iters >= 12:
        assert {"fewer", "more", "k"} <= kinds
    st.close()


def test_sparsity_lowered_after_creation_reallocates_scratch(P):
    """dgc_set_sparsity towards a lower sparsity needs larger candidate lists than the state
    was created with (and switches between immediate and deferred masking)."""
    numel = [400000, 70001, 2000]
    pair = P.Pair(numel, 2, 0.9, 1.0, 0.9999, seed=5)
    rep = P.ParityReport()
    rng = np.random.default_rng(29)
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    for s in (0.9999, 0.99, 0.5, 0.999, 0.0, 0.9):
        pair.set_sparsity(s)
        for t in range(2):
            g = P.arena_with_padding_poison(L, off, numel)
            for o, n in zip(off, numel):
                g[o:o + n] = rng.standard_normal(n).astype(np.float32)
            pair.step(g, rep, check_state=(t == 1))
    pair.close()


@pytest.mark.parametrize("clip,T", [(1.0, 3), (0.0, 10)])
def test_compress_batch_matches_oracle_per_worker(P, clip, T):
    """dgc_compress_batch (what bench.py times): all 8 workers of the ResNet-50-shaped set in
    one call; every worker bit for bit against its oracle, then the one-pass receive side.
    Once with clipping on (so that the norm kernels run ahead too), and once in the
    benchmark's own configuration (clipping off) for the 10 iterations the workload states."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    wl = I.workload("resnet50")
    NW = 8
    states = [B.State(wl.numel, NW, wl.momentum, clip, wl.sparsity, seed=I.BASE_SEED + w)
              for w in range(NW)]
    L, off = states[0].arena_len, states[0].arena_offset
    oracles = [O.Worker(off, wl.numel, L, NW, wl.momentum, clip, wl.sparsity) for _ in range(NW)]
    nnz = states[0].max_nnz
    out_i = [torch.empty(nnz, dtype=torch.int32, device="cuda") for _ in range(NW)]
    out_v = [torch.empty(nnz, dtype=torch.float32, device="cuda") for _ in range(NW)]
    dense = torch.empty(L, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.decode_workspace_bytes(NW, L), dtype=torch.uint8, device="cuda")
    weights = torch.zeros(L, dtype=torch.float32, device="cuda")
    w_ref = np.zeros(L, np.float32)
    overrides = 0
    for t in range(T):
        hosts = []
        for w in range(NW):
            g = np.zeros(L, np.float32)
            I.fill(wl, g, off, worker=w, iteration=t)
            g *= np.float32(300.0)               # norm well above the clip threshold
            hosts.append(g)
        dev = [torch.from_numpy(g).cuda() for g in hosts]
        B.compress_batch(states, dev, out_i, out_v)
        B.decode_accumulate_sgd(out_i, out_v, dense, weights, 0.1, ws)
        torch.cuda.synchronize()
        res = []
        for w in range(NW):
            st = states[w].status()
            snap = (oracles[w].u.copy(), oracles[w].v.copy())
            r = oracles[w].compress(hosts[w])
            if clip > 0:
                assert abs(st.grad_norm - r.norm) <= 1e-6 * r.norm and r.coef < 1.0
            if np.float32(st.clip_coef).tobytes() != np.float32(r.coef).tobytes():
                oracles[w].u[:], oracles[w].v[:] = snap
                r = oracles[w].compress(hosts[w], coef_override=st.clip_coef)
                overrides += 1
            assert out_i[w].cpu().numpy().tobytes() == r.idx.tobytes(), (t, w)
            assert out_v[w].cpu().numpy().tobytes() == r.val.tobytes(), (t, w)
            res.append(r)
        ref = O.decode_accumulate([r.idx for r in res], [r.val for r in res], L)
        O.apply_sgd(w_ref, ref, 0.1)
        assert dense.cpu().numpy().tobytes() == ref.tobytes()
        assert weights.cpu().numpy().tobytes() == w_ref.tobytes()
    for w in range(NW):
        u, v = states[w].read()
        assert u.tobytes() == oracles[w].u.tobytes() and v.tobytes() == oracles[w].v.tobytes()
    assert overrides <= 1
    for st in states:
        st.close()


def test_cuda_graph_replay_matches_oracle(P):
    """One whole step (dgc_compress_batch of all workers + the one-pass receive side) captured
    into a CUDA graph and replayed: every replay is one more iteration of Algorithm 4 on the
    captured buffers, bit for bit against the oracle.  What changes between calls (sampling
    seed, status counter bank) must therefore come from the device, not from the host call."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    wl = I.workload("lstm_small")
    NW, clip, lr = 3, wl.clip_threshold, 0.05
    states = [B.State(wl.numel, NW, wl.momentum, clip, wl.sparsity, seed=I.BASE_SEED + w)
              for w in range(NW)]
    L, off = states[0].arena_len, states[0].arena_offset
    oracles = [O.Worker(off, wl.numel, L, NW, wl.momentum, clip, wl.sparsity) for _ in range(NW)]
    nnz = states[0].max_nnz
    g_dev = [torch.zeros(L, dtype=torch.float32, device="cuda") for _ in range(NW)]
    out_i = [torch.empty(nnz, dtype=torch.int32, device="cuda") for _ in range(NW)]
    out_v = [torch.empty(nnz, dtype=torch.float32, device="cuda") for _ in range(NW)]
    dense = torch.empty(L, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.decode_workspace_bytes(NW, L), dtype=torch.uint8, device="cuda")
    weights = torch.zeros(L, dtype=torch.float32, device="cuda")
    w_ref = np.zeros(L, np.float32)

    overrides = []

    def step():
        B.compress_batch(states, g_dev, out_i, out_v)
        B.decode_accumulate_sgd(out_i, out_v, dense, weights, lr, ws)

    def load(t):
        hosts = []
        for w in range(NW):
            g = np.zeros(L, np.float32)
            I.fill(wl, g, off, worker=w, iteration=t)
            g *= np.float32(40.0)                # clipping active
            g_dev[w].copy_(torch.from_numpy(g))
            hosts.append(g)
        return hosts

    def check(hosts, t):
        torch.cuda.synchronize()
        res = []
        for w in range(NW):
            st = states[w].status()
            assert st.iterations == t + 1
            snap = (oracles[w].u.copy(), oracles[w].v.copy())
            r = oracles[w].compress(hosts[w])
            if clip > 0:
                assert abs(st.grad_norm - r.norm) <= 1e-6 * r.norm and r.coef < 1.0
            if np.float32(st.clip_coef).tobytes() != np.float32(r.coef).tobytes():
                oracles[w].u[:], oracles[w].v[:] = snap
                r = oracles[w].compress(hosts[w], coef_override=st.clip_coef)
                overrides.append((t, w))
            assert out_i[w].cpu().numpy().tobytes() == r.idx.tobytes(), (t, w)
            assert out_v[w].cpu().numpy().tobytes() == r.val.tobytes(), (t, w)
            res.append(r)
        ref = O.decode_accumulate([r.idx for r in res], [r.val for r in res], L)
        O.apply_sgd(w_ref, ref, lr)
        assert dense.cpu().numpy().tobytes() == ref.tobytes(), t
        assert weights.cpu().numpy().tobytes() == w_ref.tobytes(), t

    hosts = load(0)
    step()                                       # plain call first (creates the side streams)
    check(hosts, 0)
    graph = torch.cuda.CUDAGraph()
    hosts = load(1)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph):
        step()                                   # captured, not run
    for t in range(1, 5):
        if t > 1:
            hosts = load(t)
        graph.replay()
        check(hosts, t)
    for w in range(NW):
        u, v = states[w].read()
        assert u.tobytes() == oracles[w].u.tobytes() and v.tobytes() == oracles[w].v.tobytes()
    assert len(overrides) <= 1
    del graph
    for st in states:
        st.close()


def test_checkpoint_resume_paper_literal_needs_the_call_count(P):
    """Paper-literal mode draws its sample from (seed, call count): a resumed state gives the
    uninterrupted run's lists only with u, v AND the count restored (dgc_state_set_iterations);
    the resumed calls are also checked against the oracle at the restored iteration numbers."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    numel, seed, s = [300000, 9000, 70001], 31, 0.999
    a = B.State(numel, 2, 0.9, 0.0, s, seed=seed, select_mode=1)
    L, off = a.arena_len, a.arena_offset
    cpu = O.Worker(off, numel, L, 2, 0.9, 0.0, s)
    rng = np.random.default_rng(12)
    gs = []
    for _ in range(5):
        g = np.zeros(L, np.float32)
        for o, n in zip(off, numel):
            g[o:o + n] = rng.standard_normal(n).astype(np.float32)
        gs.append(g)
    oi = torch.empty(a.max_nnz, dtype=torch.int32, device="cuda")
    ov = torch.empty(a.max_nnz, dtype=torch.float32, device="cuda")
    for t in range(3):
        a.compress(torch.from_numpy(gs[t]).cuda(), oi, ov)
        O.compress_sampled(cpu, gs[t], seed=seed, iteration=t)
    u, v = a.read()
    done = a.status().iterations
    assert done == 3
    b = B.State(numel, 2, 0.9, 0.0, s, seed=seed, select_mode=1)
    b.write(u, v)
    b.set_iterations(done)
    assert b.status().iterations == 3
    oi2, ov2 = torch.empty_like(oi), torch.empty_like(ov)
    for t in range(3, 5):
        gd = torch.from_numpy(gs[t]).cuda()
        a.compress(gd, oi, ov)
        b.compress(gd, oi2, ov2)
        na, pa = a.nnz()
        nb, pb = b.nnz()
        r, nnz = O.compress_sampled(cpu, gs[t], seed=seed, iteration=t)
        assert na == nb == r.idx.size and pa.tolist() == pb.tolist() == nnz.tolist()
        assert oi2[:nb].cpu().numpy().tobytes() == r.idx.tobytes()
        assert ov2[:nb].cpu().numpy().tobytes() == r.val.tobytes()
        assert torch.equal(oi[:na], oi2[:nb])
        assert torch.equal(ov[:na].view(torch.int32), ov2[:nb].view(torch.int32))
    ua, va = a.read()
    ub, vb = b.read()
    assert ua.tobytes() == ub.tobytes() == cpu.u.tobytes()
    assert va.tobytes() == vb.tobytes() == cpu.v.tobytes()
    with pytest.raises(Exception):
        b.set_iterations(-1)
    a.close()
    b.close()


@pytest.mark.parametrize("case", range(24))
def test_randomised_shapes_distributions_and_sparsities(P, case):
    """Seeded fuzz over what the selection paths branch on: tensor sizes around the segment,
    part and sampling boundaries, sparsities on both sides of the deferred-masking and
    emission-from-v' switches, clipping and Nesterov on or off, and value distributions with
    heavy tails, exact zeros, few distinct magnitudes or constants.  Three iterations each,
    bit for bit against the oracle; the slow full-selection path must never be needed."""
    rng = np.random.default_rng(1000 + case)
    pool = [1, 3, 31, 512, 513, 4095, 8192, 8193, 20000, 70001, 262144, 262145, 300000,
            524288 + 7, 1 << 20, (1 << 21) + 5, 3000000]
    numel = [int(x) for x in rng.choice(pool, size=int(rng.integers(2, 6)))]
    if case % 3 == 0:
        numel.append(int(rng.choice([1 << 22, 5000000])))       # multi-block selection at low s
    sparsity = float(rng.choice([0.0, 0.5, 0.75, 0.9, 0.9375, 0.99, 0.996, 0.999, 0.9999]))
    clip = float(rng.choice([0.0, 1.0]))
    nest = bool(rng.integers(0, 2))
    pair = P.Pair(numel, 4, 0.9, clip, sparsity, seed=int(rng.integers(1, 1 << 30)), nesterov=nest)
    rep = P.ParityReport()
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    kinds = ["normal", "student", "sparse", "levels", "const", "zero"]
    for t in range(3):
        g = P.arena_with_padding_poison(L, off, numel)
        for o, n in zip(off, numel):
            kind = kinds[int(rng.integers(0, len(kinds)))]
            if kind == "normal":
                x = rng.standard_normal(n)
            elif kind == "student":
                x = rng.standard_t(3, size=n) * 1e-4
            elif kind == "sparse":
                x = rng.standard_normal(n) * (rng.random(n) < 0.003)
            elif kind == "levels":
                x = rng.integers(-2, 3, size=n) * 0.125
            elif kind == "const":
                x = np.full(n, 0.5) * (rng.integers(0, 2, size=n) * 2 - 1)
            else:
                x = np.zeros(n)
            g[o:o + n] = x.astype(np.float32)
        _, _, st = pair.step(g, rep, check_state=(t == 2))
        assert st.full_select_last == 0, (case, t, numel, sparsity, st.flags)
    pair.close()


def test_timeline_aid_orders_the_kernels_of_a_call(P):
    """dgc_timeline_*: block start times on the GPU clock, per kernel of a compress call.  The
    results of the call do not change; the kernels appear in the order the algorithm needs."""
    from paper_1712_01887_b200 import binding as B
    numel = [300000, 5000, 70001]
    rng = np.random.default_rng(5)
    a = B.State(numel, 1, 0.9, 0.0, 0.999, seed=3)
    b = B.State(numel, 1, 0.9, 0.0, 0.999, seed=3)
    L = a.arena_len
    g = torch.from_numpy(rng.standard_normal(L).astype(np.float32)).cuda()
    oa = (torch.empty(a.max_nnz, dtype=torch.int32, device="cuda"),
          torch.empty(a.max_nnz, dtype=torch.float32, device="cuda"))
    ob = (torch.empty_like(oa[0]), torch.empty_like(oa[1]))
    with pytest.raises(B.DgcError):
        a.timeline_read()                        # not enabled
    a.timeline_enable(True)
    a.compress(g, *oa)
    b.compress(g, *ob)
    tl = a.timeline_read().astype(np.int64)
    assert (tl[:, 0] <= tl[:, 1]).all() and (tl[:, 0] > 0).all()
    assert tl[0, 0] <= tl[1, 0] <= tl[2, 0] <= tl[3, 0]          # sample, stream, select, emit
    assert tl[0, 1] <= tl[1, 0] and tl[1, 1] <= tl[2, 0] and tl[2, 1] <= tl[3, 0]
    assert torch.equal(oa[0], ob[0]) and torch.equal(oa[1].view(torch.int32), ob[1].view(torch.int32))
    empty = a.timeline_read()
    assert (empty[:, 1] == 0).all() and (empty[:, 0] == np.iinfo(np.uint64).max).all()
    a.timeline_enable(False)
    a.compress(g, *oa)
    with pytest.raises(B.DgcError):
        a.timeline_read()
    a.close()
    b.close()


@pytest.mark.parametrize("case", range(12))
def test_randomised_option_combinations(P, case):
    """Seeded fuzz over the options that the other tests take one at a time: paper-literal
    selection with Nesterov momentum and with clipping on or off, per-tensor clipping at every
    masking and emission mode (with Nesterov or not), each through dgc_compress and through
    dgc_compress_batch (two workers).  Three iterations, bit for bit against the oracle."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    rng = np.random.default_rng(7000 + case)
    pool = [1, 513, 8192, 8193, 20000, 70001, 262145, 300000, 524288 + 7, (1 << 21) + 5]
    numel = [int(x) for x in rng.choice(pool, size=int(rng.integers(2, 5)))]
    literal = case % 2 == 0
    nest = bool(rng.integers(0, 2))
    batch = bool(rng.integers(0, 2))
    sparsity = float(rng.choice([0.75, 0.9375, 0.99, 0.999]))
    clip = float(rng.choice([0.0, 1.0])) if literal else 1.0
    scope = 0 if literal else 1
    seed, NW = 300 + case, 2
    sts = [B.State(numel, 4, 0.9, clip, sparsity, seed=seed, nesterov=nest,
                   select_mode=int(literal), clip_scope=scope) for _ in range(NW)]
    L, off = sts[0].arena_len, sts[0].arena_offset
    cpus = [O.Worker(off, numel, L, 4, 0.9, clip, sparsity, nesterov=nest) for _ in range(NW)]
    cap = sts[0].max_nnz
    oi = [torch.empty(cap, dtype=torch.int32, device="cuda") for _ in range(NW)]
    ov = [torch.empty(cap, dtype=torch.float32, device="cuda") for _ in range(NW)]
    for t in range(3):
        gs = []
        for w in range(NW):
            g = P.arena_with_padding_poison(L, off, numel)
            for o, n in zip(off, numel):
                scale = 10.0 ** float(rng.integers(-2, 2))       # some tensors clipped, some not
                g[o:o + n] = (rng.standard_normal(n) * scale).astype(np.float32)
            gs.append(g)
        dev = [torch.from_numpy(g).cuda() for g in gs]
        if batch:
            B.compress_batch(sts, dev, oi, ov)
        else:
            for w in range(NW):
                sts[w].compress(dev[w], oi[w], ov[w])
        for w in range(NW):
            status = sts[w].status()
            snap = (cpus[w].u.copy(), cpus[w].v.copy())
            if literal:
                r, nnz = O.compress_sampled(cpus[w], gs[w], seed=seed, iteration=t)
                if np.float32(status.clip_coef).tobytes() != np.float32(r.coef).tobytes():
                    cpus[w].u[:], cpus[w].v[:] = snap
                    r, nnz = O.compress_sampled(cpus[w], gs[w], seed=seed, iteration=t,
                                                coef_override=status.clip_coef)
                total, per = sts[w].nnz()
                assert per.tolist() == nnz.tolist(), (case, t, w)
            else:
                norms, coefs = sts[w].clip()
                r = cpus[w].compress_clip_per_tensor(gs[w])
                assert np.all(np.abs(norms - r.norm) <= 1e-6 * np.maximum(r.norm, 1e-300))
                if coefs.tobytes() != r.coef.tobytes():
                    cpus[w].u[:], cpus[w].v[:] = snap
                    r = cpus[w].compress_clip_per_tensor(gs[w], coef_override=coefs)
                total = cap
            assert total == r.idx.size, (case, t, w)
            assert oi[w][:total].cpu().numpy().tobytes() == r.idx.tobytes(), (case, t, w)
            assert ov[w][:total].cpu().numpy().tobytes() == r.val.tobytes(), (case, t, w)
    for w in range(NW):
        u, v = sts[w].read()
        assert u.tobytes() == cpus[w].u.tobytes() and v.tobytes() == cpus[w].v.tobytes(), (case, w)
        sts[w].close()


@pytest.mark.parametrize("case", range(16))
def test_randomised_wide(P, case):
    """A wider seeded fuzz: 1 to 7 tensors of sizes around every boundary (up to 2^23 elements),
    every sparsity the schedule and the sweeps use and the switch points between them, momentum
    0 to 0.99, 1 to 64 workers in the clip scale, sample ratios 0.1 % to 50 %, sparsity changed
    between iterations, and values that are denormal, near the fp32 maximum (sums overflow to
    Inf, Inf - Inf gives NaN) or infinite.  Indices bit for bit; values and state bit for bit
    with a NaN matching any NaN."""
    rng = np.random.default_rng(90000 + case)
    pool = [1, 2, 3, 4, 5, 31, 32, 33, 511, 512, 513, 1023, 4096, 8191, 8192, 8193, 8704, 16385,
            20000, 65536, 70001, 131073, 262143, 262144, 262145, 300000, 524288, 524289, 786433,
            1 << 20, (1 << 21) + 5, 3000000, 4194304 + 1, 6000000]
    numel = [int(x) for x in rng.choice(pool, size=int(rng.integers(1, 7)))]
    if case % 7 == 0:
        numel.append(1 << 23)
    sparsity = float(rng.choice([0.0, 0.25, 0.5, 0.75, 0.8749, 0.875, 0.9, 0.9375, 0.984375, 0.99,
                                 0.996, 0.999, 0.9999, 0.99999]))
    clip = float(rng.choice([0.0, 0.3, 1.0, 1e6]))
    pair = P.Pair(numel, int(rng.choice([1, 2, 8, 64])), float(rng.choice([0.0, 0.5, 0.9, 0.99])),
                  clip, sparsity, seed=int(rng.integers(1, 1 << 30)),
                  nesterov=bool(rng.integers(0, 2)),
                  sample_ratio=float(rng.choice([0.001, 0.003, 0.01, 0.05, 0.5])))
    rep = P.ParityReport()
    off, L = pair.gpu.arena_offset, pair.gpu.arena_len
    kinds = ["normal", "student", "sparse", "levels", "const", "zero", "denorm", "huge", "special"]
    iters = int(rng.integers(2, 6))
    for t in range(iters):
        if t > 0 and rng.random() < 0.3:
            pair.set_sparsity(float(rng.choice([0.5, 0.75, 0.9375, 0.99, 0.999, 0.9999])))
        g = P.arena_with_padding_poison(L, off, numel)
        for o, n in zip(off, numel):
            kind = kinds[int(rng.integers(0, len(kinds)))]
            if kind == "normal":
                x = rng.standard_normal(n)
            elif kind == "student":
                x = rng.standard_t(2, size=n) * 1e-4
            elif kind == "sparse":
                x = rng.standard_normal(n) * (rng.random(n) < 0.003)
            elif kind == "levels":
                x = rng.integers(-2, 3, size=n) * 0.125
            elif kind == "const":
                x = np.full(n, 0.5) * (rng.integers(0, 2, size=n) * 2 - 1)
            elif kind == "denorm":
                x = rng.standard_normal(n) * 1e-41
            elif kind == "huge":
                x = rng.standard_normal(n) * 1e30
            elif kind == "special":
                x = rng.standard_normal(n)
                if clip == 0.0 and n > 8:
                    m = rng.integers(0, n, size=2)
                    x[m[0]], x[m[1]] = np.inf, -np.inf
            else:
                x = np.zeros(n)
            with np.errstate(over="ignore"):
                g[o:o + n] = x.astype(np.float32)
        pair.step(g, rep, check_state=(t == iters - 1))
    pair.close()


@pytest.mark.parametrize("case", range(16))
def test_randomised_receive_side_and_wire_format(P, case):
    """Seeded fuzz of the receive side: 1 to 64 workers, dense lengths around the 4096-element
    tile and up to 5 Mi, lists from empty to complete, values denormal to near the fp32 maximum
    (sums overflow).  Decode, SGD, the fused sparse and the one-pass forms through
    parity_util.receive_side; the workspace-free decode where its limit allows; the run-length
    wire format of one list, encoded and decoded, against the oracle's."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    rng = np.random.default_rng(50000 + case)
    N = int(rng.choice([1, 2, 3, 4, 8, 17, 64]))
    L = int(rng.choice([1, 2, 511, 4095, 4096, 4097, 8192, 100000, 262144, 1 << 20, 3000001,
                        5 << 20]))
    il, vl = [], []
    for w in range(N):
        dens = float(rng.choice([0.0, 1e-5, 1e-3, 0.01, 0.25, 1.0]))
        m = int(min(L, rng.binomial(L, dens))) if dens < 1.0 else L
        idx = (np.sort(rng.choice(L, size=m, replace=False)).astype(np.int32) if m < L
               else np.arange(L, dtype=np.int32))
        kind = int(rng.integers(0, 4))
        val = (rng.standard_normal(m) * [1.0, 1e-41, 1e30][kind] if kind < 3
               else rng.integers(-2, 3, size=m) * 0.5)
        with np.errstate(over="ignore"):
            il.append(idx)
            vl.append(val.astype(np.float32))
    w0 = rng.standard_normal(L).astype(np.float32)
    ref, _ = P.receive_side(il, vl, L, w0, float(rng.choice([0.0, 0.1, 1.0, 1e-3])))
    if N * ((L + 4095) // 4096 + 1025) <= B.STATIC_DECODE_WORDS:
        di = [torch.from_numpy(a).cuda() for a in il]
        dv = [torch.from_numpy(a).cuda() for a in vl]
        dense = torch.full((L,), float("nan"), dtype=torch.float32, device="cuda")
        B.decode_accumulate_static(di, dv, dense)
        P._assert_bits(dense.cpu().numpy(), ref, "workspace-free decode")
        assert B.decode_rejected(N, L) == 0
    for idx, val in zip(il, vl):
        if idx.size == 0:
            continue
        runs, values = B.encode_runlength(torch.from_numpy(idx).cuda(),
                                          torch.from_numpy(val).cuda(), L)
        ro, vo = O.encode_runlength(idx, val, B.runlength_max_entries(idx.size, L))
        assert runs.cpu().numpy().tobytes() == ro.tobytes()
        P._assert_bits(values.cpu().numpy(), vo, "run-length values")
        i2, v2, _ = B.decode_runlength(runs, values)
        io, vo2 = O.decode_runlength(ro, vo)
        assert i2.cpu().numpy().tobytes() == io.tobytes()
        P._assert_bits(v2.cpu().numpy(), vo2, "run-length decoded values")
        break


@pytest.mark.parametrize("case", range(12))
def test_randomised_paper_literal_selection(P, case):
    """Seeded fuzz of select_mode = 1 (Sec. 5 as stated): tensor sizes from 1 element to 2^23,
    sample ratios 0.1 % to 10 %, sparsities 50 % to 99.99 %, momentum, Nesterov and clipping on or
    off, value distributions with ties, zeros and heavy tails.  Per-tensor counts, indices, values
    and state bit for bit against the oracle, which draws the same positions from the same
    counter-based generator."""
    from oracle import dgc_oracle as O
    from paper_1712_01887_b200 import binding as B
    rng = np.random.default_rng(30000 + case)
    pool = [1, 2, 3, 5, 31, 512, 513, 4096, 8192, 8193, 20000, 70001, 262144, 262145, 300000,
            524289, 1 << 20, (1 << 21) + 5, 3000000]
    numel = [int(x) for x in rng.choice(pool, size=int(rng.integers(1, 6)))]
    if case % 9 == 0:
        numel.append(int(rng.choice([1 << 22, 6000000, (1 << 23) + 5])))
    sparsity = float(rng.choice([0.5, 0.75, 0.9375, 0.99, 0.996, 0.999, 0.9999]))
    ratio = float(rng.choice([0.001, 0.002, 0.01, 0.03, 0.1]))
    clip = float(rng.choice([0.0, 1.0]))
    nest = bool(rng.integers(0, 2))
    mom = float(rng.choice([0.0, 0.9]))
    seed = int(rng.integers(1, 1 << 40))
    st = B.State(numel, 4, mom, clip, sparsity, seed=seed, select_mode=1, sample_ratio=ratio,
                 nesterov=nest)
    L, off = st.arena_len, st.arena_offset
    cpu = O.Worker(off, numel, L, 4, mom, clip, sparsity, nesterov=nest)
    oi = torch.empty(st.max_nnz, dtype=torch.int32, device="cuda")
    ov = torch.empty(st.max_nnz, dtype=torch.float32, device="cuda")
    kinds = ["normal", "student", "sparse", "levels", "const", "zero"]
    for t in range(int(rng.integers(2, 5))):
        g = P.arena_with_padding_poison(L, off, numel)
        for o, n in zip(off, numel):
            kind = kinds[int(rng.integers(0, len(kinds)))]
            if kind == "normal":
                x = rng.standard_normal(n)
            elif kind == "student":
                x = rng.standard_t(2, size=n) * 1e-4
            elif kind == "sparse":
                x = rng.standard_normal(n) * (rng.random(n) < 0.003)
            elif kind == "levels":
                x = rng.integers(-2, 3, size=n) * 0.125
            elif kind == "const":
                x = np.full(n, 0.5) * (rng.integers(0, 2, size=n) * 2 - 1)
            else:
                x = np.zeros(n)
            g[o:o + n] = x.astype(np.float32)
        st.compress(torch.from_numpy(g).cuda(), oi, ov)
        status = st.status()
        total, per = st.nnz()
        snap = (cpu.u.copy(), cpu.v.copy())
        r, nnz = O.compress_sampled(cpu, g, seed=seed, iteration=t, sample_ratio=ratio)
        if np.float32(status.clip_coef).tobytes() != np.float32(r.coef).tobytes():
            cpu.u[:], cpu.v[:] = snap
            r, nnz = O.compress_sampled(cpu, g, seed=seed, iteration=t, sample_ratio=ratio,
                                        coef_override=status.clip_coef)
        assert per.tolist() == nnz.tolist(), (case, t, numel, sparsity, ratio)
        assert oi[:total].cpu().numpy().tobytes() == r.idx.tobytes(), (case, t)
        assert ov[:total].cpu().numpy().tobytes() == r.val.tobytes(), (case, t)
    u, v = st.read()
    assert u.tobytes() == cpu.u.tobytes() and v.tobytes() == cpu.v.tobytes()
    st.close()


def test_host_buffer_calls_follow_sparsity_changes(P):
    """dgc_compress_host and dgc_compress_host_batch across dgc_set_sparsity in both directions
    (their device staging must grow with the list length): bit for bit what dgc_compress gives
    on device buffers, lists and final state."""
    from paper_1712_01887_b200 import binding as B
    numel = [300000, 70001, 64, 9000, 600000]
    NW = 3
    rng = np.random.default_rng(5)
    dev = [B.State(numel, NW, 0.9, 1.0, 0.999, seed=w) for w in range(NW)]
    host = [B.State(numel, NW, 0.9, 1.0, 0.999, seed=w) for w in range(NW)]
    L = dev[0].arena_len
    for t, s in enumerate([0.999, 0.75, 0.75, 0.9999, 0.5, 0.999, 0.99]):
        for st in dev + host:
            st.set_sparsity(s)
        nnz = dev[0].max_nnz
        hi = [torch.empty(nnz, dtype=torch.int32).pin_memory() for _ in range(NW)]
        hv = [torch.empty(nnz, dtype=torch.float32).pin_memory() for _ in range(NW)]
        gh = [torch.from_numpy(rng.standard_normal(L).astype(np.float32)).pin_memory()
              for _ in range(NW)]
        if t % 2 == 0:
            B.compress_host_batch(host, gh, hi, hv)
        else:
            for w in range(NW):
                host[w].compress_host(gh[w], hi[w], hv[w])
        for w in range(NW):
            oi = torch.empty(nnz, dtype=torch.int32, device="cuda")
            ov = torch.empty(nnz, dtype=torch.float32, device="cuda")
            dev[w].compress(gh[w].cuda(), oi, ov)
            assert torch.equal(oi.cpu(), hi[w]), (t, w)
            assert torch.equal(ov.cpu().view(torch.int32), hv[w].view(torch.int32)), (t, w)
    for w in range(NW):
        a, b = dev[w].read(), host[w].read()
        assert a[0].tobytes() == b[0].tobytes() and a[1].tobytes() == b[1].tobytes()
        dev[w].close()
        host[w].close()
