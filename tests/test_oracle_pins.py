"""Pins for the CPU oracle: every check here compares the oracle against
something other than itself -- hand-worked traces (tests/golden), closed forms
of the paper's equations, brute force, numpy library routines, invariants."""
import json
import os

import numpy as np
import pytest

from oracle import dgc_oracle as O


def _load(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return json.load(f)


def _f32(x):
    return np.asarray(x, dtype=np.float32)


def _single(n, momentum, sparsity, clip=0.0, workers=1):
    return O.Worker([0], [n], n, workers, momentum, clip, sparsity)


# ------------------------------------------------------------------ hand-worked traces

def test_alg4_two_iterations_trace(golden_dir):
    G = _load(golden_dir, "alg4_two_iterations.json")
    for brute in (False, True):
        w = _single(G["n"], G["momentum"], G["sparsity"])
        assert w.k.tolist() == [G["k"]]
        for it in G["iterations"]:
            r = w.compress(_f32(it["g"]), brute_force=brute)
            assert r.idx.tolist() == it["sent_idx"]
            assert r.val.tolist() == it["sent_val"]
            assert w.u.tolist() == it["u_after"]
            assert w.v.tolist() == it["v_after"]
            assert r.coef == np.float32(1.0)


def test_alg5_nesterov_trace(golden_dir):
    G = _load(golden_dir, "alg5_nesterov_two_iterations.json")
    w = O.Worker([0], [G["n"]], G["n"], 1, G["momentum"], 0.0, G["sparsity"], nesterov=True)
    assert w.k.tolist() == [G["k"]]
    for it in G["iterations"]:
        r = w.compress(_f32(it["g"]))
        assert r.idx.tolist() == it["sent_idx"]
        assert r.val.tolist() == it["sent_val"]
        assert w.u.tolist() == it["u_after"]
        assert w.v.tolist() == it["v_after"]


def test_nesterov_matches_eq8_parametrisation():
    """Appendix B, Eq. 8: u' = m u + g ; v' = v + (m u' + g).  Algorithm 5 stores U = m u'.
    A float64 shadow of Eq. 8 must track the oracle's Algorithm 5 state on unsent entries."""
    rng = np.random.default_rng(13)
    n, T, m = 50, 10, 0.9
    w = O.Worker([0], [n], n, 1, m, 0.0, 0.98, nesterov=True)      # k = 1
    G = rng.standard_normal((T, n)).astype(np.float32)
    G[:, 7] = 1e6
    u_eq = np.zeros(n)
    v_eq = np.zeros(n)
    for t in range(T):
        r = w.compress(G[t].copy())
        assert r.idx.tolist() == [7]
        u_eq = m * u_eq + G[t].astype(np.float64)
        v_eq = v_eq + (m * u_eq + G[t].astype(np.float64))
    keep = np.arange(n) != 7
    np.testing.assert_allclose(w.u[keep], (m * u_eq)[keep], rtol=2e-5, atol=1e-6)
    np.testing.assert_allclose(w.v[keep], v_eq[keep], rtol=2e-5, atol=1e-6)
    # constant gradient closed form: u_eq,t = g (1 - m^t)/(1 - m); v_T = sum_t (m u_eq,t + g)
    w2 = O.Worker([0], [4], 4, 1, 0.5, 0.0, 0.75, nesterov=True)
    g = _f32([0.25, 0.25, 0.25, 4096.0])
    for t in range(1, 7):
        w2.compress(g.copy())
        u_t = [0.25 * (1 - 0.5 ** i) / 0.5 for i in range(1, t + 1)]
        assert w2.u[0] == np.float32(0.5 * u_t[-1])
        assert w2.v[0] == np.float32(sum(0.5 * x + 0.25 for x in u_t))


def test_tie_goes_to_lower_index(golden_dir):
    G = _load(golden_dir, "tie_rule.json")
    for brute in (False, True):
        w = _single(G["n"], G["momentum"], G["sparsity"])
        assert w.k.tolist() == [G["k"]]
        r = w.compress(_f32(G["g"]), brute_force=brute)
        assert r.idx.tolist() == G["sent_idx"]
        assert r.val.tolist() == G["sent_val"]


def test_clip_345(golden_dir):
    G = _load(golden_dir, "clip_345.json")
    g = _f32(G["g"])
    for c in G["cases"]:
        norm, coef = O.clip_coef([0], [4], g, c["clip_threshold"], G["num_workers"])
        assert norm == c["norm"]
        assert coef == np.float32(c["coef"])
        # s = 0 sends everything, so the sent values are the clipped gradient itself
        w = O.Worker([0], [4], 4, G["num_workers"], 0.9, c["clip_threshold"], 0.0)
        r = w.compress(g)
        assert r.val.tolist() == c["gc"]
        if c["coef"] == 1.0:
            assert r.val.tobytes() == g.tobytes()     # identity bit for bit


def test_decode_and_sgd(golden_dir):
    G = _load(golden_dir, "decode_sgd.json")
    idx = [np.asarray(w["idx"], dtype=np.int32) for w in G["workers"]]
    val = [_f32(w["val"]) for w in G["workers"]]
    dense = O.decode_accumulate(idx, val, G["dense_len"])
    assert dense.tolist() == G["dense"]
    w = _f32(G["w_before"]).copy()
    O.apply_sgd(w, dense, G["lr"])
    assert w.tolist() == G["w_after"]


def test_warmup_schedule_and_k(golden_dir):
    G = _load(golden_dir, "warmup_schedule.json")
    assert [O.warmup_sparsity(i) for i in range(5)] == G["sparsity"]
    assert O.warmup_sparsity(5) == -1.0 and O.warmup_sparsity(-1) == -1.0
    assert [O.topk_count(G["n"], s) for s in G["sparsity"]] == G["k"]
    for c in G["more_k"]:
        assert O.topk_count(c["n"], c["sparsity"]) == c["k"], c


# ------------------------------------------------------------------ selection vs brute force / numpy

def _numpy_topk(v, k):
    key = (v.view(np.uint32) & np.uint32(0x7FFFFFFF)).astype(np.int64)
    order = np.argsort(-key, kind="stable")      # ties keep ascending index
    return np.sort(order[:k])


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 31, 32, 33, 255, 1000, 4095, 4096])
def test_selection_matches_full_sort(n):
    rng = np.random.default_rng(n)
    for trial in range(6):
        if trial % 3 == 0:
            v = rng.standard_normal(n).astype(np.float32)
        elif trial % 3 == 1:      # heavy ties, both signs, zeros
            v = rng.integers(-3, 4, size=n).astype(np.float32)
        else:                     # mostly zeros
            v = rng.standard_normal(n).astype(np.float32)
            v[rng.random(n) < 0.9] = 0.0
        for k in sorted({1, max(1, n // 1000), max(1, n // 4), max(1, n - 1), n}):
            ref = _numpy_topk(v, k)
            assert np.array_equal(O.select_topk(v, k, brute_force=True), ref)
            assert np.array_equal(O.select_topk(v, k, brute_force=False), ref)


def test_selection_special_values():
    v = _f32([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-45, -1e-45, 1.0])
    # NaN first, then the two infinities by index, then 1.0, then denormals by index
    assert O.select_topk(v, 1).tolist() == [4]
    assert O.select_topk(v, 3).tolist() == [2, 3, 4]
    assert O.select_topk(v, 4).tolist() == [2, 3, 4, 7]
    assert O.select_topk(v, 5).tolist() == [2, 3, 4, 5, 7]
    assert O.select_topk(v, 7).tolist() == [0, 2, 3, 4, 5, 6, 7]


def test_selected_dominate_unselected():
    rng = np.random.default_rng(7)
    n = 50000
    v = rng.standard_t(3, n).astype(np.float32)
    k = O.topk_count(n, 0.999)
    assert k == 50
    sel = O.select_topk(v, k)
    mask = np.zeros(n, bool)
    mask[sel] = True
    assert np.all(np.diff(sel) > 0)
    assert np.abs(v[mask]).min() >= np.abs(v[~mask]).max()


# ------------------------------------------------------------------ closed forms of Eq. 4 / Eq. 5

def test_momentum_correction_closed_form_unsent():
    """Eq. 4: an entry that is not sent for T iterations has accumulated
    sum_t g_t * sum_{tau=0}^{T-t} m^tau.  One decoy entry with a huge gradient
    is the top-1 pick every iteration, so entries 1.. are never sent."""
    rng = np.random.default_rng(3)
    n, T, m = 64, 12, 0.9
    w = _single(n, m, 0.999)          # k = 1
    G = rng.standard_normal((T, n)).astype(np.float32)
    G[:, 0] = 1e6
    for t in range(T):
        r = w.compress(G[t].copy())
        assert r.idx.tolist() == [0]
    g64 = G.astype(np.float64)
    expect_v = np.zeros(n)
    expect_u = np.zeros(n)
    for t in range(T):
        geo = (1.0 - m ** (T - t)) / (1.0 - m)       # sum_{tau=0}^{T-t-1} m^tau  (t is 0-based)
        expect_v += g64[t] * geo
        expect_u += g64[t] * m ** (T - 1 - t)
    np.testing.assert_allclose(w.v[1:], expect_v[1:], rtol=2e-5, atol=1e-6)
    np.testing.assert_allclose(w.u[1:], expect_u[1:], rtol=2e-5, atol=1e-6)
    assert w.v[0] == 0.0 and w.u[0] == 0.0


def test_constant_gradient_geometric_sum_exact():
    """u_t = g (1 - m^t)/(1 - m) for a constant gradient; exact for dyadic m, g."""
    n, m = 16, 0.5
    w = _single(n, m, 0.999)
    g = np.full(n, 0.25, np.float32)
    g[5] = 1024.0                      # always the one that is sent
    for t in range(1, 9):
        w.compress(g.copy())
        u_expect = 0.25 * (1 - m ** t) / (1 - m)
        v_expect = sum(0.25 * (1 - m ** i) / (1 - m) for i in range(1, t + 1))
        assert w.u[0] == np.float32(u_expect)
        assert w.v[0] == np.float32(v_expect)


def test_zero_momentum_is_plain_accumulation():
    """m = 0 reduces Algorithm 4 to Algorithm 1: v is the running sum of g."""
    rng = np.random.default_rng(11)
    n, T = 100, 7
    w = _single(n, 0.0, 0.99)          # k = 1
    G = rng.integers(-8, 9, size=(T, n)).astype(np.float32)   # small integers: exact sums
    G[:, 3] = 1000.0
    for t in range(T):
        w.compress(G[t].copy())
    expect = G.sum(axis=0)
    expect[3] = 0
    assert np.array_equal(w.v, expect)


def test_sparsity_zero_is_dense_sgd():
    """s = 0: every entry is sent every iteration, u and v end at zero, the sent
    values are the (clipped) gradient: plain synchronous SGD (Algorithm 2)."""
    rng = np.random.default_rng(5)
    n = 257
    w = _single(n, 0.9, 0.0, clip=0.0)
    for t in range(3):
        g = rng.standard_normal(n).astype(np.float32)
        r = w.compress(g)
        assert r.idx.tolist() == list(range(n))
        assert r.val.tobytes() == g.tobytes()
        assert not w.u.any() and not w.v.any()


# ------------------------------------------------------------------ clipping vs numpy

def test_clip_norm_matches_numpy_and_lands_on_threshold():
    rng = np.random.default_rng(9)
    numel = [1000, 37, 4096]
    offset = [0, 1024, 1100]
    arena = np.full(1100 + 4096, np.float32(np.nan))       # gaps hold NaN: must not be read
    for o, n in zip(offset, numel):
        arena[o:o + n] = rng.standard_normal(n).astype(np.float32)
    flat = np.concatenate([arena[o:o + n] for o, n in zip(offset, numel)]).astype(np.float64)
    norm, coef = O.clip_coef(offset, numel, arena, 4.0, 16)      # thr_local = 1.0
    assert abs(norm - np.linalg.norm(flat)) <= 1e-12 * norm
    assert abs(np.float64(coef) - 1.0 / np.linalg.norm(flat)) <= 1e-7 * coef
    clipped = flat.astype(np.float32) * coef
    assert abs(np.linalg.norm(clipped.astype(np.float64)) - 1.0) < 1e-6
    # N^-1/2: four workers halve the threshold exactly
    _, c1 = O.clip_coef(offset, numel, arena, 2.0, 1)
    _, c4 = O.clip_coef(offset, numel, arena, 4.0, 4)
    assert c1 == c4
    # below threshold: untouched
    _, c0 = O.clip_coef(offset, numel, arena, 1e6, 4)
    assert c0 == np.float32(1.0)


def test_clipping_happens_before_accumulation():
    """Sec. 3.2: clip the new gradient, not the accumulated one."""
    w = O.Worker([0], [4], 4, 1, 0.5, 1.0, 0.75)      # k = 1, thr_local = 1
    r = w.compress(_f32([8, 0, 0, 6]))                 # norm 10 -> coef 0.1
    assert r.coef == np.float32(0.1)
    expect = _f32([8, 0, 0, 6]) * np.float32(0.1)
    assert r.idx.tolist() == [0] and r.val[0] == expect[0]
    assert w.v[3] == expect[3] and w.u[3] == expect[3]
    r = w.compress(_f32([0, 0.5, 0, 0]))               # norm 0.5 < 1: no clip although |v| is larger
    assert r.coef == np.float32(1.0)
    assert r.idx.tolist() == [3]                       # v = [0, 0.5, 0, 0.6 + 0.3]
    assert w.u[1] == np.float32(0.5) and w.v[1] == np.float32(0.5)


def test_clip_per_tensor_option():
    """Clipping per tensor: each tensor is scaled by thr_local / ||g[j]|| iff its own norm
    exceeds thr_local; dyadic example by hand, numpy norms, and the difference from the
    whole-set reading."""
    # two tensors, N = 4, thr_G = 10 -> thr_local = 5: [6, 8] has norm 10 -> coef 0.5;
    # [3, 4, 0] has norm 5, not above the threshold -> untouched
    w = O.Worker([0, 2], [2, 3], 5, 4, 0.0, 10.0, 0.0)          # s = 0: everything is sent
    g = _f32([6, 8, 3, 4, 0])
    r = w.compress_clip_per_tensor(g)
    assert r.norm.tolist() == [10.0, 5.0] and r.coef.tolist() == [0.5, 1.0]
    assert r.val.tolist() == [3.0, 4.0, 3.0, 4.0, 0.0]
    # the whole-set reading clips both by one coefficient: norm sqrt(125) > 5
    w0 = O.Worker([0, 2], [2, 3], 5, 4, 0.0, 10.0, 0.0)
    r0 = w0.compress(g)
    assert r0.coef == np.float32(5.0 / np.sqrt(125.0)) and r0.val[2] != 3.0
    # numpy: per-tensor norms, coefficients and clipped norms on random data with gaps
    rng = np.random.default_rng(12)
    numel, offset, L = [1000, 37, 4096], [0, 1024, 1100], 1100 + 4096
    arena = np.full(L, np.float32(np.nan))
    scale = [1.0, 0.01, 3.0]
    for o, n, sc in zip(offset, numel, scale):
        arena[o:o + n] = (rng.standard_normal(n) * sc).astype(np.float32)
    w = O.Worker(offset, numel, L, 4, 0.0, 20.0, 0.0)           # thr_local = 10
    r = w.compress_clip_per_tensor(arena)
    for j, (o, n) in enumerate(zip(offset, numel)):
        ref = np.linalg.norm(arena[o:o + n].astype(np.float64))
        assert abs(r.norm[j] - ref) <= 1e-12 * ref
        if ref > 10.0:
            assert abs(np.float64(r.coef[j]) - 10.0 / ref) <= 1e-7 * r.coef[j]
            sent = r.val[w.out_offset[j]:w.out_offset[j + 1]].astype(np.float64)
            assert abs(np.linalg.norm(sent) - 10.0) < 1e-5
        else:
            assert r.coef[j] == 1.0
    assert (r.coef < 1).tolist() == [True, False, True]
    # clipping off: identical to the plain iteration
    a = O.Worker(offset, numel, L, 4, 0.9, 0.0, 0.99)
    b = O.Worker(offset, numel, L, 4, 0.9, 0.0, 0.99)
    ra, rb = a.compress_clip_per_tensor(arena), b.compress(arena)
    assert ra.idx.tobytes() == rb.idx.tobytes() and ra.val.tobytes() == rb.val.tobytes()
    assert a.u[:1000].tobytes() == b.u[:1000].tobytes()
    # the override replaces the computed coefficients
    c = O.Worker([0, 2], [2, 3], 5, 4, 0.0, 10.0, 0.0)
    rc = c.compress_clip_per_tensor(g, coef_override=[0.25, 0.5])
    assert rc.val.tolist() == [1.5, 2.0, 1.5, 2.0, 0.0]


# ------------------------------------------------------------------ invariants on a multi-tensor run

def _run_multi(seed, numel, T, momentum, sparsity, clip, workers=4):
    rng = np.random.default_rng(seed)
    offset, pos = [], 0
    for n in numel:
        offset.append(pos)
        pos += n + 5                      # gaps between tensors
    arena_len = pos
    w = O.Worker(offset, numel, arena_len, workers, momentum, clip, sparsity)
    valid = np.zeros(arena_len, bool)
    for o, n in zip(offset, numel):
        valid[o:o + n] = True
    shadow_u = np.zeros(arena_len)
    shadow_acc = np.zeros(arena_len)
    sent_sum = np.zeros(arena_len)
    for t in range(T):
        g = np.zeros(arena_len, np.float32)
        g[valid] = (rng.standard_normal(valid.sum()) * 10.0 ** rng.uniform(-3, 0)).astype(np.float32)
        g[~valid] = np.nan                # the oracle must never read a gap
        u_before, v_before = w.u.copy(), w.v.copy()
        r = w.compress(g)
        # float64 shadow of Eq. 5 with the same coefficient and the same mask
        gc = np.where(valid, g.astype(np.float64) * np.float64(r.coef), 0.0)
        shadow_u = momentum * shadow_u + gc
        shadow_acc += shadow_u
        shadow_u[r.idx] = 0.0
        sent_sum[r.idx] += r.val.astype(np.float64)
        yield w, r, g, u_before, v_before, valid, shadow_acc, sent_sum


@pytest.mark.parametrize("sparsity", [0.999, 0.984375, 0.75])
def test_invariants_multi_tensor(sparsity):
    numel = [64, 1, 5000, 333, 20000]
    momentum = 0.9
    for w, r, g, u_before, v_before, valid, shadow_acc, sent_sum in _run_multi(
            1, numel, 8, momentum, sparsity, clip=1.0):
        # nnz = ceil(n (1 - s)) per tensor
        k = [max(1, int(np.ceil(n * (1 - sparsity) - 1e-9))) for n in numel]
        assert w.k.tolist() == k
        assert r.idx.size == sum(k)
        # segments ascending, inside their tensor
        for j, (o, n) in enumerate(zip(w.offset, w.numel)):
            seg = r.idx[w.out_offset[j]:w.out_offset[j + 1]]
            assert np.all(np.diff(seg) > 0)
            assert seg.min() >= o and seg.max() < o + n
        # u, v zero at sent entries; elsewhere equal to one step of Eq. 5 from the previous state
        assert not w.u[r.idx].any() and not w.v[r.idx].any()
        gc = (g * r.coef).astype(np.float32)
        u_new = (np.float32(momentum) * u_before + gc).astype(np.float32)
        v_new = (v_before + u_new).astype(np.float32)
        unsent = valid.copy()
        unsent[r.idx] = False
        assert np.array_equal(w.u[unsent], u_new[unsent])
        assert np.array_equal(w.v[unsent], v_new[unsent])
        assert np.array_equal(r.val, v_new[r.idx])
        # gaps never written
        assert not w.u[~valid].any() and not w.v[~valid].any()
        # selected dominate unselected, per tensor
        for j, (o, n) in enumerate(zip(w.offset, w.numel)):
            seg = r.idx[w.out_offset[j]:w.out_offset[j + 1]]
            m = np.zeros(n, bool)
            m[seg - o] = True
            a = np.abs(v_new[o:o + n])
            if (~m).any():
                assert a[m].min() >= a[~m].max()
        # conservation: sent so far + residual v = accumulated velocity (Eq. 5 in float64)
        tol = 1e-5 * (np.abs(shadow_acc).max() + 1e-30)
        np.testing.assert_allclose(sent_sum + w.v, shadow_acc, atol=tol, rtol=0)


def test_selection_path_equals_brute_force_path_over_iterations():
    numel = [4096, 17, 1000]
    runs = []
    for brute in (False, True):
        rng = np.random.default_rng(21)
        w = O.Worker([0, 4096, 4200], numel, 5200, 2, 0.9, 0.5, 0.99)
        out = []
        for t in range(6):
            g = np.zeros(5200, np.float32)
            g[:] = rng.integers(-4, 5, size=5200).astype(np.float32) * np.float32(0.125)
            r = w.compress(g, brute_force=brute)
            out.append((r.idx.copy(), r.val.copy(), w.u.copy(), w.v.copy()))
        runs.append(out)
    for a, b in zip(*runs):
        for x, y in zip(a, b):
            assert np.array_equal(x, y)


# ------------------------------------------------------------------ decode / sgd vs numpy

def test_decode_matches_numpy_add_at_in_worker_order():
    rng = np.random.default_rng(2)
    L, N = 10000, 5
    idx = [np.sort(rng.choice(L, size=rng.integers(0, 400), replace=False)).astype(np.int32)
           for _ in range(N)]
    idx[2] = idx[0].copy()                    # full overlap between two workers
    val = [rng.standard_normal(a.size).astype(np.float32) for a in idx]
    dense = O.decode_accumulate(idx, val, L)
    ref = np.zeros(L, np.float32)
    for a, b in zip(idx, val):
        ref[a] = ref[a] + b                   # unique indices per worker: plain fp32 adds, in order
    assert dense.tobytes() == ref.tobytes()
    # one worker: pure scatter; signed zero start is +0
    one = O.decode_accumulate(idx[:1], val[:1], L)
    ref1 = np.zeros(L, np.float32)
    ref1[idx[0]] = val[0]
    assert np.array_equal(one, ref1)
    assert not np.signbit(one[np.setdiff1d(np.arange(L), idx[0])]).any()
    # empty lists
    z = O.decode_accumulate([np.zeros(0, np.int32)], [np.zeros(0, np.float32)], 7)
    assert z.tolist() == [0.0] * 7


def test_sgd_matches_numpy_two_roundings():
    rng = np.random.default_rng(4)
    w = rng.standard_normal(1001).astype(np.float32)
    G = rng.standard_normal(1001).astype(np.float32)
    lr = np.float32(0.1)
    ref = (w - (lr * G).astype(np.float32)).astype(np.float32)
    O.apply_sgd(w, G, float(lr))
    assert w.tobytes() == ref.tobytes()


def test_end_to_end_matches_dense_momentum_sgd_when_everything_is_eventually_sent():
    """Eq. 3 vs Eq. 5: with momentum correction, what one worker has sent plus what
    it still holds equals the dense momentum-SGD velocity sum -- as long as the
    masking never fired on a non-zero u (here: s = 0 is excluded, so use the
    residual form: sum of sent + v = sum_t u_t with u following the masked recurrence).
    Checked exactly on dyadic data."""
    n, m = 8, 0.5
    w = _single(n, m, 0.75)
    rng = np.random.default_rng(0)
    acc = np.zeros(n)
    u = np.zeros(n)
    sent = np.zeros(n)
    for t in range(6):
        g = rng.integers(-4, 5, size=n).astype(np.float32)
        r = w.compress(g.copy())
        u = m * u + g
        acc += u
        u[r.idx] = 0
        sent[r.idx] += r.val
        assert np.array_equal(sent + w.v, acc)


# ------------------------------------------------------------------ encode(): values + 16-bit zero runs

def test_encode_runlength_hand_example(golden_dir):
    G = _load(golden_dir, "encode_runlength.json")
    runs, values = O.encode_runlength(np.asarray(G["idx"], np.int32), _f32(G["val"]), 16)
    assert runs.tolist() == G["runs"] and values.tolist() == G["values"]
    idx, val = O.decode_runlength(runs, values)
    assert idx.tolist() == G["decoded_idx"] and val.tolist() == G["values"]
    with pytest.raises(ValueError):
        O.encode_runlength(np.asarray(G["idx"], np.int32), _f32(G["val"]), 5)


def test_encode_runlength_round_trip_and_size():
    rng = np.random.default_rng(77)
    for L, k in ((1000, 0), (1000, 1000), (5_000_000, 5000), (3_000_000, 7), (70000, 2)):
        idx = np.sort(rng.choice(L, size=k, replace=False)).astype(np.int32)
        val = rng.standard_normal(k).astype(np.float32)
        runs, values = O.encode_runlength(idx, val, k + L // 65536 + 1)
        # fillers: one per full 65536 positions of every gap
        gaps = np.diff(np.concatenate([[-1], idx.astype(np.int64)])) - 1
        assert runs.size == k + int((gaps // 65536).sum())
        di, dv = O.decode_runlength(runs, values)
        dense = np.zeros(L, np.float32)
        dense[idx] = val
        back = np.zeros(L, np.float32)
        back[di] = dv
        assert back.tobytes() == dense.tobytes()
        assert np.all(np.diff(di) > 0)
    # compression ratio of a 99.9 %-sparse vector stays below the format's bound 4/(6*0.001)
    L, k = 2_000_000, 2000
    idx = np.sort(rng.choice(L, size=k, replace=False)).astype(np.int32)
    runs, values = O.encode_runlength(idx, np.ones(k, np.float32), k + 64)
    ratio = 4 * L / (6 * runs.size)
    assert 600 < ratio <= 4 / (6 * 0.001) + 1e-9


# ------------------------------------------------------------------ paper-literal sampled selection (Sec. 5)
# The selection takes the sample positions as an input, so it is pinned here on positions
# chosen by hand, against numpy's partition of |v| at those positions; the position generator
# is pinned separately against the published SplitMix64 outputs.

def _numpy_topk_set(v, k):
    return set(_numpy_topk(v, k).tolist())


def _numpy_from_sample(v, positions, k, sparsity):
    """Sec. 5 with numpy: threshold = the ceil(S (1 - s))-th largest sampled |v| (np.partition),
    mask |v| > thr, exact top-k when more than 2k pass."""
    a = np.abs(v)
    samp = a[np.asarray(positions)]
    S = samp.size
    ks = max(1, -((-S * round((1 - sparsity) * 10**9)) // 10**9))      # ceil in integers
    thr = np.partition(samp, S - ks)[S - ks]
    passed = np.flatnonzero(a > thr)
    if passed.size > 2 * k:
        return _numpy_topk(v, k), thr
    return passed, thr


def test_sample_threshold_rank_is_ceil_S_times_1_minus_s():
    """Distinct magnitudes 1..n at known places: the sample's sorted values are known, so the
    threshold is readable by eye, and rank k_s - 1 or k_s + 1 would give another count."""
    n = 1000
    v = _f32(np.arange(1, n + 1))                         # |v_i| = i + 1
    v[::2] *= -1                                          # signs must not matter
    # S = 20 positions holding the values 50, 100, ..., 1000; s = 0.9 -> k_s = ceil(2.0) = 2
    positions = np.arange(49, n, 50)
    sel, thr = O.select_from_sample(v, positions, k=500, sparsity=0.9)
    assert np.array([thr], np.uint32).view(np.float32)[0] == 950.0    # 2nd largest of the sample
    assert sel.tolist() == list(range(950, 1000))         # the 50 values above 950, ascending
    # S(1-s) an exact integer must not be rounded up by a float ceil: s = 0.75, S = 20 -> 5
    sel, thr = O.select_from_sample(v, positions, k=500, sparsity=0.75)
    assert np.array([thr], np.uint32).view(np.float32)[0] == 800.0
    assert sel.size == 200
    # s = 0.999 -> k_s = ceil(0.02) = 1: the sample maximum; nothing exceeds 1000 -> nothing sent
    sel, thr = O.select_from_sample(v, positions, k=500, sparsity=0.999)
    assert np.array([thr], np.uint32).view(np.float32)[0] == 1000.0 and sel.size == 0
    # s = 0.94 -> S(1-s) = 1.2 -> k_s = 2 (ceil, not round)
    sel, thr = O.select_from_sample(v, positions, k=500, sparsity=0.94)
    assert np.array([thr], np.uint32).view(np.float32)[0] == 950.0
    # order of the positions is irrelevant, a repeated position counts as two draws
    sel2, thr2 = O.select_from_sample(v, positions[::-1].copy(), k=500, sparsity=0.9)
    assert sel2.tolist() == list(range(950, 1000)) and thr2 == thr
    rep = np.concatenate([positions, [999]])              # 1000 drawn twice: S = 21, k_s = 3
    sel3, thr3 = O.select_from_sample(v, rep, k=500, sparsity=0.9)
    assert np.array([thr3], np.uint32).view(np.float32)[0] == 950.0   # 1000, 1000, 950
    assert sel3.tolist() == list(range(950, 1000))


def test_sample_threshold_ties_and_strict_compare():
    """Entries equal to the threshold are not sent (strict >), also when the sample holds the
    threshold value several times."""
    v = _f32([5, 3, 3, 3, 1, 0, 7, 3, 9, 2])
    # sample = {3, 3, 9, 1}: s = 0.5 -> k_s = 2 -> thr = 3 -> sent: 5, 7, 9
    sel, thr = O.select_from_sample(v, np.array([1, 2, 8, 4]), k=4, sparsity=0.5)
    assert np.array([thr], np.uint32).view(np.float32)[0] == 3.0
    assert sel.tolist() == [0, 6, 8]
    # threshold 0 (sample of zeros): every non-zero passes; 8 > 2k = 4 -> exact top-2 = {8, 6}
    sel, thr = O.select_from_sample(v, np.array([5, 5, 5]), k=2, sparsity=0.5)
    assert thr == 0 and sel.tolist() == [6, 8]


def test_far_more_than_expected_is_more_than_2k():
    """Exactly 2k passing entries are sent as they are; 2k + 1 trigger the precise top-k."""
    n = 100
    v = _f32(np.arange(n))                                # |v_i| = i
    # sample {89}: thr = 89 -> 10 entries pass (90..99)
    sel, _ = O.select_from_sample(v, np.array([89]), k=5, sparsity=0.9)     # 10 == 2k
    assert sel.tolist() == list(range(90, 100))
    sel, _ = O.select_from_sample(v, np.array([88]), k=5, sparsity=0.9)     # 11 > 2k
    assert sel.tolist() == list(range(95, 100))
    # and the precise selection keeps the tie rule (lower index first)
    v = _f32([4, 4, 4, 4, 4, 4, 1, 0])
    sel, _ = O.select_from_sample(v, np.array([6]), k=2, sparsity=0.5)      # 6 pass > 4
    assert sel.tolist() == [0, 1]


@pytest.mark.parametrize("seed", range(6))
def test_selection_from_sample_matches_numpy_partition(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(50, 20000))
    s = float(rng.choice([0.5, 0.9, 0.99, 0.999]))
    v = rng.standard_t(3, n).astype(np.float32)
    if seed % 2:
        v = np.round(v * 4) / 4                           # many exact ties
        v = v.astype(np.float32)
    S = int(rng.integers(1, max(2, n // 10)))
    positions = rng.integers(0, n, S)
    k = O.topk_count(n, s)
    sel, thr = O.select_from_sample(v, positions, k, s)
    ref, thr_ref = _numpy_from_sample(v, positions, k, s)
    assert np.array([thr], np.uint32).view(np.float32)[0] == thr_ref
    assert sel.tolist() == ref.tolist()


def test_sample_size_is_the_configured_share_of_the_tensor():
    """Sec. 5: 0.1 % to 1 % of the gradients; ceil, at least one, never more than n."""
    assert O.sample_count(400000, 0.01) == 4000
    assert O.sample_count(400001, 0.01) == 4001
    assert O.sample_count(1 << 28, 0.01) == 2684355       # no cap: still 1 % of 2^28
    assert O.sample_count(1 << 28, 0.001) == 268436
    assert O.sample_count(64, 0.01) == 1
    assert O.sample_count(1, 0.01) == 1
    assert O.sample_count(3, 0.5) == 2
    assert O.sample_count(1000, 0.0) == 10                # 0 selects the default 1 %


def test_position_generator_is_splitmix64_scaled_to_n():
    """The hash is the SplitMix64 step, pinned by its published outputs (state 0: first three
    outputs; state 1234567: first two); a position is floor(h n / 2^64)."""
    G = 0x9E3779B97F4A7C15
    assert O.mix64(0) == 0xE220A8397B1DCDAF
    assert O.mix64(G) == 0x6E789E6AA1B965F4
    assert O.mix64(2 * G & (2**64 - 1)) == 0x06C45D188009454F
    assert O.mix64(1234567) == 6457827717110365317
    assert O.mix64((1234567 + G) & (2**64 - 1)) == 3203168211198807973
    # call seed 0, tensor 0: draw r hashes the counter r itself
    n = 1000
    pos = O.sample_positions(n, 3, 0, 0)
    assert pos.tolist() == [(0xE220A8397B1DCDAF * n) >> 64, (O.mix64(1) * n) >> 64,
                            (O.mix64(2) * n) >> 64]
    # the tensor index enters in the upper word, the call seed by xor
    pos = O.sample_positions(77, 2, 5, 3)
    assert pos.tolist() == [(O.mix64(5 ^ (3 << 32) ^ r) * 77) >> 64 for r in range(2)]
    assert O.call_seed(2, 7) == O.mix64((2 * G + 7) % 2**64)
    # consecutive calls must not draw (nearly) the same positions
    a = set(O.sample_positions(100000, 1000, O.call_seed(5, 0), 0).tolist())
    b = set(O.sample_positions(100000, 1000, O.call_seed(5, 1), 0).tolist())
    assert len(a & b) < 50


def test_positions_are_uniform_over_the_tensor():
    n, S = 1000, 200000
    pos = O.sample_positions(n, S, 12345, 7)
    assert pos.min() >= 0 and pos.max() < n
    counts = np.bincount(pos, minlength=n)
    chi2 = ((counts - S / n) ** 2 / (S / n)).sum()
    assert 800 < chi2 < 1200                              # 999 degrees of freedom: mean 999, sd 45
    # n close to 2^31: still inside the range and spread over it
    big = O.sample_positions((1 << 31) - 5, 10000, 1, 0)
    assert big.min() >= 0 and big.max() < (1 << 31) - 5
    assert (big < (1 << 30)).mean() == pytest.approx(0.5, abs=0.03)
    # other tensors and other calls draw other positions
    assert O.sample_positions(n, 50, 12345, 8).tolist() != pos[:50].tolist()
    assert O.sample_positions(n, 50, 12346, 7).tolist() != pos[:50].tolist()


def test_compress_sampled_is_the_selection_applied_per_tensor():
    """One iteration of the paper-literal mode = clip, Eq. 5, then for every tensor the
    generator's positions fed to the selection; packed output; sent entries masked."""
    rng = np.random.default_rng(43)
    numel = [400000, 64, 9000]
    off = [0, 400384, 400896]
    L = 410112
    s, seed, it = 0.99, 7, 3
    w = O.Worker(off, numel, L, 1, 0.9, 0.0, s)
    g = np.zeros(L, np.float32)
    for o, n in zip(off, numel):
        g[o:o + n] = rng.standard_normal(n).astype(np.float32)
    r, nnz = O.compress_sampled(w, g.copy(), seed=seed, iteration=it)
    exp_idx = []
    for j, (o, n) in enumerate(zip(off, numel)):
        pos = O.sample_positions(n, O.sample_count(n, 0.01), O.call_seed(seed, it), j)
        ref, _ = _numpy_from_sample(g[o:o + n], pos, O.topk_count(n, s), s)
        assert nnz[j] == ref.size
        exp_idx += (ref + o).tolist()
    assert r.idx.tolist() == exp_idx
    assert r.val.tobytes() == g[exp_idx].tobytes()
    assert not w.u[r.idx].any() and not w.v[r.idx].any()
    k = O.topk_count(400000, s)
    assert 0.5 * k < nnz[0] < 1.6 * k                     # 40 of 4000 sampled lie above thr


def test_sampled_selection_outcomes_fewer_more_exact():
    """n = 100000 at 99.9 %: 1000 sampled elements, k_s = 1, so thr is the sample maximum and
    the number of entries above it is roughly geometric with mean k: all three outcomes
    (fewer than k, between k and 2k, precise top-k) occur over 60 calls."""
    rng = np.random.default_rng(53)
    n, s = 100000, 0.999
    k = O.topk_count(n, s)
    g = rng.standard_normal(n).astype(np.float32)
    top = _numpy_topk(g, k)
    kinds = set()
    for it in range(60):
        w = O.Worker([0], [n], n, 1, 0.0, 0.0, s)
        r, nnz = O.compress_sampled(w, g.copy(), seed=5, iteration=it)
        c = int(nnz[0])
        assert c <= 2 * k
        sent = np.zeros(n, bool)
        sent[r.idx] = True
        if c:
            assert np.abs(g[sent]).min() > np.abs(g[~sent]).max()
        if c == k:
            assert r.idx.tolist() == top.tolist()
        kinds.add("exact" if c == k else ("fewer" if c < k else "more"))
    assert kinds == {"exact", "fewer", "more"}
