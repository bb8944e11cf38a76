"""The synthetic gradient generator: shapes of the paper's models, determinism,
and the stated value distributions."""
import json
import os

import numpy as np

from paper_1712_01887_b200 import inputs as I


def test_model_sizes(golden_dir):
    with open(os.path.join(golden_dir, "model_sizes.json")) as f:
        G = json.load(f)
    r = I.workload("resnet50")
    assert len(r.shapes) == G["resnet50"]["tensors"] and r.total == G["resnet50"]["total"]
    assert round(r.total * 4 / 2 ** 20, 2) == G["resnet50"]["mib"]
    l = I.workload("lstm")
    assert len(l.shapes) == G["lstm"]["tensors"] and l.total == G["lstm"]["total"]
    d = I.workload("deepspeech")
    assert len(d.shapes) == G["deepspeech"]["tensors"] and d.total == G["deepspeech"]["total"]
    sizes = sorted(r.numel)
    assert sizes[0] == 64 and sizes[-1] == 2359296
    assert sizes.count(64) == 14 and sizes.count(262144) == 11 and sizes.count(2359296) == 3


def test_fill_is_deterministic_and_worker_dependent():
    wl = I.workload("cfg1")
    off, L = I.packed_layout(wl.numel, align=512)
    a = np.zeros(L, np.float32)
    b = np.zeros(L, np.float32)
    I.fill(wl, a, off, worker=1, iteration=2)
    I.fill(wl, b, off, worker=1, iteration=2)
    assert a.tobytes() == b.tobytes()
    I.fill(wl, b, off, worker=2, iteration=2)
    assert a.tobytes() != b.tobytes()
    I.fill(wl, b, off, worker=1, iteration=3)
    assert a.tobytes() != b.tobytes()
    # N(0,1e-3) bulk with 1% Laplace(0,1e-2) outliers: norm about 1.77 as the design notes state
    assert 1.5 < np.linalg.norm(a.astype(np.float64)) < 2.0
    assert 0.005 < np.mean(np.abs(a) > 5e-3) < 0.012


def test_layout_gaps_untouched_and_lstm_rows_sparse():
    wl = I.workload("lstm_small")
    off, L = I.packed_layout(wl.numel, align=512)
    assert all(o % 512 == 0 for o in off) and L % 512 == 0
    a = np.full(L, np.float32(7.0))
    I.fill(wl, a, off, worker=0, iteration=0)
    valid = np.zeros(L, bool)
    for o, n in zip(off, wl.numel):
        valid[o:o + n] = True
    assert np.all(a[~valid] == 7.0)
    rows, cols = wl.shapes[0]
    emb = a[off[0]:off[0] + rows * cols].reshape(rows, cols)
    live = np.any(emb != 0, axis=1)
    assert 0.005 < live.mean() < 0.05
    assert np.all(emb[~live] == 0) and not np.signbit(emb[~live]).any()


def test_resnet_sigma_range_and_student_t_tail():
    r = I.workload("resnet50")
    assert r.sigma.shape == (161,) and r.sigma.min() >= 1e-5 and r.sigma.max() <= 1e-2
    d = I.workload("deepspeech_small")
    off, L = I.packed_layout(d.numel, align=1)
    a = np.zeros(L, np.float32)
    I.fill(d, a, off, worker=0, iteration=0)
    x = a / 1e-4
    # Student-t(3): P(|t| > 3.182) = 0.05
    assert 0.045 < np.mean(np.abs(x) > 3.182) < 0.055
