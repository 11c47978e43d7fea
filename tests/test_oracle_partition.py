"""Pins for the oracle's Adaptive Region Partition (CPU only)."""
import math

import numpy as np
import pytest

from oracle import regione_oracle as orc
from paper_2510_25590_b200 import synth


def test_worked_values_from_fixture():
    # tests/golden/partition_closed_forms.txt: hand-derived closed forms (3-4-5 triangles).
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "partition_closed_forms.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    for metric, x0, x1, r0, r1, num, den in rows:
        s = orc.token_score(np.array([[float(x0), float(x1)]]), np.array([[float(r0), float(r1)]]),
                            orc.COSINE if metric == "cos" else orc.L2)
        want = float(num) / float(den) if metric == "cos" else math.sqrt(float(num)) / float(den)
        assert abs(s[0] - want) < 1e-15


def test_straight_line_velocity_recovers_target_exactly():
    # Rectified flow: X_t = (1-t) X0 + t X1 and v = X1 - X0  =>  X_t - t v = X0.
    rng = np.random.default_rng(0)
    X0, X1 = rng.standard_normal((2, 3, 50, 16))
    for t in (0.1, 22 / 28, 1.0):
        x_t = (1 - t) * X0 + t * X1
        x0_hat = orc.one_step_estimate(x_t, t, X1 - X0)
        assert np.max(np.abs(x0_hat - X0)) < 1e-14
        p = orc.partition(x_t, X1 - X0, X0, t, orc.COSINE, 0.93)
        assert np.all(np.abs(p["score"] - 1.0) < 1e-12)
        assert p["n_edit"].tolist() == [0, 0, 0] and not p["mask"].any()
        p = orc.partition(x_t, X1 - X0, X0, t, orc.L2, 0.1)
        assert np.all(p["score"] < 1e-12) and p["n_edit"].tolist() == [0, 0, 0]


def test_euler_invariance_of_estimate():
    # x0_hat from (X_t, t) equals x0_hat from (X_t - dt v, t - dt) for the same v.
    rng = np.random.default_rng(1)
    x, v = rng.standard_normal((2, 4, 16))
    t, dt = 0.8, 1 / 28
    a = orc.one_step_estimate(x, t, v)
    b = orc.one_step_estimate(x - dt * v, t - dt, v)
    assert np.max(np.abs(a - b)) < 1e-14


def test_sign_of_the_velocity_term():
    # a wrong sign (x + t v) must fail: x=1, v=2, t=0.5 -> 0
    assert orc.one_step_estimate(np.array([1.0]), 0.5, np.array([2.0]))[0] == 0.0


def test_cosine_special_cases():
    a = np.array([[1.0, -2.0, 3.0, 0.5]])
    assert abs(orc.token_score(a, a, orc.COSINE)[0] - 1) < 1e-15
    assert abs(orc.token_score(a, -a, orc.COSINE)[0] + 1) < 1e-15
    assert abs(orc.token_score(a, 7.0 * a, orc.COSINE)[0] - 1) < 1e-15   # scale invariant
    orth = np.array([[2.0, 1.0, 0.0, 0.0]])
    assert abs(orc.token_score(a, orth, orc.COSINE)[0]) < 1e-15
    assert orc.token_score(np.zeros((1, 4)), a, orc.COSINE)[0] == 0.0     # clamped denominator


def test_threshold_polarity_and_ties():
    s = np.array([0.5, 0.93, 0.95])
    assert orc.edit_mask(s, orc.COSINE, 0.93).tolist() == [1, 1, 0]      # similar > eta => unedited
    d = np.array([0.05, 0.1, 0.2])
    assert orc.edit_mask(d, orc.L2, 0.1).tolist() == [0, 0, 1]           # far > tau => edited


def _brute_partition(x_t, v, ref, t, metric, thr):
    """Independent pure-Python loops with the math module."""
    N, C = len(x_t), len(x_t[0])
    mask, e, k, slot = [], [], [], []
    for n in range(N):
        dot = xx = rr = dd = 0.0
        for c in range(C):
            h = x_t[n][c] - t * v[n][c]
            dot += h * ref[n][c]
            xx += h * h
            rr += ref[n][c] * ref[n][c]
            dd += (h - ref[n][c]) ** 2
        if metric == "cos":
            s = dot / max(math.sqrt(xx) * math.sqrt(rr), 1e-12)
            m = 0 if s > thr else 1
        else:
            m = 1 if math.sqrt(dd) > thr else 0
        mask.append(m)
        if m:
            slot.append(len(e)); e.append(n)
        else:
            slot.append(-1); k.append(n)
    return mask, e, k, slot


@pytest.mark.parametrize("metric,thr", [("cos", 0.2), ("l2", 5.0)])
def test_brute_force_tiny(metric, thr):
    rng = np.random.default_rng(2)
    x, v, r = rng.standard_normal((3, 1, 61, 8))
    t = 0.7
    p = orc.partition(x, v, r, t, orc.COSINE if metric == "cos" else orc.L2, thr)
    mask, e, k, slot = _brute_partition(x[0].tolist(), v[0].tolist(), r[0].tolist(), t, metric, thr)
    assert 0 < len(e) < 61
    assert p["mask"][0].tolist() == mask
    assert p["n_edit"][0] == len(e)
    assert p["edit_idx"][0, :len(e)].tolist() == e
    assert p["keep_idx"][0, :len(k)].tolist() == k
    assert p["slot"][0].tolist() == slot


def _check_index_invariants(p, b=0):
    mask = p["mask"][b].astype(bool)
    N = mask.shape[0]
    ne = int(p["n_edit"][b])
    e, k, slot = p["edit_idx"][b, :ne], p["keep_idx"][b, :N - ne], p["slot"][b]
    assert ne == int(mask.sum())
    assert np.all(np.diff(e) > 0) and np.all(np.diff(k) > 0)
    assert np.array_equal(np.sort(np.concatenate([e, k])), np.arange(N))
    assert np.array_equal(slot[e], np.arange(ne))
    assert np.all(slot[k] == -1)
    assert np.all(mask[e]) and not np.any(mask[k])


CASES = [(1, None), (2, None), (3, 0.05), (3, 0.10), (3, 0.25), (3, 0.50), (3, 1.00), (4, None),
         (5, None)]


@pytest.mark.parametrize("cfg,ratio", CASES)
def test_planted_mask_is_recovered_with_margin(cfg, ratio):
    wl = synth.WORKLOADS[cfg]
    lat = synth.make_latents(wl, ratio)
    metric = orc.COSINE if wl.metric == "cosine" else orc.L2
    p = orc.partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], metric, wl.threshold)
    assert np.array_equal(p["mask"], lat["mask"])
    # every token stays at least 1e-3 (relative) away from the threshold
    assert np.min(np.abs(p["score"] - wl.threshold)) >= 1e-3 * abs(wl.threshold)
    want = round((wl.ratios[0] if ratio is None else ratio) * wl.n_img)
    for b in range(wl.batch):
        assert abs(int(p["n_edit"][b]) - want) <= 1
        _check_index_invariants(p, b)


def test_all_zero_and_all_one_masks():
    for m in (np.zeros(17, np.uint8), np.ones(17, np.uint8)):
        e, k, slot, ne = orc.compact_indices(m)
        assert ne == int(m.sum())
        if ne:
            assert e.tolist() == list(range(17)) and slot.tolist() == list(range(17))
        else:
            assert k.tolist() == list(range(17)) and np.all(slot == -1)


def test_morphology_matches_library_and_removes_speckle():
    from scipy import ndimage as ndi
    rng = np.random.default_rng(3)
    grid = (12, 9)
    m = (rng.random(grid) < 0.45).astype(np.uint8)
    st = np.ones((3, 3), bool)
    er = lambda a: ndi.binary_erosion(a, st, border_value=1)
    di = lambda a: ndi.binary_dilation(a, st, border_value=0)
    want = er(di(di(er(m.astype(bool))))).astype(np.uint8)
    got = orc.open_close(m.reshape(-1), grid).reshape(grid)
    assert np.array_equal(got, want)
    # an isolated edited pixel disappears (opening); a one-pixel hole is filled (closing)
    a = np.zeros((9, 9), np.uint8); a[4, 4] = 1
    assert not orc.open_close(a.reshape(-1), (9, 9)).any()
    b = np.ones((9, 9), np.uint8); b[4, 4] = 0
    assert orc.open_close(b.reshape(-1), (9, 9)).all()
    # a solid 5x5 block survives unchanged
    c = np.zeros((9, 9), np.uint8); c[2:7, 2:7] = 1
    assert np.array_equal(orc.open_close(c.reshape(-1), (9, 9)).reshape(9, 9), c)
