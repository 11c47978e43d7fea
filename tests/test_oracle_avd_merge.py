"""Pins for the oracle's AVDCache, Euler update, merge and stage schedule (CPU only)."""
import numpy as np

from oracle import regione_oracle as orc


def test_gamma_one_reduces_to_solver_product():
    # Appendix (analysis of AVDCache): with gamma = 1 the decay is prod (1 - dt); uniform steps
    # of 1/T give (1 - 1/T)^k.
    T = 28
    p = 1.0
    for k in range(1, 8):
        p, reuse = orc.avd_step(p, 1.0 / T, 1.0, delta=0.99)
        assert reuse and abs(p - (1 - 1 / T) ** k) < 1e-15


def test_residual_cache_equals_decayed_velocity_cache():
    # Appendix: caching Delta = v - X and reusing it after an Euler step gives v' = (1 - dt) v.
    rng = np.random.default_rng(0)
    x, v = rng.standard_normal((2, 5, 16))
    ts = [0.8, 0.75, 0.7, 0.62]
    prod = 1.0
    v_cur, x_cur = v.copy(), x.copy()
    for a, b in zip(ts[:-1], ts[1:]):
        delta_res = v_cur - x_cur
        x_cur = x_cur - (a - b) * v_cur
        v_cur = x_cur + delta_res
        prod, reuse = orc.avd_step(prod, a - b, 1.0, delta=10.0)
        assert reuse
        assert np.max(np.abs(v_cur - prod * v)) < 1e-14


def test_delta_extremes_and_monotone_criterion():
    T = 28
    ts = np.arange(T + 1) / T
    g = 0.9 + 0.1 * np.random.default_rng(1).random(T + 1)
    always = orc.avd_schedule(ts, g, -1.0, 22, 18)
    assert [r for _, r, _ in always] == [False] * 5
    never = orc.avd_schedule(ts, g, 1.0, 22, 3)
    assert [r for _, r, _ in never] == [False] + [True] * 19
    scales = [s for _, _, s in never[1:]]
    assert all(b < a for a, b in zip(scales, scales[1:]))          # criterion 1 - P non-decreasing
    # hand-computed: uniform steps, gamma = 1, delta = 0.05 -> compute, reuse, compute, reuse ...
    alt = orc.avd_schedule(ts, np.ones(T + 1), 0.05, 10, 5)
    assert [r for _, r, _ in alt] == [False, True, False, True, False, True]
    assert abs(alt[1][2] - (1 - 1 / 28)) < 1e-15
    # decay-factor equation with gamma: scale is (1 - dt) * gamma at the first reuse
    one = orc.avd_schedule(ts, np.full(T + 1, 0.99), 0.06, 10, 9)
    assert one[1][1] and abs(one[1][2] - (1 - 1 / 28) * 0.99) < 1e-15


def test_velocity_decay_is_the_euler_update():
    rng = np.random.default_rng(2)
    x, v = rng.standard_normal((2, 2, 6, 4))
    xn, vu = orc.velocity_decay(v, 0.5, 0.25, x, [6, 2])
    assert np.allclose(vu, 0.5 * v, atol=0, rtol=0)
    assert np.max(np.abs(xn[0] - (x[0] - 0.125 * v[0]))) < 1e-15
    assert np.array_equal(xn[1, 2:], x[1, 2:]) and np.max(np.abs(xn[1, :2] - (x[1, :2] - 0.125 * v[1, :2]))) < 1e-15
    # scale 1 on a straight line lands on the line: X_{t-dt} = (1-(t-dt)) X0 + (t-dt) X1
    X0, X1 = rng.standard_normal((2, 1, 6, 4))
    t, dt = 0.7, 0.1
    xn, _ = orc.velocity_decay(X1 - X0, 1.0, dt, (1 - t) * X0 + t * X1, [6])
    assert np.max(np.abs(xn - ((1 - (t - dt)) * X0 + (t - dt) * X1))) < 1e-15


def test_merge_special_cases():
    rng = np.random.default_rng(3)
    B, N, C = 2, 21, 4
    x, v = rng.standard_normal((2, B, N, C))
    xe = rng.standard_normal((B, N, C))
    none = np.full((B, N), -1, np.int32)
    assert np.max(np.abs(orc.merge(x, v, xe, none, 0.3) - (x - 0.3 * v))) < 1e-15     # zero-edit mask
    full = np.broadcast_to(np.arange(N, dtype=np.int32), (B, N))
    assert np.array_equal(orc.merge(x, v, xe, full, 0.3), xe)                          # full mask
    # mixed, against partition's slot; unedited straight-line tokens land on the line
    X0, X1 = rng.standard_normal((2, B, N, C))
    t, tf = 22 / 28, 17 / 28
    m = (rng.random((B, N)) < 0.4)
    slot = np.stack([orc.compact_indices(m[b])[2] for b in range(B)])
    out = orc.merge((1 - t) * X0 + t * X1, X1 - X0, xe, slot, t - tf)
    line = (1 - tf) * X0 + tf * X1
    for b in range(B):
        assert np.max(np.abs(out[b, ~m[b]] - line[b, ~m[b]])) < 1e-14
        assert np.array_equal(out[b, m[b]], xe[b, :m[b].sum()])


def test_stage_schedule_counts():
    # Implementation details: T = 28, six stabilization steps, forced update at 16, two smooth steps.
    s = orc.stage_schedule(28, 6, (16,), 2)
    assert [i for i, _ in s] == list(range(28, 0, -1))
    kinds = [k for _, k in s]
    assert kinds.count("region") == 19 and kinds.count("full") + kinds.count("full_store") == 9
    assert kinds[:6] == ["full"] * 5 + ["full_store"]
    assert dict(s)[17] == "full_store" and dict(s)[2] == "full_store" and dict(s)[1] == "full"
    assert all(dict(s)[j] == "region" for j in list(range(22, 17, -1)) + list(range(16, 2, -1)))


def test_gamma_fit_recovers_planted_corrections_and_reduces_to_one_for_the_residual_cache():
    # Appendix: under residual caching v_{i} = (1 - dt_i) v_{i+1}, i.e. gamma = 1; a planted extra
    # factor g_i per step must come back exactly, whatever the direction and scale of the samples
    rng = np.random.default_rng(3)
    S, T, n = 5, 7, 64
    dt = rng.uniform(0.01, 0.1, T)
    g = rng.uniform(0.9, 1.0, T)
    v = np.empty((S, T + 1, n))
    v[:, T] = rng.standard_normal((S, n)) * rng.uniform(0.5, 3.0, (S, 1))
    for i in range(T - 1, -1, -1):
        v[:, i] = (1.0 - dt[i]) * g[i] * v[:, i + 1]
    norms, gamma = orc.gamma_fit(v, dt)
    assert np.allclose(gamma, g, rtol=1e-12)
    assert np.allclose(norms[:, 0] / norms[:, T], np.prod((1 - dt) * g), rtol=1e-12)
    _, gamma1 = orc.gamma_fit(v / g.prod(), dt)                     # a global rescale changes nothing
    assert np.allclose(gamma1, g, rtol=1e-12)
    # brute force on one entry
    i = 3
    want = np.mean([np.linalg.norm(v[s, i]) / np.linalg.norm(v[s, i + 1]) for s in range(S)]) / (1 - dt[i])
    assert abs(gamma[i] - want) < 1e-14
