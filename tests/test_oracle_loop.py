"""Pins of the sampler loop: schedule arithmetic of the two schedules, and what the loop must return
when the velocity model is the exact straight-line field (closed forms, no reference to the CUDA path)."""
import numpy as np
import pytest

from oracle import loop_oracle, regione_oracle as orc
from paper_2510_25590_b200 import loop as gpu_loop      # schedule builders are plain host code
from paper_2510_25590_b200 import synth


def test_paper_schedule_counts_and_order():
    kinds, after = gpu_loop.paper_schedule()
    assert len(kinds) == 28 and after == 6
    assert kinds.count("F") == 9 and kinds.count("R") == 19
    assert kinds == "F" * 6 + "R" * 5 + "F" + "R" * 14 + "F" + "F"
    # the oracle's own statement of the same schedule (written separately) agrees step by step
    want = "".join("R" if kind == "region" else "F" for _, kind in orc.stage_schedule())
    assert kinds == want


def test_alternating_schedule_counts():
    kinds, after = gpu_loop.alternating_schedule()
    full = [k + 1 for k, c in enumerate(kinds) if c == "F"]
    assert full == [1, 2, 3, 4, 5, 6, 11, 16, 21, 26, 27, 28] and after == 6
    assert kinds.count("R") == 16


def _setup(seed=3, B=2, grid=(8, 8), C=16, ratio=0.25):
    wl = synth.scaled_workload(synth.WORKLOADS[1], grid=grid, batch=B)
    lat = synth.make_latents(wl, ratio, stream=seed)
    rng = np.random.default_rng(seed)
    ref = lat["ref"].astype(np.float64)
    m = lat["mask"].astype(bool)
    # target: the reference on unedited tokens, something unrelated on edited ones
    target = np.where(m[..., None], rng.standard_normal(ref.shape), ref)
    noise = rng.standard_normal(ref.shape)
    return wl, ref, m, target, noise


@pytest.mark.parametrize("which", ["paper", "alternating"])
def test_straight_line_model_without_reuse_lands_on_the_target(which):
    wl, ref, m, target, noise = _setup()
    kinds, after = gpu_loop.paper_schedule() if which == "paper" else gpu_loop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    model = loop_oracle.StraightLineModel(target)
    res = loop_oracle.run_loop(noise, ref, model, kinds, after, ts, np.ones(T + 1), -1.0, orc.COSINE, 0.9)
    # delta < 0: never reuse; Euler on a straight line is exact, and so is the one-step prediction
    assert all(w != "reuse" for _, _, w, _ in res["log"])
    assert np.allclose(res["x"], target, atol=1e-12)
    assert np.array_equal(res["partition"]["mask"].astype(bool), m)     # the planted mask is recovered


def test_reuse_pattern_and_decay_scale_of_the_alternating_schedule():
    wl, ref, m, target, noise = _setup()
    kinds, after = gpu_loop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    model = loop_oracle.StraightLineModel(target)
    res = loop_oracle.run_loop(noise, ref, model, kinds, after, ts, np.ones(T + 1), 0.05, orc.COSINE, 0.9)
    region = [(k, w, s) for k, kind, w, s in res["log"] if kind == "R"]
    assert [w for _, w, _ in region] == ["compute", "reuse"] * 8          # every other region step reuses
    assert all(abs(s - (1.0 - 1.0 / T)) < 1e-15 for _, w, s in region if w == "reuse")
    # the last full step runs to t = 0 with dt = t, which lands on the target from anywhere
    assert np.allclose(res["x"], target, atol=1e-12)


def test_reused_steps_leave_the_closed_form_deviation_at_the_end_of_a_run():
    # first run of region steps only (steps 7..10 of the alternating schedule: compute, reuse, compute,
    # reuse), merged at t_10.  With u = x - target and V = noise - target: a computed step keeps u on
    # the line (u = t V k), a reused step applies (1 - dt) times the velocity cached one step earlier,
    # which by direct substitution multiplies k by (1 + dt^2 / t_after).
    wl, ref, m, target, noise = _setup()
    kinds, after = gpu_loop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    model = loop_oracle.StraightLineModel(target)
    res = loop_oracle.run_loop(noise, ref, model, kinds[:10], after, ts[:11], np.ones(T + 1), 0.05, orc.COSINE, 0.9)
    assert [w for _, kind, w, _ in res["log"] if kind == "R"] == ["compute", "reuse", "compute", "reuse"]
    dt, V = 1.0 / T, noise - target
    kappa = (1.0 + dt * dt / ts[8]) * (1.0 + dt * dt / ts[10])
    assert np.allclose(res["x"][m], (target + ts[10] * kappa * V)[m], atol=1e-12)
    # unedited tokens never see the cache: one step over the whole run keeps them exactly on the line
    assert np.allclose(res["x"][~m], (target + ts[10] * V)[~m], atol=1e-12)
