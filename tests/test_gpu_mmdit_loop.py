"""The sampler loop around the stand-in transformer stack (the Step1X-Edit-shaped configuration, reduced
in size so that the fp64 oracle finishes in seconds): the stack's full and region steps against the
oracle's on the same inputs, and the whole 28-step loop against the oracle loop."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, host_f64
from oracle import loop_oracle, mmdit_oracle, regione_oracle as orc
from paper_2510_25590_b200 import binding, loop as gloop, synth
from paper_2510_25590_b200.mmdit_scaffold import MMDiTScaffold

pytestmark = pytest.mark.gpu

H, D, C, L, N_TEXT = 2, 128, 16, 2, 40


def _setup(grid=(16, 16), seed=3, membership="paper"):
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[4], grid=grid, n_text=N_TEXT, heads=H)
    lat = synth.make_latents(wl, 0.20, stream=seed)
    ref, planted = lat["ref"], lat["mask"].astype(bool)
    n_img = wl.n_img
    w = synth.make_mmdit_weights(H * D, D, C, N_TEXT, L, seed=seed)
    cos, sin = synth.rope_tables(N_TEXT + 2 * n_img, D)
    om = mmdit_oracle.MMDiTOracle(w, N_TEXT, n_img, n_img, H, D, L, cos, sin, ref, planted, membership)
    gm = MMDiTScaffold({k: dev_bf16(v) for k, v in w.items()}, N_TEXT, n_img, n_img, H, D, L,
                       torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda(), dev_bf16(ref),
                       torch.from_numpy(planted).cuda(),
                       binding.ROWS_PAPER if membership == "paper" else binding.ROWS_EDITED_QUERIES)
    rng = np.random.default_rng(seed)
    noise = synth.bf16_round(rng.standard_normal(ref.shape).astype(np.float32))
    return wl, om, gm, ref, planted, noise


def _rel(got, want):
    return float(np.sqrt(np.mean((got - want) ** 2)) / np.sqrt(np.mean(want ** 2)))


@pytest.mark.parametrize("membership", ["paper", "edited_queries"])
def test_full_and_region_steps_of_the_stack_match_the_oracle(membership):
    """Same latent, same time, same weights: the velocity of a full step, the K / V it keeps, and the
    velocity of a region step against those, each against the oracle's.  The stack's own arithmetic is bf16
    (library GEMMs of the scaffold), so the velocity is compared loosely and the latent after the Euler
    step, which is what the method hands on, at the stated tolerance."""
    import torch
    wl, om, gm, ref, planted, x = _setup(membership=membership)
    n_img = wl.n_img
    t, dt = 0.75, 1.0 / 28.0
    lp = gloop.RegionELoop(1, n_img, C, gloop.LoopConfig("F", 1, [t, t - dt], [1.0, 1.0], 0.05, binding.METRIC_L2, 0.1))
    gm.bind(lp)
    v_gpu = gm.full(dev_bf16(x), t, True)
    v_orc = om.full(x, t)
    assert _rel(host_f64(v_gpu), v_orc) < 3e-2
    assert_close(x - dt * host_f64(v_gpu), x - dt * v_orc, "latent after a full step")
    for l in range(L):                                          # what the blocks keep: K and V as they entered the softmax
        assert _rel(host_f64(gm.k_full[l]), om.k_full[l]) < 2e-2 and _rel(host_f64(gm.v_full[l]), om.v_full[l]) < 2e-2
    # the partition on the oracle's velocity recovers the planted mask; the same lists drive both region steps
    p = orc.partition(x, synth.bf16_round(v_orc.astype(np.float32)), ref, np.float32(t), orc.L2, np.float32(0.1))
    assert np.array_equal(p["mask"].astype(bool), planted)
    binding.partition(dev_bf16(x), v_gpu, dev_bf16(ref), t, binding.METRIC_L2, 0.1, lp.mask, lp.edit_idx, lp.keep_idx,
                      lp.slot, lp.n_edit)
    assert np.array_equal(lp.mask.cpu().numpy().astype(bool), planted)
    ne = int(p["n_edit"][0])
    x_e = np.zeros_like(x); x_e[0, :ne] = x[0, p["edit_idx"][0, :ne]] * 0.9
    x_e = synth.bf16_round(x_e.astype(np.float32))
    t2 = t - dt
    ve_gpu = gm.region(dev_bf16(x_e), t2, lp.edit_idx, lp.n_edit)
    ve_orc = om.region(x_e, t2, p["edit_idx"], p["n_edit"])
    torch.cuda.synchronize()
    assert int(gm.dev_status[0]) == 0
    assert _rel(host_f64(ve_gpu)[0, :ne], ve_orc[0, :ne]) < 3e-2
    assert_close(x_e[0, :ne] - dt * host_f64(ve_gpu)[0, :ne], x_e[0, :ne] - dt * ve_orc[0, :ne], "region latent after the step")
    assert np.all(host_f64(ve_gpu)[0, ne:] == 0.0)


def test_region_step_on_unchanged_inputs_reproduces_the_full_step_on_the_gpu():
    """The method's premise, on the device: with nothing changed since the full step, recomputing only the
    region against the kept K / V gives the full step's velocity there (up to the bf16 of the stack)."""
    import torch
    wl, om, gm, ref, planted, x = _setup()
    lp = gloop.RegionELoop(1, wl.n_img, C, gloop.LoopConfig("F", 1, [0.7, 0.6], [1.0, 1.0], 0.05, binding.METRIC_L2, 0.1))
    gm.bind(lp)
    xd = dev_bf16(x)
    v = gm.full(xd, 0.7, True)
    binding.partition(xd, v, dev_bf16(ref), 0.7, binding.METRIC_L2, 0.1, lp.mask, lp.edit_idx, lp.keep_idx, lp.slot, lp.n_edit)
    ne = int(lp.n_edit[0])
    x_e = torch.zeros_like(xd); x_e[0, :ne] = xd[0, lp.edit_idx[0, :ne].long()]
    v_e = gm.region(x_e, 0.7, lp.edit_idx, lp.n_edit)
    want = host_f64(v)[0, lp.edit_idx[0, :ne].cpu().numpy()]
    assert _rel(host_f64(v_e)[0, :ne], want) < 1e-2


def test_28_step_loop_around_the_stack_matches_the_oracle_loop():
    import torch
    wl, om, gm, ref, planted, noise = _setup(seed=5)
    kinds, after = gloop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    cfg = gloop.LoopConfig(kinds, after, ts, [1.0] * (T + 1), 0.05, binding.METRIC_L2, 0.1)
    lp = gloop.RegionELoop(1, wl.n_img, C, cfg)
    gm.bind(lp)
    x, trace = lp.run(dev_bf16(noise), dev_bf16(ref), gm)
    torch.cuda.synchronize()
    assert int(lp.dev_status[0]) == 0 and int(gm.dev_status[0]) == 0
    res = loop_oracle.run_loop(noise, ref, om, kinds, after, ts, np.ones(T + 1), 0.05, orc.L2, 0.1)
    assert [(k, kind, w) for k, kind, w, _ in trace.steps] == [(k, kind, w) for k, kind, w, _ in res["log"]]
    assert np.array_equal(lp.mask.cpu().numpy().astype(bool), planted)
    assert np.array_equal(res["partition"]["mask"].astype(bool), planted)
    assert trace.model_region_calls == sum(1 for _, _, w, _ in res["log"] if w == "compute") > 0
    got = host_f64(x)
    rel = _rel(got, res["x"])
    print(f"28-step loop around the stack: end-state rel-RMS {rel:.3e}, max-abs {np.max(np.abs(got - res['x'])):.3e}")
    assert rel <= 3e-2
