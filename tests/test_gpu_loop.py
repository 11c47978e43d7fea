"""GPU parity of the sampler loop: every library call the loop makes is recomputed by the fp64 oracle
from the inputs the GPU actually saw (teacher forcing), the compute / reuse pattern is compared with
the oracle loop's, and the end state is compared with the oracle loop run on the same model."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, host_f64
from oracle import loop_oracle, regione_oracle as orc
from paper_2510_25590_b200 import binding, loop as gloop, synth

pytestmark = pytest.mark.gpu


class TorchStraightLine:
    """Stand-in velocity model on the device (scaffold around the path, not part of it)."""

    def __init__(self, target_bf16):
        self.target = target_bf16.float()

    def full(self, x, t, store):
        return ((x.float() - self.target) / t).to(x.dtype)

    def region(self, x_e, t, edit_idx, n_edit):
        import torch
        B, cap, C = x_e.shape
        idx = edit_idx.long().clamp(0, self.target.shape[1] - 1)
        tgt = torch.gather(self.target, 1, idx.unsqueeze(-1).expand(B, cap, C))
        return ((x_e.float() - tgt) / t).to(x_e.dtype)


def _case(seed=5, B=2, grid=(24, 24), ratio=0.25, base=1):
    wl = synth.scaled_workload(synth.WORKLOADS[base], grid=grid, batch=B)
    lat = synth.make_latents(wl, ratio, stream=seed)
    rng = np.random.default_rng(seed)
    ref = lat["ref"]
    m = lat["mask"].astype(bool)
    target = synth.bf16_round(np.where(m[..., None], rng.standard_normal(ref.shape), ref).astype(np.float32))
    noise = synth.bf16_round(rng.standard_normal(ref.shape).astype(np.float32))
    return wl, ref, m, target, noise


@pytest.mark.parametrize("which,n_steps,full_size", [("alternating", 28, False), ("alternating", 10, False),
                                                     ("paper", 28, False), ("alternating", 28, True),
                                                     ("paper", 28, True)])
def test_loop_calls_match_oracle_step_by_step(which, n_steps, full_size):
    """full_size: the Step1X-Edit-shaped loop at its own size (64 x 64 latent = 4096 tokens of 16 channels,
    one request, two-ellipse mask of 20 %, per-token L2 threshold 0.1), 28 steps under either schedule."""
    import torch
    if full_size:
        wl, ref, m, target, noise = _case(seed=4, B=1, grid=(64, 64), ratio=0.20, base=4)
        metric_g, metric_o, thr = binding.METRIC_L2, orc.L2, 0.1
    else:
        wl, ref, m, target, noise = _case()
        metric_g, metric_o, thr = binding.METRIC_COSINE, orc.COSINE, 0.9
    kinds, after = gloop.alternating_schedule() if which == "alternating" else gloop.paper_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    kinds, ts = kinds[:n_steps], ts[:n_steps + 1]
    delta = 0.05 if which == "alternating" else 0.04
    cfg = gloop.LoopConfig(kinds, after, ts, [1.0] * (T + 1), delta, metric_g, thr)
    B, N, C = noise.shape
    lp = gloop.RegionELoop(B, N, C, cfg)
    pending = {}
    checked = []

    def hook(event, k, tensors):
        grab = {n: (host_f64(v) if isinstance(v, torch.Tensor) else v) for n, v in tensors.items()}
        if event.endswith("_in"):
            pending[event[:-3]] = grab
            return
        name, inp = event[:-4], pending.pop(event[:-4])
        if name == "euler":
            want = inp["x"] - np.float32(inp["dt"]).astype(np.float64) * inp["v"]
            assert_close(grab["x"], want, f"euler step {k}")
        elif name == "partition":
            p = orc.partition(inp["x"], inp["v"], inp["ref"], np.float32(inp["t"]), metric_o, np.float32(thr))
            assert np.array_equal(grab["mask"], p["mask"]) and np.array_equal(grab["slot"], p["slot"])
            assert np.array_equal(grab["n_edit"], p["n_edit"])
            assert np.array_equal(p["mask"].astype(bool), m)
        elif name == "decay":
            ne = inp["n_edit"]
            want, _ = orc.velocity_decay(inp["v"], np.float32(inp["scale"]), np.float32(inp["dt"]), inp["x_e"], ne)
            for b in range(B):
                assert_close(grab["x_e"][b, :ne[b]], want[b, :ne[b]], f"region step {k}")
        elif name == "merge":
            want = orc.merge(inp["x"], inp["v"], inp["x_e"], inp["slot"].astype(np.int64), np.float32(inp["dt_unedited"]))
            assert_close(grab["x"], want, f"merge before step {k}")
        checked.append(name)

    lp.hook = hook
    x = dev_bf16(noise)
    x, trace = lp.run(x, dev_bf16(ref), TorchStraightLine(dev_bf16(target)))
    torch.cuda.synchronize()
    assert int(lp.dev_status[0]) == 0
    assert {"euler", "partition", "decay", "merge"} <= set(checked)

    res = loop_oracle.run_loop(noise, ref, loop_oracle.StraightLineModel(target), kinds, after, ts,
                               np.ones(T + 1), delta, metric_o, thr)
    assert [(k, kind, w) for k, kind, w, _ in trace.steps] == [(k, kind, w) for k, kind, w, _ in res["log"]]
    for (_, _, _, s_gpu), (_, _, _, s_orc) in zip(trace.steps, res["log"]):
        assert abs(s_gpu - s_orc) < 1e-12
    assert trace.model_region_calls == sum(1 for _, _, w, _ in res["log"] if w == "compute")
    # end state: bf16 rounding of the latent after each of up to 28 steps accumulates, so the bound
    # is looser than for a single call (each step adds at most half a bf16 ulp of |x| <= ~4)
    got = host_f64(x)
    assert np.max(np.abs(got - res["x"])) <= 28 * 2.0 ** -7
    rel = np.sqrt(np.mean((got - res["x"]) ** 2)) / np.sqrt(np.mean(res["x"] ** 2))
    assert rel <= 3e-2, rel
