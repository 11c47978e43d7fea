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
    """Stand-in velocity model on the device (scaffold around the path, not part of it).  Accepts one
    time for the batch or a list with one entry per request (None = that request is not asked)."""

    def __init__(self, target_bf16):
        self.target = target_bf16.float()

    def _t(self, t, like):
        import torch
        if isinstance(t, (list, tuple)):
            return torch.tensor([1.0 if v is None else v for v in t], device=like.device).view(-1, 1, 1)
        return t

    def full(self, x, t, store):
        return ((x.float() - self.target) / self._t(t, x)).to(x.dtype)

    def region(self, x_e, t, edit_idx, n_edit):
        import torch
        B, cap, C = x_e.shape
        idx = edit_idx.long().clamp(0, self.target.shape[1] - 1)
        tgt = torch.gather(self.target, 1, idx.unsqueeze(-1).expand(B, cap, C))
        return ((x_e.float() - tgt) / self._t(t, x_e)).to(x_e.dtype)


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
        act = inp.get("active", list(range(B)))
        if name == "euler":
            for r in range(B):
                if r in act:
                    want = inp["x"][r] - np.float32(inp["dt"][r]).astype(np.float64) * inp["v"][r]
                    assert_close(grab["x"][r], want, f"euler step {k} request {r}")
                else:
                    assert np.array_equal(grab["x"][r], inp["x"][r])         # sat the launch out
        elif name == "partition":
            for r in act:
                p = orc.partition(inp["x"][r:r + 1], inp["v"][r:r + 1], inp["ref"][r:r + 1],
                                  np.float32(inp["t"][r]), metric_o, np.float32(thr))
                assert np.array_equal(grab["mask"][r], p["mask"][0]) and np.array_equal(grab["slot"][r], p["slot"][0])
                assert grab["n_edit"][r] == p["n_edit"][0]
                assert np.array_equal(p["mask"][0].astype(bool), m[r])
        elif name == "decay":
            ne = inp["n_edit"]
            for r in range(B):
                if r in act:
                    want, _ = orc.velocity_decay(inp["v"][r:r + 1], np.float32(inp["scale"][r]),
                                                 np.float32(inp["dt"][r]), inp["x_e"][r:r + 1], ne[r:r + 1])
                    assert_close(grab["x_e"][r, :ne[r]], want[0, :ne[r]], f"region step {k} request {r}")
                else:
                    assert np.array_equal(grab["x_e"][r], inp["x_e"][r])
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


def test_requests_offset_by_three_steps_match_two_independent_oracle_loops():
    """Two requests in one batch, the second one three sampler steps behind the first: their Euler
    updates share launches with per-request time, step length and decay product (a request that has
    no work in a launch sits it out).  Each request must follow exactly the oracle loop run on that
    request alone, and every shared launch is checked per request against the oracle."""
    import torch
    wl, ref, m, target, noise = _case(seed=9, B=2, grid=(20, 20))
    kinds, after = gloop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    cfg = gloop.LoopConfig(kinds, after, ts, [1.0] * (T + 1), 0.05, binding.METRIC_COSINE, 0.9)
    B, N, C = noise.shape
    lp = gloop.RegionELoop(B, N, C, cfg)
    seen = []

    def hook(event, k, tensors):
        if event in ("euler_in", "decay_in"):
            seen.append((event, tuple(tensors["active"])))
            host = {n: (host_f64(v) if isinstance(v, torch.Tensor) else v) for n, v in tensors.items()}
            hook.pending = host
        elif event in ("euler_out", "decay_out"):
            inp, key = hook.pending, ("x" if event == "euler_out" else "x_e")
            got = host_f64(tensors[key])
            for r in range(B):
                if r in inp["active"]:
                    scale = 1.0 if event == "euler_out" else inp["scale"][r]
                    n = N if event == "euler_out" else int(inp["n_edit"][r])
                    want, _ = orc.velocity_decay(inp["v"][r:r + 1], np.float32(scale), np.float32(inp["dt"][r]),
                                                 inp[key][r:r + 1], [n])
                    assert_close(got[r, :n], want[0, :n], f"{event} request {r}")
                else:
                    assert np.array_equal(got[r], inp[key][r])

    lp.hook = hook
    x, trace = lp.run(dev_bf16(noise), dev_bf16(ref), TorchStraightLine(dev_bf16(target)), offsets=[0, 3])
    torch.cuda.synchronize()
    assert int(lp.dev_status[0]) == 0
    # launches were shared whenever both requests had the same kind of work, and split otherwise
    assert any(len(a) == 2 for _, a in seen) and any(len(a) == 1 for _, a in seen)
    got = host_f64(x)
    for r in range(B):
        res = loop_oracle.run_loop(noise[r:r + 1], ref[r:r + 1], loop_oracle.StraightLineModel(target[r:r + 1]),
                                   kinds, after, ts, np.ones(T + 1), 0.05, orc.COSINE, 0.9)
        assert [(k, kind, w) for k, kind, w, _ in trace.per_request[r]] == [(k, kind, w) for k, kind, w, _ in res["log"]]
        for (_, _, _, s_gpu), (_, _, _, s_orc) in zip(trace.per_request[r], res["log"]):
            assert abs(s_gpu - s_orc) < 1e-12
        assert np.max(np.abs(got[r] - res["x"][0])) <= 28 * 2.0 ** -7
        assert np.array_equal(lp.mask[r].cpu().numpy().astype(bool), m[r])
