"""GPU parity: the whole region-aware step (every hot-path stage chained) against the oracle chain."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, host_f64
from oracle import step_oracle
from paper_2510_25590_b200 import binding, synth
from paper_2510_25590_b200.step import RegionStep, StepShapes, plan_capacity

pytestmark = pytest.mark.gpu


def run_step(wl, membership="edited_queries", ratio=None):
    import torch
    lat = synth.make_latents(wl, ratio)
    qkv = synth.make_qkv_full(wl)
    t, scale, dt, dt_u = lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0
    d = {k: dev_bf16(lat[k]) for k in ("x_t", "v", "ref")}
    dq, dk, dv = (dev_bf16(qkv[k]) for k in ("q", "k", "v"))
    metric = binding.METRIC_COSINE if wl.metric == "cosine" else binding.METRIC_L2
    cap = plan_capacity(d["x_t"], d["v"], d["ref"], t, metric, wl.threshold)
    shp = StepShapes(wl.batch, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads, wl.head_dim, cap,
                     metric, wl.threshold,
                     binding.ROWS_PAPER if membership == "paper" else binding.ROWS_EDITED_QUERIES)
    step = RegionStep(shp)
    step.o_full.fill_(0)
    step.run(d["x_t"], d["v"], d["ref"], dq, dk, dv, t, scale, dt, dt_u)
    torch.cuda.synchronize()
    assert int(step.dev_status[0]) == 0
    want = step_oracle.region_step(wl, lat, qkv, t, np.float32(scale), np.float32(dt), np.float32(dt_u),
                                   membership)
    p = want["partition"]
    assert np.array_equal(step.mask.cpu().numpy(), p["mask"])
    assert np.array_equal(step.n_edit.cpu().numpy(), p["n_edit"])
    assert np.array_equal(step.slot.cpu().numpy(), p["slot"])
    assert np.array_equal(step.n_q.cpu().numpy(), want["n_q"])
    assert np.array_equal(step.n_cache.cpu().numpy(), want["n_cache"])
    for b in range(wl.batch):
        nq, nc = int(want["n_q"][b]), int(want["n_cache"][b])
        assert np.array_equal(step.query_rows[b, :nq].cpu().numpy(), want["query_rows"][b, :nq])
        assert np.array_equal(step.cache_rows[b, :nc].cpu().numpy(), want["cache_rows"][b, :nc])
        assert np.array_equal(host_f64(step.k_cache[b, :nc]), want["k_cache"][b, :nc])      # copies: bit-exact
        assert np.array_equal(host_f64(step.v_cache[b, :nc]), want["v_cache"][b, :nc])
        o_rows = step.o_full[b][step.query_rows[b, :nq].long()]      # attention rows, where the step put them
        assert_close(host_f64(o_rows), want["o_e"][b, :nq], "attention rows")
        ne = int(p["n_edit"][b])
        assert_close(host_f64(step.x_e[b, :ne]), want["x_e"][b, :ne], "x_e")
    assert_close(host_f64(step.o_full), want["o_full"], "scattered attention output")
    assert_close(host_f64(step.x_out), want["x_out"], "merged latents")


def test_config1_whole_step():
    run_step(synth.WORKLOADS[1])


def test_config1_whole_step_paper_membership():
    run_step(synth.WORKLOADS[1], membership="paper")


def test_config5_shape_small_batch_of_four():
    run_step(synth.scaled_workload(synth.WORKLOADS[5], grid=(24, 24), n_text=48, heads=4))


def test_config4_shape_small_l2_metric():
    run_step(synth.scaled_workload(synth.WORKLOADS[4], grid=(24, 24), n_text=32, heads=4), membership="paper")


def test_zero_edit_mask_is_one_step_prediction_everywhere():
    run_step(synth.scaled_workload(synth.WORKLOADS[2], grid=(16, 16), n_text=16, heads=2), ratio=0.0)


def test_step_that_reuses_the_cache_of_an_earlier_step():
    """Algorithm 1 refreshes the cache at full steps only: a step run with ``store_cache=False`` after a
    storing step, on new Q / K / V of a later sampler step, attends over the fresh rows of the new tensors
    and the cached rows of the old ones (oracle: attention with the first step's cache), in 7 launches."""
    import torch
    from oracle import regione_oracle as orc
    wl = synth.scaled_workload(synth.WORKLOADS[2], grid=(24, 24), n_text=70, heads=4)
    lat = synth.make_latents(wl)
    old, new = synth.make_qkv_full(wl), synth.make_qkv_full(wl, stream=1)
    t, scale, dt, dt_u = lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0
    d = {k: dev_bf16(lat[k]) for k in ("x_t", "v", "ref")}
    cap = plan_capacity(d["x_t"], d["v"], d["ref"], t, binding.METRIC_COSINE, wl.threshold)
    step = RegionStep(StepShapes(wl.batch, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads, wl.head_dim,
                                 cap, binding.METRIC_COSINE, wl.threshold, binding.ROWS_EDITED_QUERIES))
    step.run(d["x_t"], d["v"], d["ref"], *(dev_bf16(old[k]) for k in ("q", "k", "v")), t, scale, dt, dt_u)
    before = step.launches
    step.o_full.fill_(0)
    step.run(d["x_t"], d["v"], d["ref"], *(dev_bf16(new[k]) for k in ("q", "k", "v")), t, scale, dt, dt_u,
             store_cache=False)
    torch.cuda.synchronize()
    assert int(step.dev_status[0]) == 0 and step.launches - before == 7
    rows = orc.region_rows(lat["mask"][0], wl.n_text, wl.n_ref, "edited_queries")
    nq, nc = len(rows["query"]), len(rows["cache"])
    assert int(step.n_q[0]) == nq and int(step.n_cache[0]) == nc
    assert np.array_equal(host_f64(step.k_cache[0, :nc]), old["k"][0, rows["cache"]].astype(np.float64))
    want = orc.region_attention(new["q"][:, rows["query"]], new["k"][:, rows["fresh"]], new["v"][:, rows["fresh"]],
                                old["k"][:, rows["cache"]], old["v"][:, rows["cache"]], [nq], [nq], [nc])
    got = host_f64(step.o_full[0][step.query_rows[0, :nq].long()])
    assert_close(got, want[0, :nq], "attention over the earlier step's cache")


def test_step_replayed_from_a_cuda_graph_matches_the_eager_step():
    """The launches of a step (each with programmatic stream serialization, two streams) captured into a
    CUDA graph and replayed give bit-identical buffers to the same step launched eagerly."""
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[2], grid=(24, 24), n_text=70)
    lat = synth.make_latents(wl)
    qkv = synth.make_qkv_full(wl)
    t, scale, dt, dt_u = lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0
    d = {k: dev_bf16(lat[k]) for k in ("x_t", "v", "ref")}
    dq, dk, dv = (dev_bf16(qkv[k]) for k in ("q", "k", "v"))
    cap = plan_capacity(d["x_t"], d["v"], d["ref"], t, binding.METRIC_COSINE, wl.threshold)
    shp = StepShapes(wl.batch, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads, wl.head_dim, cap,
                     binding.METRIC_COSINE, wl.threshold, binding.ROWS_EDITED_QUERIES)
    step = RegionStep(shp)
    names = ("mask", "slot", "n_edit", "k_cache", "v_cache", "o_full", "x_e", "x_out")
    def run():
        step.run(d["x_t"], d["v"], d["ref"], dq, dk, dv, t, scale, dt, dt_u)
    step.o_full.fill_(0)
    run()                                   # eager (also the first-call set-up, outside any capture)
    torch.cuda.synchronize()
    eager = {n: getattr(step, n).clone() for n in names}
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            run()
    for n in names:
        getattr(step, n).zero_()
    torch.cuda.synchronize()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert int(step.dev_status[0]) == 0
    for n in names:
        a, b = eager[n], getattr(step, n)
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), n


def test_guidance_pair_two_batch_entries_sharing_one_mask():
    """Classifier-free guidance evaluates the model twice per step (the paper's editors run with guidance
    scales 6, 2.5 and 4): the conditional and the unconditional branch are two batch entries with the same
    latent, hence the same edit mask and index lists, but their own Q / K / V.  One launch of every stage
    serves both; each entry must match the oracle on its own inputs."""
    import torch
    base = synth.scaled_workload(synth.WORKLOADS[2], grid=(24, 24), n_text=40, heads=3)
    wl = synth.scaled_workload(base, batch=2)
    one = synth.make_latents(base)
    lat = {k: (np.concatenate([one[k], one[k]]) if isinstance(one[k], np.ndarray) else one[k]) for k in one}
    qkv = synth.make_qkv_full(wl)                       # two different Q / K / V sets
    assert not np.array_equal(qkv["q"][0], qkv["q"][1])
    t, scale, dt, dt_u = lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0
    d = {k: dev_bf16(lat[k]) for k in ("x_t", "v", "ref")}
    dq, dk, dv = (dev_bf16(qkv[k]) for k in ("q", "k", "v"))
    cap = plan_capacity(d["x_t"], d["v"], d["ref"], t, binding.METRIC_COSINE, wl.threshold)
    step = RegionStep(StepShapes(2, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads, wl.head_dim, cap,
                                 binding.METRIC_COSINE, wl.threshold, binding.ROWS_EDITED_QUERIES))
    step.run(d["x_t"], d["v"], d["ref"], dq, dk, dv, t, scale, dt, dt_u)
    torch.cuda.synchronize()
    assert int(step.dev_status[0]) == 0
    assert torch.equal(step.mask[0], step.mask[1]) and torch.equal(step.query_rows[0], step.query_rows[1])
    assert int(step.n_q[0]) == int(step.n_q[1]) > 0
    want = step_oracle.region_step(wl, lat, qkv, t, np.float32(scale), np.float32(dt), np.float32(dt_u))
    for b in range(2):
        nq = int(want["n_q"][b])
        rows = step.query_rows[b, :nq].long()
        assert_close(host_f64(step.o_full[b][rows]), want["o_e"][b, :nq], f"guidance branch {b}")
    assert not torch.equal(step.o_full[0], step.o_full[1])
    assert_close(host_f64(step.x_out), want["x_out"], "merged latents")
