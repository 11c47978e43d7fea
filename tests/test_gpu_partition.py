"""GPU parity: Adaptive Region Partition, morphology and row lists against the fp64 oracle."""
import numpy as np
import pytest

from gpu_util import dev_bf16, dev_i32, host_f64
from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding, synth

pytestmark = pytest.mark.gpu


def run_partition(x_t, v, ref, t, metric, thr):
    import torch
    B, N, _ = x_t.shape
    dx, dv, dr = dev_bf16(x_t), dev_bf16(v), dev_bf16(ref)
    mask = torch.full((B, N), 77, dtype=torch.uint8, device="cuda")
    e = torch.full((B, N), -7, dtype=torch.int32, device="cuda")
    k = torch.full((B, N), -7, dtype=torch.int32, device="cuda")
    s = torch.full((B, N), -7, dtype=torch.int32, device="cuda")
    ne = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    score = torch.full((B, N), float("nan"), dtype=torch.float32, device="cuda")
    binding.partition(dx, dv, dr, t, metric, thr, mask, e, k, s, ne, score=score)
    torch.cuda.synchronize()
    return dict(mask=mask.cpu().numpy(), edit_idx=e.cpu().numpy(), keep_idx=k.cpu().numpy(),
                slot=s.cpu().numpy(), n_edit=ne.cpu().numpy(), score=score.cpu().numpy())


def check_against_oracle(got, want, N, decided=None):
    """Bit-exact masks and indices.  `decided` restricts the mask comparison to tokens whose
    oracle score is at least 1e-3 (relative) away from the threshold."""
    B = want["mask"].shape[0]
    if decided is None:
        assert np.array_equal(got["mask"], want["mask"])
        assert np.array_equal(got["n_edit"], want["n_edit"])
        assert np.array_equal(got["slot"], want["slot"])
        for b in range(B):
            ne = int(want["n_edit"][b])
            assert np.array_equal(got["edit_idx"][b, :ne], want["edit_idx"][b, :ne])
            assert np.array_equal(got["keep_idx"][b, :N - ne], want["keep_idx"][b, :N - ne])
            assert np.all(got["edit_idx"][b, ne:] == -7)            # tail untouched
            assert np.all(got["keep_idx"][b, N - ne:] == -7)
    else:
        assert np.array_equal(got["mask"][decided], want["mask"][decided])
        for b in range(B):      # the lists must be the exact compaction of the GPU's own mask
            e, k, s, ne = orc.compact_indices(got["mask"][b])
            assert ne == got["n_edit"][b] and np.array_equal(got["slot"][b], s)
            assert np.array_equal(got["edit_idx"][b, :ne], e[:ne])
            assert np.array_equal(got["keep_idx"][b, :N - ne], k[:N - ne])
    assert np.max(np.abs(got["score"] - want["score"])) < 2e-5 * max(1.0, np.max(np.abs(want["score"])))


CASES = [(1, None), (2, None), (3, 0.05), (3, 0.10), (3, 0.25), (3, 0.50), (3, 1.00), (4, None),
         (5, None)]


@pytest.mark.parametrize("cfg,ratio", CASES)
def test_configs_full_size(cfg, ratio):
    wl = synth.WORKLOADS[cfg]
    lat = synth.make_latents(wl, ratio)
    metric = orc.COSINE if wl.metric == "cosine" else orc.L2
    want = orc.partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], metric, wl.threshold)
    got = run_partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], metric, wl.threshold)
    check_against_oracle(got, want, wl.n_img)
    assert np.array_equal(got["mask"], lat["mask"])              # the planted mask


@pytest.mark.parametrize("metric", [orc.COSINE, orc.L2])
def test_threshold_sweep_through_the_score_distribution(metric):
    # thresholds inside the bulk of the scores: every token that is not within 1e-3 (relative) of
    # the threshold must be decided exactly as the oracle decides it
    rng = np.random.default_rng(11)
    B, N, C = 2, 3000, 16
    x, v, r = (synth.bf16_round(rng.standard_normal((B, N, C)).astype(np.float32)) for _ in range(3))
    r = synth.bf16_round((0.7 * x + 0.7 * r).astype(np.float32))
    t = 0.25
    sc = orc.token_score(orc.one_step_estimate(x, t, v), r, metric)
    for thr in np.quantile(sc, [0.02, 0.3, 0.5, 0.9]):
        want = orc.partition(x, v, r, t, metric, float(np.float32(thr)))
        got = run_partition(x, v, r, t, metric, float(np.float32(thr)))
        decided = np.abs(want["score"] - np.float32(thr)) >= 1e-3 * abs(thr)
        assert decided.mean() > 0.98
        check_against_oracle(got, want, N, decided)


@pytest.mark.parametrize("N,C,B", [(1, 16, 1), (31, 16, 2), (127, 8, 1), (129, 16, 3), (513, 32, 2),
                                   (4097, 16, 1), (1000, 64, 2), (777, 256, 1), (300, 512, 2),
                                   (150, 1024, 1), (140001, 16, 1), (9216, 16, 4),
                                   # requests long enough for the two-launch form (decisions, then compaction)
                                   (32768, 16, 2), (40000, 32, 3), (65539, 24, 2), (33000, 256, 1)])
def test_ragged_sizes_and_channel_counts(N, C, B):
    rng = np.random.default_rng(N * 7 + C)
    r = rng.standard_normal((B, N, C))
    planted = rng.random((B, N, 1)) < 0.37
    x0 = np.where(planted, -r + 0.1 * rng.standard_normal((B, N, C)), r)
    noise = rng.standard_normal((B, N, C))
    t = 0.6
    x_t = synth.bf16_round(((1 - t) * x0 + t * noise).astype(np.float32))
    v = synth.bf16_round((noise - x0).astype(np.float32))
    ref = synth.bf16_round(r.astype(np.float32))
    for metric, thr in ((orc.COSINE, 0.5), (orc.L2, 0.5 * np.sqrt(C))):
        want = orc.partition(x_t, v, ref, t, metric, thr)
        got = run_partition(x_t, v, ref, t, metric, thr)
        check_against_oracle(got, want, N)
        assert np.array_equal(got["mask"], planted[..., 0].astype(np.uint8))


def test_all_edited_and_none_edited():
    wl = synth.scaled_workload(synth.WORKLOADS[2], grid=(40, 40))
    for ratio in (0.0, 1.0):
        lat = synth.make_latents(wl, ratio)
        want = orc.partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], orc.COSINE, wl.threshold)
        got = run_partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], orc.COSINE, wl.threshold)
        check_against_oracle(got, want, wl.n_img)
        assert got["n_edit"][0] == (0 if ratio == 0.0 else wl.n_img)


def test_straight_line_velocity_gives_empty_edit_set():
    rng = np.random.default_rng(3)
    X0 = synth.bf16_round(rng.standard_normal((1, 2048, 16)).astype(np.float32))
    X1 = synth.bf16_round(rng.standard_normal((1, 2048, 16)).astype(np.float32))
    t = 0.5                                   # exactly representable mixing keeps x_t in bf16 range
    x_t = synth.bf16_round(((1 - t) * X0 + t * X1).astype(np.float32))
    v = synth.bf16_round((X1 - X0).astype(np.float32))
    got = run_partition(x_t, v, X0, t, orc.COSINE, 0.93)
    assert got["n_edit"][0] == 0 and not got["mask"].any()


def test_morphological_open_close_matches_oracle():
    import torch
    rng = np.random.default_rng(4)
    for (rows, cols, B) in ((64, 64, 2), (96, 96, 1), (17, 33, 3), (1, 9, 1), (128, 128, 1)):
        N = rows * cols
        noisy = np.stack([np.where(rng.random(N) < 0.04, 1 - m, m) for m in
                          (synth.mask_blobs(rng, (rows, cols), 0.3) for _ in range(B))]).astype(np.uint8)
        d_in = torch.from_numpy(noisy).cuda()
        d_out = torch.full((B, N), 9, dtype=torch.uint8, device="cuda")
        e, k, s = (torch.full((B, N), -7, dtype=torch.int32, device="cuda") for _ in range(3))
        ne = torch.zeros(B, dtype=torch.int32, device="cuda")
        binding.mask_open_close(d_in, rows, cols, d_out, e, k, s, ne)
        torch.cuda.synchronize()
        for b in range(B):
            want = orc.open_close(noisy[b], (rows, cols))
            assert np.array_equal(d_out[b].cpu().numpy(), want)
            we, wk, ws, wn = orc.compact_indices(want)
            assert int(ne[b]) == wn and np.array_equal(s[b].cpu().numpy(), ws)
            assert np.array_equal(e[b, :wn].cpu().numpy(), we[:wn])
            assert np.array_equal(k[b, :N - wn].cpu().numpy(), wk[:N - wn])


@pytest.mark.parametrize("membership", ["edited_queries", "paper"])
def test_region_rows_match_the_oracle_membership_rule(membership):
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[5], grid=(48, 48), n_text=77, batch=3)
    lat = synth.make_latents(wl)
    p = orc.partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], orc.COSINE, wl.threshold)
    B, N = wl.batch, wl.n_img
    q_cap, c_cap = N + wl.n_text, wl.n_full
    qr = torch.full((B, q_cap), -7, dtype=torch.int32, device="cuda")
    cr = torch.full((B, c_cap), -7, dtype=torch.int32, device="cuda")
    nq, nc = (torch.zeros(B, dtype=torch.int32, device="cuda") for _ in range(2))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.region_rows(dev_i32(p["edit_idx"]), dev_i32(p["keep_idx"]), dev_i32(p["n_edit"]), wl.n_text,
                        wl.n_ref, binding.ROWS_PAPER if membership == "paper" else binding.ROWS_EDITED_QUERIES,
                        qr, nq, cr, nc, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    for b in range(B):
        want = orc.region_rows(p["mask"][b], wl.n_text, wl.n_ref, membership)
        assert int(nq[b]) == len(want["query"]) and int(nc[b]) == len(want["cache"])
        assert np.array_equal(qr[b, :int(nq[b])].cpu().numpy(), want["query"])
        assert np.array_equal(cr[b, :int(nc[b])].cpu().numpy(), want["cache"])
        assert np.all(qr[b, int(nq[b]):].cpu().numpy() == -7)


@pytest.mark.parametrize("membership", ["edited_queries", "paper"])
@pytest.mark.parametrize("grid,n_text,batch", [((48, 48), 77, 3), ((64, 64), 512, 1), ((9, 7), 0, 2), ((96, 96), 33, 2),
                                               ((200, 190), 40, 2)])          # 38000 tokens: the two-launch form
def test_partition_with_row_lists_in_one_launch(membership, grid, n_text, batch):
    """regione_partition_rows = regione_partition + regione_region_rows: every output bit-exact
    against the oracle partition and the oracle row lists, tails untouched."""
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[5], grid=grid, n_text=n_text, batch=batch)
    lat = synth.make_latents(wl)
    p = orc.partition(lat["x_t"], lat["v"], lat["ref"], lat["t"], orc.COSINE, wl.threshold)
    B, N = wl.batch, wl.n_img
    q_cap, c_cap = N + wl.n_text + 3, wl.n_full + 5
    i32 = torch.int32
    mask = torch.full((B, N), 77, dtype=torch.uint8, device="cuda")
    e, k, s = (torch.full((B, N), -7, dtype=i32, device="cuda") for _ in range(3))
    ne = torch.full((B,), -7, dtype=i32, device="cuda")
    qr = torch.full((B, q_cap), -7, dtype=i32, device="cuda")
    cr = torch.full((B, c_cap), -7, dtype=i32, device="cuda")
    nq, nc = (torch.full((B,), -7, dtype=i32, device="cuda") for _ in range(2))
    st = torch.zeros(1, dtype=i32, device="cuda")
    score = torch.full((B, N), float("nan"), dtype=torch.float32, device="cuda")
    binding.partition_rows(dev_bf16(lat["x_t"]), dev_bf16(lat["v"]), dev_bf16(lat["ref"]), lat["t"],
                           binding.METRIC_COSINE, wl.threshold, mask, e, k, s, ne, wl.n_text, wl.n_ref,
                           binding.ROWS_PAPER if membership == "paper" else binding.ROWS_EDITED_QUERIES,
                           qr, nq, cr, nc, score=score, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    got = dict(mask=mask.cpu().numpy(), edit_idx=e.cpu().numpy(), keep_idx=k.cpu().numpy(),
               slot=s.cpu().numpy(), n_edit=ne.cpu().numpy(), score=score.cpu().numpy())
    check_against_oracle(got, p, N)
    for b in range(B):
        want = orc.region_rows(p["mask"][b], wl.n_text, wl.n_ref, membership)
        assert int(nq[b]) == len(want["query"]) and int(nc[b]) == len(want["cache"])
        assert np.array_equal(qr[b, :int(nq[b])].cpu().numpy(), want["query"])
        assert np.array_equal(cr[b, :int(nc[b])].cpu().numpy(), want["cache"])
        assert np.all(qr[b, int(nq[b]):].cpu().numpy() == -7)
        assert np.all(cr[b, int(nc[b]):].cpu().numpy() == -7)


def test_partition_with_row_lists_reports_lists_that_do_not_fit():
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[5], grid=(32, 32), n_text=16, batch=1)
    lat = synth.make_latents(wl)
    B, N = wl.batch, wl.n_img
    i32 = torch.int32
    mask = torch.zeros((B, N), dtype=torch.uint8, device="cuda")
    e, k, s = (torch.zeros((B, N), dtype=i32, device="cuda") for _ in range(3))
    ne, nq, nc = (torch.zeros(B, dtype=i32, device="cuda") for _ in range(3))
    qr = torch.full((B, 8), -7, dtype=i32, device="cuda")            # far too small
    cr = torch.full((B, 8), -7, dtype=i32, device="cuda")
    st = torch.zeros(1, dtype=i32, device="cuda")
    binding.partition_rows(dev_bf16(lat["x_t"]), dev_bf16(lat["v"]), dev_bf16(lat["ref"]), lat["t"],
                           binding.METRIC_COSINE, wl.threshold, mask, e, k, s, ne, wl.n_text, wl.n_ref,
                           binding.ROWS_EDITED_QUERIES, qr, nq, cr, nc, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == binding.DEV_BOUNDS
    assert int(nq[0]) == 8 and int(nc[0]) == 8                       # clamped, nothing written past the end


@pytest.mark.parametrize("B", [3, 130])
def test_requests_at_their_own_sampler_times(B):
    """Each request of a batch carries its own t (requests sitting at different sampler steps, or the
    two guidance branches of one request sharing a mask): request b must equal the oracle run on that
    request alone with t[b].  B = 130 crosses the 128-requests-per-launch chunk of the time array."""
    wl = synth.scaled_workload(synth.WORKLOADS[5], grid=(20, 20), batch=B)
    ts = [(22.0 - (b % 5)) / 28.0 for b in range(B)]
    lats = [synth.make_latents(synth.scaled_workload(wl, batch=1), stream=b, t=ts[b]) for b in range(B)]
    x_t, v, ref = (np.concatenate([l[k] for l in lats]) for k in ("x_t", "v", "ref"))
    got = run_partition(x_t, v, ref, ts, orc.COSINE, wl.threshold)
    for b in range(B):
        want = orc.partition(x_t[b:b + 1], v[b:b + 1], ref[b:b + 1], np.float32(ts[b]), orc.COSINE, wl.threshold)
        one = {k: a[b:b + 1] for k, a in got.items()}
        check_against_oracle(one, want, wl.n_img)
        assert np.array_equal(one["mask"][0], lats[b]["mask"][0])
    # the same batch with every request at the first request's time decides some tokens differently
    # (otherwise this test would not notice a kernel that ignores the per-request values)
    same = run_partition(x_t, v, ref, ts[0], orc.COSINE, wl.threshold)
    assert not np.array_equal(same["score"], got["score"])


def test_long_requests_sit_a_call_out_too():
    """The two-launch form of long requests honours the NaN convention in both of its launches."""
    import torch
    rng = np.random.default_rng(12)
    B, N, C = 3, 33000, 16
    x_t, v, ref = (synth.bf16_round(rng.standard_normal((B, N, C)).astype(np.float32)) for _ in range(3))
    ts = [0.6, float("nan"), 0.7]
    got = run_partition(x_t, v, ref, ts, orc.COSINE, 0.1)
    for b in (0, 2):
        want = orc.partition(x_t[b:b + 1], v[b:b + 1], ref[b:b + 1], np.float32(ts[b]), orc.COSINE, 0.1)
        decided = np.abs(want["score"] - np.float32(0.1)) >= 1e-4
        check_against_oracle({k: a[b:b + 1] for k, a in got.items()}, want, N, decided)
    assert np.all(got["mask"][1] == 77) and np.all(got["slot"][1] == -7) and got["n_edit"][1] == -7
    assert np.all(np.isnan(got["score"][1]))
