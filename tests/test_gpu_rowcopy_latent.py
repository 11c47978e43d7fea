"""GPU parity: gather / scatter / RIKV store (bit-exact) and the latent updates (fp tolerance)."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, dev_i32, host_f64
from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _rand_bf16(rng, shape):
    return synth.bf16_round(rng.standard_normal(shape).astype(np.float32))


@pytest.mark.parametrize("rows,cap,inner,B", [(50, 20, (8,), 1), (4096, 819, (16,), 1), (333, 333, (24,), 2),
                                             (9216, 1400, (16,), 4), (600, 257, (24, 128), 2),
                                             (130, 64, (520,), 1)])
def test_gather_then_scatter(rows, cap, inner, B):
    import torch
    rng = np.random.default_rng(rows + cap)
    src = _rand_bf16(rng, (B, rows) + inner)
    n = np.array([cap if b == 0 else rng.integers(0, cap + 1) for b in range(B)], np.int32)
    idx = np.stack([np.sort(rng.permutation(rows)[:cap]) for _ in range(B)]).astype(np.int32)
    d_src = dev_bf16(src)
    d_dst = torch.full((B, cap) + inner, -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.gather(d_src, dev_i32(idx), dev_i32(n), d_dst, dev_status=st)
    got = host_f64(d_dst)
    want = orc.gather(src, idx, n)
    live = ~np.isnan(want)
    assert np.array_equal(got[live], want[live])                 # bit-exact copy
    assert np.all(got[~live] == -3.0)                            # rows past n[b] untouched
    # scatter back into a poisoned image: edited rows restored, nothing else touched
    d_back = torch.full((B, rows) + inner, 5.0, dtype=torch.bfloat16, device="cuda")
    binding.scatter(d_dst, dev_i32(idx), dev_i32(n), d_back, dev_status=st)
    want_back = orc.scatter(np.full(src.shape, 5.0), want, idx, n)
    assert np.array_equal(host_f64(d_back), want_back)
    assert int(st[0]) == 0


def test_gather_reports_out_of_range_rows_without_touching_memory():
    import torch
    rng = np.random.default_rng(1)
    src = _rand_bf16(rng, (1, 10, 8))
    idx = np.array([[0, 3, 10, -1, 9]], np.int32)
    d_dst = torch.full((1, 5, 8), -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.gather(dev_bf16(src), dev_i32(idx), dev_i32([5]), d_dst, dev_status=st)
    got = host_f64(d_dst)
    assert int(st[0]) == binding.DEV_BOUNDS
    assert np.array_equal(got[0, [0, 1, 4]], src[0, [0, 3, 9]]) and np.all(got[0, [2, 3]] == -3.0)
    st.zero_()
    binding.gather(dev_bf16(src), dev_i32(idx[:, :2]), dev_i32([7]), d_dst[:, :2].contiguous(), dev_status=st)
    assert int(st[0]) == binding.DEV_BOUNDS                       # count above capacity is clamped


@pytest.mark.parametrize("n_full,H,D,B", [(300, 4, 64, 2), (2112, 4, 64, 1), (1000, 24, 128, 2)])
def test_rikv_store(n_full, H, D, B):
    import torch
    rng = np.random.default_rng(n_full)
    k, v = _rand_bf16(rng, (B, n_full, H, D)), _rand_bf16(rng, (B, n_full, H, D))
    cap = n_full
    n = np.array([n_full if b == 0 else n_full // 3 + 7 for b in range(B)], np.int32)
    keep = np.stack([np.arange(n_full) if b == 0 else np.sort(rng.permutation(n_full)) for b in range(B)]).astype(np.int32)
    kc = torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    vc = torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.rikv_store(dev_bf16(k), dev_bf16(v), dev_i32(keep), dev_i32(n), kc, vc, dev_status=st)
    wk, wv = orc.rikv_store(k, v, keep, n)
    for got, want in ((host_f64(kc), wk), (host_f64(vc), wv)):
        live = ~np.isnan(want)
        assert np.array_equal(got[live], want[live]) and np.all(got[~live] == -3.0)
    assert np.array_equal(host_f64(kc)[0], k[0])                  # identity keep list = plain copy
    assert int(st[0]) == 0


@pytest.mark.parametrize("B,cap,C", [(1, 819, 16), (4, 1400, 16), (2, 77, 64), (1, 1, 8)])
def test_velocity_decay(B, cap, C):
    import torch
    rng = np.random.default_rng(cap)
    v, x = _rand_bf16(rng, (B, cap, C)), _rand_bf16(rng, (B, cap, C))
    n = np.array([cap if b == 0 else rng.integers(0, cap + 1) for b in range(B)], np.int32)
    for scale, dt, store in ((1.0, 1 / 28, True), (0.9298, 1 / 28, False), (0.5, 0.25, True)):
        dx = dev_bf16(x)
        vc = torch.full((B, cap, C), -3.0, dtype=torch.bfloat16, device="cuda")
        binding.velocity_decay(dev_bf16(v), scale, dt, dx, dev_i32(n), v_cache_out=vc if store else None)
        want, _ = orc.velocity_decay(v, np.float32(scale), np.float32(dt), x, n)
        assert_close(host_f64(dx), want, "velocity_decay")
        # one bf16 rounding of an fp32 result: at most half an ulp (2^-8 relative) plus fp32 noise
        assert np.all(np.abs(host_f64(dx) - want) <= 2.0 ** -8 * np.abs(want) + 1e-6)
        for b in range(B):
            assert np.array_equal(host_f64(dx)[b, n[b]:], x[b, n[b]:])          # dead rows untouched
            if store:
                assert np.array_equal(host_f64(vc)[b, :n[b]], v[b, :n[b]])
                assert np.all(host_f64(vc)[b, n[b]:] == -3.0)


@pytest.mark.parametrize("cfg,grid", [(1, None), (2, None), (5, (48, 48))])
def test_merge(cfg, grid):
    import torch
    wl = synth.WORKLOADS[cfg] if grid is None else synth.scaled_workload(synth.WORKLOADS[cfg], grid=grid)
    lat = synth.make_latents(wl)
    rng = np.random.default_rng(cfg)
    B, N, C = wl.batch, wl.n_img, wl.channels
    slot = np.stack([orc.compact_indices(lat["mask"][b])[2] for b in range(B)])
    cap = int(lat["mask"].sum(axis=1).max())
    x_e = _rand_bf16(rng, (B, cap, C))
    dt = 5.0 / 28.0
    for sl in (slot, np.full_like(slot, -1)):                      # planted mask, then zero-edit mask
        out = torch.full((B, N, C), -3.0, dtype=torch.bfloat16, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.merge(dev_bf16(lat["x_t"]), dev_bf16(lat["v"]), dev_bf16(x_e), dev_i32(sl), dt, out, dev_status=st)
        want = orc.merge(lat["x_t"], lat["v"], x_e, sl, np.float32(dt))
        got = host_f64(out)
        assert_close(got, want, "merge")
        assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-6)
        edited = sl >= 0
        assert np.array_equal(got[edited], want[edited])            # copied rows are bit-exact
        assert int(st[0]) == 0
    # full mask: output is x_e in token order; in-place on x_full is allowed
    full = np.broadcast_to(np.arange(N, dtype=np.int32), (B, N)).copy()
    x_e_full = _rand_bf16(rng, (B, N, C))
    buf = dev_bf16(lat["x_t"])
    binding.merge(buf, dev_bf16(lat["v"]), dev_bf16(x_e_full), dev_i32(full), dt, buf)
    assert np.array_equal(host_f64(buf), x_e_full)


@pytest.mark.parametrize("S,T1,n", [(3, 5, 8), (4, 29, 4096 * 16), (2, 2, 1000 * 8)])
def test_gamma_fit(S, T1, n):
    import torch
    rng = np.random.default_rng(S * 100 + T1)
    v = synth.bf16_round(rng.standard_normal((S, T1, n)).astype(np.float32) *
                         np.linspace(1.0, 2.0, T1, dtype=np.float32)[None, :, None])
    dt = np.full(T1 - 1, 1.0 / 28.0, np.float32)
    norms = torch.full((S, T1), -1.0, dtype=torch.float32, device="cuda")
    gamma = torch.full((T1 - 1,), -1.0, dtype=torch.float32, device="cuda")
    binding.gamma_fit(dev_bf16(v), torch.from_numpy(dt).cuda(), norms, gamma)
    torch.cuda.synchronize()
    want_n, want_g = orc.gamma_fit(v, dt)
    assert np.allclose(norms.cpu().numpy(), want_n, rtol=2e-6)
    assert np.allclose(gamma.cpu().numpy(), want_g, rtol=1e-5)


def test_gather_multi_matches_single_gathers():
    import torch
    rng = np.random.default_rng(9)
    B, rows, cap, inner = 2, 300, 120, (3, 64)
    srcs = [dev_bf16(synth.bf16_round(rng.standard_normal((B, rows) + inner).astype(np.float32))) for _ in range(3)]
    idx = torch.stack([torch.randperm(rows, device="cuda")[:cap].sort()[0] for _ in range(B)]).to(torch.int32).contiguous()
    n = torch.tensor([cap, 77], dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    one = [torch.full((B, cap) + inner, -3.0, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    many = [t.clone() for t in one]
    for s_, d_ in zip(srcs, one):
        binding.gather(s_, idx, n, d_, dev_status=st)
    binding.gather_multi(srcs, idx, n, many, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    for a, b_ in zip(one, many):
        assert torch.equal(a, b_)
    with pytest.raises(binding.RegionEError):
        binding.gather_multi(srcs * 2, idx, n, many * 2)


@pytest.mark.parametrize("B", [4, 131])
def test_velocity_decay_and_merge_with_per_request_steps(B):
    """Requests of one batch at different sampler steps: scale, dt and dt_unedited are arrays of B
    values; request b must match the oracle called on that request alone with its own values."""
    import torch
    rng = np.random.default_rng(B)
    cap, C, N = 90, 16, 160
    v, x = _rand_bf16(rng, (B, cap, C)), _rand_bf16(rng, (B, cap, C))
    n = rng.integers(1, cap + 1, B).astype(np.int32)
    scale = (0.8 + 0.2 * rng.random(B)).astype(np.float32)
    dt = ((1 + rng.integers(0, 4, B)) / 28.0).astype(np.float32)
    dx = dev_bf16(x)
    binding.velocity_decay(dev_bf16(v), scale, dt, dx, dev_i32(n))
    got = host_f64(dx)
    for b in range(B):
        want, _ = orc.velocity_decay(v[b:b + 1], scale[b], dt[b], x[b:b + 1], n[b:b + 1])
        assert np.all(np.abs(got[b] - want[0]) <= 2.0 ** -8 * np.abs(want[0]) + 1e-6), b
    assert len(set(np.round(dt * scale, 6).tolist())) > 2          # the values really differ
    # merge
    xf, vf = _rand_bf16(rng, (B, N, C)), _rand_bf16(rng, (B, N, C))
    slot = np.full((B, N), -1, np.int32)
    for b in range(B):
        ids = np.sort(rng.permutation(N)[:n[b]])
        slot[b, ids] = np.arange(n[b])
    dtu = ((2 + rng.integers(0, 6, B)) / 28.0).astype(np.float32)
    out = torch.full((B, N, C), -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.merge(dev_bf16(xf), dev_bf16(vf), dev_bf16(x), dev_i32(slot), dtu, out, dev_status=st)
    got = host_f64(out)
    assert int(st[0]) == 0
    for b in range(B):
        want = orc.merge(xf[b:b + 1], vf[b:b + 1], x[b:b + 1], slot[b:b + 1], dtu[b])
        assert np.all(np.abs(got[b] - want[0]) <= 2.0 ** -8 * np.abs(want[0]) + 1e-6), b
    with pytest.raises(binding.RegionEError):
        binding.merge(dev_bf16(xf), dev_bf16(vf), dev_bf16(x), dev_i32(slot), dtu[:2], out)
