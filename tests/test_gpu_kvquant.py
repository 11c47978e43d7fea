"""GPU parity of the 8-bit (E4M3) cache variant: codes and scales bit-exact against the oracle, the
widened cache bit-exact against the oracle's decode, and the region attention over the widened cache
within tolerance of the oracle's attention over the same quantised values."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, dev_i32, errors, host_f64
from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _rand_bf16(rng, shape, std=1.0):
    return synth.bf16_round((rng.standard_normal(shape, dtype=np.float32) * np.float32(std)))


def _store_load(k, v, keep, n_keep):
    import torch
    B, N, H, D = k.shape
    cap = keep.shape[1]
    kq = torch.full((B, cap, H, D), 0x55, dtype=torch.uint8, device="cuda")
    vq = torch.full((B, cap, H, D), 0x55, dtype=torch.uint8, device="cuda")
    ks = torch.full((B, cap, H), -7.0, dtype=torch.float32, device="cuda")
    vs = torch.full((B, cap, H), -7.0, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.rikv_store_e4m3(dev_bf16(k), dev_bf16(v), dev_i32(keep), dev_i32(n_keep), kq, vq, ks, vs, dev_status=st)
    kc = torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    vc = torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    binding.rikv_load_e4m3(kq, vq, ks, vs, dev_i32(n_keep), kc, vc, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    return kq.cpu().numpy(), vq.cpu().numpy(), ks.cpu().numpy(), vs.cpu().numpy(), kc, vc


@pytest.mark.parametrize("D,H", [(128, 5), (64, 3), (128, 24)])
def test_codes_scales_and_widened_cache_are_bit_exact(D, H):
    rng = np.random.default_rng(D + H)
    B, N = 2, 300
    k = _rand_bf16(rng, (B, N, H, D), 0.09)
    v = _rand_bf16(rng, (B, N, H, D), 1.0)
    k[0, 7, 0] = 0.0                                     # an all-zero row and head: scale 1, codes 0
    k[1, 9, 1, 3] = 448.0 * 4.0                          # an element exactly at the top of the scaled format
    v[0, 5, 1] = synth.bf16_round(v[0, 5, 1] * np.float32(1e-27))    # a tiny row: the scale follows it down
    v[0, 11, 2] = synth.bf16_round(v[0, 11, 2] * np.float32(1e-30))  # tinier still: the exponent floor holds
    # 200 distinct rows per request, the special rows 5, 7, 9, 11 among the first few
    keep = np.stack([np.unique(np.concatenate([[5, 7, 9, 11], rng.permutation(N)[:200]]))[:200]
                     for _ in range(B)]).astype(np.int32)
    n_keep = np.array([200, 57], np.int32)
    assert np.all(keep[:, :57].min(axis=1) <= 5) and all(11 in keep[b, :57] for b in range(B))
    kq, vq, ks, vs, kc, vc = _store_load(k, v, keep, n_keep)
    wkq, wvq, wks, wvs = orc.rikv_store_e4m3(k, v, keep, n_keep)
    wk, wv = orc.rikv_load_e4m3(wkq, wvq, wks, wvs, n_keep)
    for b in range(B):
        n = n_keep[b]
        # (+0 and -0 are the same value; compare codes up to the sign of zero)
        for got, want in ((kq, wkq), (vq, wvq)):
            zero = (want[b, :n] & 0x7f) == 0
            assert np.array_equal(got[b, :n][~zero], want[b, :n][~zero])
            assert np.all((got[b, :n][zero] & 0x7f) == 0)
            assert np.all(got[b, n:] == 0x55)                                   # tail untouched
        assert np.array_equal(ks[b, :n].astype(np.float64), wks[b, :n]) and np.all(ks[b, n:] == -7.0)
        assert np.array_equal(vs[b, :n].astype(np.float64), wvs[b, :n])
        assert np.array_equal(host_f64(kc)[b, :n], wk[b, :n]) and np.array_equal(host_f64(vc)[b, :n], wv[b, :n])
        assert np.all(host_f64(kc)[b, n:] == -3.0)


def test_region_attention_over_the_8_bit_cache():
    """Config 2's shape at a reduced token count: the attention over the widened 8-bit cache matches the
    oracle's attention over the same quantised values within the stated tolerance; the distance to the
    attention over the unquantised cache is reported, not asserted."""
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[2], grid=(24, 24), n_text=70)
    mask = synth.make_latents(wl)["mask"][0]
    qkv = synth.make_qkv_full(wl)
    rows = orc.region_rows(mask, wl.n_text, wl.n_ref, "edited_queries")
    nq, nc = len(rows["query"]), len(rows["cache"])
    keep = np.zeros((1, nc), np.int32); keep[0] = rows["cache"]
    kq, vq, ks, vs, kc, vc = _store_load(qkv["k"], qkv["v"], keep, np.array([nc], np.int32))
    q = qkv["q"][:, rows["query"]]; kf = qkv["k"][:, rows["fresh"]]; vf = qkv["v"][:, rows["fresh"]]
    out = torch.full(q.shape, -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(binding.region_attention_workspace(1, nq, nq, nc, wl.heads, wl.head_dim), 256),
                     dtype=torch.uint8, device="cuda")
    binding.region_attention(dev_bf16(q), dev_bf16(kf), dev_bf16(vf), kc, vc, dev_i32([nq]), dev_i32([nq]),
                             dev_i32([nc]), out, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    wkq, wvq, wks, wvs = orc.rikv_store_e4m3(qkv["k"], qkv["v"], keep, [nc])
    wk, wv = orc.rikv_load_e4m3(wkq, wvq, wks, wvs, [nc])
    want_q = orc.region_attention(q, kf, vf, wk, wv, [nq], [nq], [nc])
    assert_close(host_f64(out), want_q, "attention over the quantised cache")
    want_full = orc.region_attention(q, kf, vf, qkv["k"][:, rows["cache"]], qkv["v"][:, rows["cache"]], [nq], [nq], [nc])
    ma, rr = errors(host_f64(out), want_full)
    print(f"8-bit cache vs unquantised cache: max-abs {ma:.3e}, rel-RMS {rr:.3e}")
    assert rr < 0.1                                        # (a sanity bound only: E4M3 carries 3 mantissa bits)


def test_bad_row_index_is_reported():
    import torch
    rng = np.random.default_rng(1)
    k = _rand_bf16(rng, (1, 50, 2, 64)); v = _rand_bf16(rng, (1, 50, 2, 64))
    keep = np.array([[3, 70, 5]], np.int32)
    kq = torch.zeros((1, 3, 2, 64), dtype=torch.uint8, device="cuda"); vq = torch.zeros_like(kq)
    ks = torch.zeros((1, 3, 2), dtype=torch.float32, device="cuda"); vs = torch.zeros_like(ks)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.rikv_store_e4m3(dev_bf16(k), dev_bf16(v), dev_i32(keep), dev_i32([3]), kq, vq, ks, vs, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == binding.DEV_BOUNDS and float(ks[0, 1, 0]) == 0.0 and float(ks[0, 2, 0]) > 0.0
