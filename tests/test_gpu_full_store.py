"""GPU parity of the full attention step that refreshes the Region-Instruction KV cache in the same
launch: output against the fp64 oracle's attention, cache against the oracle's row copy (bit-exact),
and both against the two separate library calls."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, dev_i32, host_f64
from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _rand_bf16(rng, shape, std=1.0):
    return synth.bf16_round((rng.standard_normal(shape, dtype=np.float32) * np.float32(std)))


def _run(q, k, v, n_rows, keep, n_keep):
    import torch
    B, N, H, D = q.shape
    cap = keep.shape[1]
    dq, dk, dv = dev_bf16(q), dev_bf16(k), dev_bf16(v)
    kc = torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    vc = torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    out = torch.full((B, N, H, D), -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(binding.full_attention_store_workspace(B, N, H, D), 256), dtype=torch.uint8, device="cuda")
    binding.full_attention_store(dq, dk, dv, dev_i32(n_rows), dev_i32(keep), dev_i32(n_keep), kc, vc, out,
                                 workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    return out, kc, vc, int(st[0]), (dq, dk, dv, ws)


def _keep_lists(rng, n_rows, fractions, cap):
    B = len(n_rows)
    keep = np.zeros((B, cap), np.int32)
    n_keep = np.zeros(B, np.int32)
    for b in range(B):
        m = int(round(fractions[b] * n_rows[b]))
        keep[b, :m] = np.sort(rng.permutation(n_rows[b])[:m])
        n_keep[b] = m
    return keep, n_keep


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("n_rows,fractions", [
    ([700, 513], [0.8, 0.33]),          # several key tiles, ragged tails, shares cutting items
    ([128, 1], [1.0, 1.0]),             # identity keep list; a one-row request
    ([300, 0, 257], [0.5, 0.0, 0.0]),   # an empty request and a request that keeps nothing
    ([100], [0.07]),                    # a lone query tile, single key tile
])
def test_output_and_cache_match_oracle(D, n_rows, fractions):
    import torch
    rng = np.random.default_rng(sum(n_rows) + D)
    B, H = len(n_rows), 3
    N = max(n_rows) + 5
    q, k, v = (_rand_bf16(rng, (B, N, H, D), s_) for s_ in (0.5, 0.5, 1.0))
    cap = N + 2
    keep, n_keep = _keep_lists(rng, n_rows, fractions, cap)
    out, kc, vc, status, dev = _run(q, k, v, n_rows, keep, n_keep)
    assert status == 0, binding.status_string(status)
    empty = np.zeros((B, 0, H, D))
    want = orc.region_attention(q, k, v, empty, empty, n_rows, n_rows, [0] * B)
    wk, wv = orc.rikv_store(k, v, keep, n_keep)
    got = host_f64(out)
    for b in range(B):
        n = n_rows[b]
        assert np.all(got[b, n:] == -3.0)
        if n:
            assert_close(got[b, :n], want[b, :n], f"attention, request {b}")
        for g, w in ((host_f64(kc), wk), (host_f64(vc), wv)):
            assert np.array_equal(g[b, :n_keep[b]], w[b, :n_keep[b]])           # copies: bit-exact
            assert np.all(g[b, n_keep[b]:] == -3.0)                             # tail untouched
    # the same bits as the two separate calls
    dq, dk, dv, ws = dev
    out2 = torch.full_like(out, -3.0)
    kc2, vc2 = torch.full_like(kc, -3.0), torch.full_like(vc, -3.0)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    zeros = dev_i32([0] * B)
    binding.region_attention(dq, dk, dv, None, None, dev_i32(n_rows), dev_i32(n_rows), zeros, out2,
                             workspace=ws, dev_status=st)
    binding.rikv_store(dk, dv, dev_i32(keep), dev_i32(n_keep), kc2, vc2, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    for a, b_ in ((out, out2), (kc, kc2), (vc, vc2)):
        assert torch.equal(a.view(torch.int16), b_.view(torch.int16))


def test_config3_size_cache_of_the_quarter_mask():
    """Qwen-Image-Edit-shaped full step (8448 rows, 24 heads x 128) that keeps text, unedited and
    reference rows of a 25 % mask: every cache row bit-exact, output identical to the plain call."""
    import torch
    wl = synth.WORKLOADS[3]
    mask = synth.make_latents(wl, 0.25)["mask"][0]
    rows = orc.region_rows(mask, wl.n_text, wl.n_ref, "edited_queries")["cache"]
    qkv = synth.make_qkv_full(wl)
    n = wl.n_full
    keep = np.zeros((1, n), np.int32); keep[0, :len(rows)] = rows
    out, kc, vc, status, dev = _run(qkv["q"], qkv["k"], qkv["v"], [n], keep, [len(rows)])
    assert status == 0
    assert np.array_equal(host_f64(kc)[0, :len(rows)], qkv["k"][0, rows].astype(np.float64))
    assert np.array_equal(host_f64(vc)[0, :len(rows)], qkv["v"][0, rows].astype(np.float64))
    assert np.all(host_f64(kc)[0, len(rows):] == -3.0)
    dq, dk, dv, ws = dev
    out2 = torch.full_like(out, -3.0)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.region_attention(dq, dk, dv, None, None, dev_i32([n]), dev_i32([n]), dev_i32([0]), out2,
                             workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0 and torch.equal(out.view(torch.int16), out2.view(torch.int16))
    # sampled rows of the output against the oracle (every row of this shape is covered by
    # test_config3_full_mask_against_vanilla_joint_attention)
    samples = [(0, r, h) for r, h in ((0, 0), (wl.n_text + 7, 5), (n - 1, 23), (4000, 11))]
    empty = np.zeros((1, 0) + qkv["q"].shape[2:])
    want = orc.region_attention_rows(qkv["q"], qkv["k"], qkv["v"], empty, empty, [n], [0], samples)
    g = host_f64(out)
    assert_close(np.stack([g[b, r, h] for b, r, h in samples]), want, "sampled rows")


def test_keep_list_out_of_order_or_out_of_range_is_reported():
    rng = np.random.default_rng(3)
    B, N, H, D = 1, 300, 2, 64
    q, k, v = (_rand_bf16(rng, (B, N, H, D), 0.5) for _ in range(3))
    keep = np.zeros((B, N), np.int32)
    keep[0, :4] = [5, 200, 100, 250]                      # 100 after 200: not ascending
    _, kc, _, status, _ = _run(q, k, v, [N], keep, [4])
    assert status == binding.DEV_BOUNDS
    keep[0, :3] = [5, 100, 299]
    _, kc, _, status, _ = _run(q, k, v, [280], keep, [3])  # row 299 does not exist in a 280-row request
    assert status == binding.DEV_BOUNDS
    assert np.array_equal(host_f64(kc)[0, :2], k[0, [5, 100]].astype(np.float64))
