"""Pins for the oracle's region attention and row copies (CPU only)."""
import math

import numpy as np
import pytest

from oracle import regione_oracle as orc


def _rand(shape, seed, std=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * std


def _brute(q, kf, vf, kc, vc, nq, nf, nc, scale):
    """Triple loops with math.exp, keys visited fresh-then-cached."""
    B, _, H, D = q.shape
    out = np.full(q.shape, np.nan)
    for b in range(B):
        keys = [(kf, vf, j) for j in range(nf[b])] + [(kc, vc, j) for j in range(nc[b])]
        for h in range(H):
            for i in range(nq[b]):
                logit = [scale * sum(q[b, i, h, d] * K[b, j, h, d] for d in range(D))
                         for (K, _, j) in keys]
                m = max(logit)
                w = [math.exp(l - m) for l in logit]
                z = sum(w)
                for d in range(D):
                    out[b, i, h, d] = sum(w[a] * V[b, j, h, d] for a, (_, V, j) in enumerate(keys)) / z
    return out


def test_brute_force_tiny():
    B, H, D = 2, 2, 4
    q, kf, vf = _rand((B, 5, H, D), 1), _rand((B, 5, H, D), 2), _rand((B, 5, H, D), 3)
    kc, vc = _rand((B, 7, H, D), 4), _rand((B, 7, H, D), 5)
    nq, nf, nc = [5, 3], [5, 3], [7, 2]
    got = orc.region_attention(q, kf, vf, kc, vc, nq, nf, nc)
    want = _brute(q, kf, vf, kc, vc, nq, nf, nc, 1 / math.sqrt(D))
    assert np.all(np.isnan(got[1, 3:])) and np.all(np.isnan(want[1, 3:]))
    ok = ~np.isnan(want)
    assert np.max(np.abs(got[ok] - want[ok])) < 1e-13
    # explicit scale argument
    got2 = orc.region_attention(q, kf, vf, kc, vc, nq, nf, nc, scale=0.3)
    want2 = _brute(q, kf, vf, kc, vc, nq, nf, nc, 0.3)
    assert np.max(np.abs(got2[ok] - want2[ok])) < 1e-13


def test_full_mask_without_cache_is_ordinary_attention():
    import torch
    B, n, H, D = 1, 33, 3, 16
    q, k, v = _rand((B, n, H, D), 6), _rand((B, n, H, D), 7), _rand((B, n, H, D), 8)
    empty = np.zeros((B, 0, H, D))
    got = orc.region_attention(q, k, v, empty, empty, [n], [n], [0])
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    assert np.max(np.abs(got - want)) < 1e-12


def test_split_and_permutation_invariance():
    B, H, D, n = 1, 2, 8, 40
    q, k, v = _rand((B, 9, H, D), 9), _rand((B, n, H, D), 10), _rand((B, n, H, D), 11)
    empty = np.zeros((B, 0, H, D))
    base = orc.region_attention(q, k, v, empty, empty, [9], [n], [0])
    for cut in (0, 1, 17, n):
        a = orc.region_attention(q, k[:, :cut], v[:, :cut], k[:, cut:], v[:, cut:], [9], [cut], [n - cut])
        assert np.max(np.abs(a - base)) < 1e-13
    perm = np.random.default_rng(12).permutation(n)
    a = orc.region_attention(q, k[:, perm[:13]], v[:, perm[:13]], k[:, perm[13:]], v[:, perm[13:]],
                             [9], [13], [n - 13])
    assert np.max(np.abs(a - base)) < 1e-13


def test_equal_keys_give_mean_of_values():
    B, H, D, n = 1, 2, 8, 12
    q, v = _rand((B, 4, H, D), 13), _rand((B, n, H, D), 14)
    k = np.broadcast_to(_rand((B, 1, H, D), 15), (B, n, H, D)).copy()
    got = orc.region_attention(q, k[:, :5], v[:, :5], k[:, 5:], v[:, 5:], [4], [5], [7])
    assert np.max(np.abs(got - v.mean(axis=1, keepdims=True))) < 1e-13


def test_dominant_key_selects_its_value_row_and_weights_sum_to_one():
    B, H, D, n = 1, 1, 4, 10
    q = np.zeros((B, 2, H, D)); q[..., 0] = 1.0
    k = np.zeros((B, n, H, D)); k[0, 6, 0, 0] = 100.0      # +50 logit margin after 1/sqrt(4)
    v = _rand((B, n, H, D), 16)
    got = orc.region_attention(q, k[:, :3], v[:, :3], k[:, 3:], v[:, 3:], [2], [3], [7])
    assert np.max(np.abs(got[0, :, 0] - v[0, 6, 0])) < 1e-12
    ones = np.ones_like(v)
    k2 = _rand((B, n, H, D), 17)
    got = orc.region_attention(_rand((B, 2, H, D), 18), k2[:, :3], ones[:, :3], k2[:, 3:], ones[:, 3:],
                               [2], [3], [7])
    assert np.max(np.abs(got - 1.0)) < 1e-14


def test_two_key_closed_form():
    # one query, two keys with logits a and b: weights are the logistic of (a - b)
    D = 4
    q = np.zeros((1, 1, 1, D)); q[..., 0] = 2.0
    kf = np.zeros((1, 1, 1, D)); kf[..., 0] = 1.5
    kc = np.zeros((1, 1, 1, D)); kc[..., 0] = -0.5
    vf = np.full((1, 1, 1, D), 10.0); vc = np.full((1, 1, 1, D), -6.0)
    a, b = 2.0 * 1.5 / 2.0, 2.0 * -0.5 / 2.0
    w = 1.0 / (1.0 + math.exp(b - a))
    got = orc.region_attention(q, kf, vf, kc, vc, [1], [1], [1])
    assert abs(got[0, 0, 0, 0] - (w * 10.0 + (1 - w) * -6.0)) < 1e-14


def test_sampled_rows_agree_with_full_and_empty_cases():
    B, H, D = 2, 3, 8
    q, kf, vf = _rand((B, 6, H, D), 19), _rand((B, 6, H, D), 20), _rand((B, 6, H, D), 21)
    kc, vc = _rand((B, 11, H, D), 22), _rand((B, 11, H, D), 23)
    nq, nf, nc = [6, 4], [6, 4], [11, 0]
    full = orc.region_attention(q, kf, vf, kc, vc, nq, nf, nc)
    samples = [(0, 0, 0), (0, 5, 2), (1, 3, 1), (1, 0, 0)]
    rows = orc.region_attention_rows(q, kf, vf, kc, vc, nf, nc, samples)
    for i, (b, r, h) in enumerate(samples):
        assert np.max(np.abs(rows[i] - full[b, r, h])) < 1e-14
    z = orc.region_attention(q, kf, vf, kc, vc, [2, 0], [0, 0], [0, 0])
    assert np.all(z[0, :2] == 0) and np.all(np.isnan(z[1]))


def test_scatter_of_gather_round_trip_touches_nothing_else():
    rng = np.random.default_rng(24)
    B, N, C = 2, 37, 8
    x = rng.standard_normal((B, N, C))
    idx = np.stack([np.sort(rng.permutation(N)[:15]), np.sort(rng.permutation(N)[:15])]).astype(np.int32)
    n = [15, 9]
    g = orc.gather(x, idx, n)
    assert np.array_equal(g[0, :15], x[0, idx[0]]) and np.all(np.isnan(g[1, 9:]))
    poison = np.full_like(x, -777.0)
    s = orc.scatter(poison, g, idx, n)
    for b in range(B):
        live = np.zeros(N, bool); live[idx[b, :n[b]]] = True
        assert np.array_equal(s[b, live], x[b, live])
        assert np.all(s[b, ~live] == -777.0)


def test_store_with_identity_keep_list_is_a_plain_copy():
    rng = np.random.default_rng(25)
    B, n, H, D = 2, 19, 2, 4
    k, v = rng.standard_normal((2, B, n, H, D))
    keep = np.broadcast_to(np.arange(n, dtype=np.int32), (B, n))
    kc, vc = orc.rikv_store(k, v, keep, [n, n])
    assert kc.tobytes() == k.tobytes() and vc.tobytes() == v.tobytes()
    # attention over a stored cache equals attention over the selected rows directly
    keep2 = np.array([[3, 4, 9, 18], [0, 1, 2, 5]], np.int32)
    kc, vc = orc.rikv_store(k, v, keep2, [4, 3])
    assert np.array_equal(kc[0, :4], k[0, keep2[0]]) and np.array_equal(vc[1, :3], v[1, keep2[1, :3]])
