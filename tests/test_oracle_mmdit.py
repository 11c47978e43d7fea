"""Pins for the oracle's stand-in transformer stack run the region-aware way (CPU only): closed forms
and the invariants the method rests on, none of which re-evaluates the stack's own code path."""
import numpy as np
import pytest

from oracle import mmdit_oracle, regione_oracle as orc
from paper_2510_25590_b200 import synth


def _model(membership="paper", zero_mod=False, seed=0):
    n_text, n_img, n_ref, H, D, C, L = 3, 12, 12, 2, 16, 16, 2
    w = synth.make_mmdit_weights(H * D, D, C, n_text, L, seed=seed)
    if zero_mod:
        for k in w:
            if k.startswith("mod"):
                w[k] = np.zeros_like(w[k])
    cos, sin = synth.rope_tables(n_text + n_img + n_ref, D)
    rng = np.random.default_rng(seed + 1)
    ref = rng.standard_normal((1, n_img, C))
    planted = np.zeros((1, n_img), bool); planted[0, [2, 3, 7, 8, 9]] = True
    m = mmdit_oracle.MMDiTOracle(w, n_text, n_img, n_ref, H, D, L, cos, sin, ref, planted, membership)
    x = rng.standard_normal((1, n_img, C))
    return m, x, ref, planted, w


def _lists(planted):
    e = np.flatnonzero(planted[0])
    idx = np.zeros((1, planted.shape[1]), np.int64); idx[0, :len(e)] = e
    return idx, [len(e)]


@pytest.mark.parametrize("membership", ["paper", "edited_queries"])
def test_region_step_on_unchanged_inputs_reproduces_the_full_step(membership):
    """The cache holds exactly what a recomputation would give while nothing has changed, so a region
    step at the same latent and time returns the full step's velocity on the edited tokens."""
    m, x, ref, planted, _ = _model(membership)
    v = m.full(x, 0.7)
    idx, ne = _lists(planted)
    v_e = m.region(x[:, idx[0]], 0.7, idx, ne)
    assert np.allclose(v_e[0, :ne[0]], v[0, idx[0, :ne[0]]], rtol=1e-9, atol=1e-11)
    assert np.all(v_e[0, ne[0]:] == 0.0)


def test_region_step_sees_other_tokens_only_through_the_cache():
    m, x, ref, planted, _ = _model()
    m.full(x, 0.7)
    idx, ne = _lists(planted)
    x2 = x.copy()
    base = m.region(x2[:, idx[0]], 0.6, idx, ne)
    # an edited token's latent matters to every edited token (fresh keys) ...
    x3 = x2.copy(); x3[0, 7] += 0.5
    moved = m.region(x3[:, idx[0]], 0.6, idx, ne)
    assert not np.allclose(moved[0, 0], base[0, 0], rtol=1e-6)
    # ... while nothing outside the region is an input of the region step at all: a new full step with a
    # changed unedited token changes the cache, and only through it the result
    x4 = x.copy(); x4[0, 0] += 0.5
    m.full(x4, 0.7)
    after = m.region(x2[:, idx[0]], 0.6, idx, ne)
    assert not np.allclose(after[0, :ne[0]], base[0, :ne[0]], rtol=1e-6)


def test_closed_form_with_the_modulation_switched_off():
    """All modulation weights zero: every gate is zero, the blocks add nothing, and the velocity is the
    normalised embedding times the output weight (planted tokens), the straight line elsewhere."""
    m, x, ref, planted, w = _model(zero_mod=True)
    v = m.full(x, 0.5)
    h = x[0] @ w["w_in"].astype(np.float64) + w["b_in"].astype(np.float64)
    ln = (h - h.mean(-1, keepdims=True)) / np.sqrt(h.var(-1, keepdims=True) + 1e-6)
    want = ln @ w["w_out"].astype(np.float64)
    assert np.allclose(v[0, planted[0]], want[planted[0]], rtol=1e-12)
    assert np.allclose(v[0, ~planted[0]], (x[0, ~planted[0]] - ref[0, ~planted[0]]) / 0.5, rtol=1e-13)


def test_straight_line_outside_the_planted_region_makes_the_partition_recover_it():
    m, x, ref, planted, _ = _model()
    v = m.full(x, 0.8)
    p = orc.partition(x, v, ref, 0.8, orc.L2, 0.1)
    assert np.array_equal(p["mask"].astype(bool), planted)


def test_full_step_attention_is_library_attention_over_the_joint_sequence():
    """One block, gates forced to one through the bias-free modulation being replaced: compare the
    attention the stack calls with a library routine on the same Q, K, V."""
    import torch
    m, x, ref, planted, _ = _model()
    got = {}
    real = orc.region_attention

    def spy(q, kf, vf, kc, vc, nq, nf, nc):
        out = real(q, kf, vf, kc, vc, nq, nf, nc)
        got.setdefault("calls", []).append((q, kf, vf, out))
        return out

    orc.region_attention = spy
    try:
        m.full(x, 0.7)
    finally:
        orc.region_attention = real
    assert len(got["calls"]) == 2                                           # one per block
    q, k, v, out = got["calls"][0]
    assert q.shape == (1, 27, 2, 16)                                        # every row of the joint sequence
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    sdpa = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    assert np.allclose(out, sdpa, rtol=1e-10, atol=1e-12)
