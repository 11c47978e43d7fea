"""Pins for the oracle's producer of fresh Q / K / V rows: RMS normalisation, rotary embedding, and
their composition with the gather (CPU only).  None of them re-evaluates the oracle's formulas: they
use a library's normalisation, complex multiplication, closed forms and invariants that a dropped
term, a wrong sign, a transposed pair or a position taken from the wrong index would break."""
import numpy as np
import pytest

from oracle import regione_oracle as orc

LAYOUTS = [orc.ROPE_INTERLEAVED, orc.ROPE_HALF]


def _angles(n_pos, D, base=10000.0):
    """The textbook angle table: position times base^(-2i/D)."""
    inv = base ** (-np.arange(D // 2, dtype=np.float64) * 2.0 / D)
    return np.arange(n_pos, dtype=np.float64)[:, None] * inv[None, :]


def test_rms_norm_agrees_with_a_library_routine():
    import torch
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 3, 64))
    w = rng.standard_normal(64)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(w), 1e-6).numpy()
    assert np.allclose(orc.rms_norm(x, w, 1e-6), want, rtol=1e-13, atol=1e-15)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (64,), None, 1e-3).numpy()
    assert np.allclose(orc.rms_norm(x, None, 1e-3), want, rtol=1e-13, atol=1e-15)


def test_rms_norm_invariants():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 128))
    y = orc.rms_norm(x, None, 0.0)
    assert np.allclose(np.mean(y * y, axis=-1), 1.0, rtol=1e-13)               # unit mean square
    assert np.allclose(orc.rms_norm(-3.5 * x, None, 0.0), -y, rtol=1e-13)        # scale drops out, sign stays
    assert np.allclose(orc.rms_norm(np.full(16, 2.0), None, 0.0), 1.0)           # constant row -> ones
    assert np.allclose(orc.rms_norm(x, np.full(128, 0.25), 0.0), 0.25 * y, rtol=1e-13)
    assert np.all(orc.rms_norm(np.zeros(8), None, 1e-6) == 0.0)                  # eps keeps a zero row finite


@pytest.mark.parametrize("layout", LAYOUTS)
def test_rotation_is_complex_multiplication(layout):
    """A pair (a, b) rotated by t is (a + ib) e^{it}: numpy's complex product is the reference."""
    rng = np.random.default_rng(2)
    D = 32
    x = rng.standard_normal((4, D))
    t = rng.uniform(-3, 3, (4, D // 2))
    got = orc.rope(x, np.cos(t), np.sin(t), layout)
    if layout == orc.ROPE_INTERLEAVED:
        z = (x[:, 0::2] + 1j * x[:, 1::2]) * np.exp(1j * t)
        want = np.empty_like(x); want[:, 0::2] = z.real; want[:, 1::2] = z.imag
    else:
        z = (x[:, :D // 2] + 1j * x[:, D // 2:]) * np.exp(1j * t)
        want = np.concatenate([z.real, z.imag], axis=1)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_rotation_special_angles_and_norms(layout):
    D = 8
    x = np.arange(1.0, D + 1.0)
    zero = np.zeros(D // 2)
    assert np.array_equal(orc.rope(x, np.cos(zero), np.sin(zero), layout), x)                 # angle 0: identity
    quarter = orc.rope(x, np.zeros(D // 2), np.ones(D // 2), layout)                          # angle pi/2: (a, b) -> (-b, a)
    if layout == orc.ROPE_INTERLEAVED:
        assert np.array_equal(quarter, [-2, 1, -4, 3, -6, 5, -8, 7])
    else:
        assert np.array_equal(quarter, [-5, -6, -7, -8, 1, 2, 3, 4])
    t = np.array([0.3, -1.1, 2.0, 0.7])
    y = orc.rope(x, np.cos(t), np.sin(t), layout)
    pairs = (lambda v: v[0::2] ** 2 + v[1::2] ** 2) if layout == orc.ROPE_INTERLEAVED else \
        (lambda v: v[:D // 2] ** 2 + v[D // 2:] ** 2)
    assert np.allclose(pairs(y), pairs(x), rtol=1e-13)                                        # a rotation keeps each pair's length
    back = orc.rope(y, np.cos(-t), np.sin(-t), layout)
    assert np.allclose(back, x, rtol=1e-13)                                                   # and is undone by the opposite angle


@pytest.mark.parametrize("layout", LAYOUTS)
def test_rotated_dot_product_depends_on_the_position_difference_only(layout):
    """The property rotary embeddings exist for: <R_m q, R_n k> = <R_{m+s} q, R_{n+s} k>."""
    rng = np.random.default_rng(3)
    D = 64
    q, k = rng.standard_normal(D), rng.standard_normal(D)
    th = _angles(40, D)
    c, s = np.cos(th), np.sin(th)
    dot = lambda m, n: float(orc.rope(q, c[m], s[m], layout) @ orc.rope(k, c[n], s[n], layout))
    assert np.isclose(dot(3, 11), dot(20, 28), rtol=1e-12) and np.isclose(dot(3, 11), dot(0, 8), rtol=1e-12)
    assert not np.isclose(dot(3, 11), dot(3, 12), rtol=1e-6)                                   # (and it does depend on it)
    assert np.isclose(dot(5, 5), float(q @ k), rtol=1e-12)                                      # equal positions: plain dot product


def test_the_two_layouts_differ_by_a_permutation_of_the_elements():
    rng = np.random.default_rng(4)
    D = 16
    x = rng.standard_normal((3, D)); t = rng.uniform(-2, 2, (3, D // 2))
    perm = np.empty(D, int); perm[0::2] = np.arange(D // 2); perm[1::2] = np.arange(D // 2) + D // 2
    # interleaved element 2i / 2i+1 = half-layout element i / i + D/2
    inter = orc.rope(x[:, perm], np.cos(t), np.sin(t), orc.ROPE_INTERLEAVED)
    half = orc.rope(x, np.cos(t), np.sin(t), orc.ROPE_HALF)
    assert np.allclose(inter, half[:, perm], rtol=1e-14)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_fresh_rows_take_the_angles_of_their_own_position(layout):
    """The composition: row j of the result is source row idx[j], normalised, rotated by the angles of
    position idx[j] (not j); V is a plain copy; rows past n are NaN.  Built here from a library
    normalisation and complex multiplication."""
    import torch
    rng = np.random.default_rng(5)
    B, N, H, D = 2, 11, 3, 16
    q, k, v = (rng.standard_normal((B, N, H, D)) for _ in range(3))
    wq, wk = rng.standard_normal(D), rng.standard_normal(D)
    idx = np.array([[9, 2, 5, 0], [1, 10, 0, 0]]); n = [4, 2]
    th = _angles(N, D); c, s = np.cos(th), np.sin(th)
    gq, gk, gv = orc.fresh_qkv(q, k, v, idx, n, wq, wk, 1e-6, c, s, layout)

    def rotate(y, t):
        if layout == orc.ROPE_INTERLEAVED:
            z = (y[..., 0::2] + 1j * y[..., 1::2]) * np.exp(1j * t)
            o = np.empty_like(y); o[..., 0::2] = z.real; o[..., 1::2] = z.imag
            return o
        z = (y[..., :D // 2] + 1j * y[..., D // 2:]) * np.exp(1j * t)
        return np.concatenate([z.real, z.imag], axis=-1)

    for b in range(B):
        for j in range(n[b]):
            r = idx[b, j]
            for src, w, got in ((q, wq, gq), (k, wk, gk)):
                y = torch.nn.functional.rms_norm(torch.from_numpy(src[b, r]), (D,), torch.from_numpy(w), 1e-6).numpy()
                assert np.allclose(got[b, j], rotate(y, th[r]), rtol=1e-12, atol=1e-14)
            assert np.array_equal(gv[b, j], v[b, r])
        assert np.all(np.isnan(gq[b, n[b]:])) and np.all(np.isnan(gk[b, n[b]:])) and np.all(np.isnan(gv[b, n[b]:]))
    # position 0 has angle 0: a gathered row 0 is only normalised
    assert np.allclose(gq[0, 3], orc.rms_norm(q[0, 0], wq, 1e-6), rtol=1e-14)


def test_compact_sources_are_the_gather_done_beforehand():
    rng = np.random.default_rng(6)
    B, N, H, D = 1, 9, 2, 8
    q, k, v = (rng.standard_normal((B, N, H, D)) for _ in range(3))
    idx = np.array([[7, 1, 4]]); n = [3]
    th = _angles(N, D); c, s = np.cos(th), np.sin(th)
    a = orc.fresh_qkv(q, k, v, idx, n, None, None, 1e-6, c, s, orc.ROPE_HALF)
    b = orc.fresh_qkv(q[:, idx[0]], k[:, idx[0]], v[:, idx[0]], idx, n, None, None, 1e-6, c, s, orc.ROPE_HALF, src_compact=True)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
