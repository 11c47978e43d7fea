"""Pins of the oracle's E4M3 cache variant: the code table against an independent library's, round
trips, ties, the scale rule's bounds, and the error bound of the format."""
import numpy as np
import pytest

from oracle import regione_oracle as orc


def test_decode_table_matches_the_library_format():
    import torch
    codes = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    mine = orc.e4m3_decode(codes)
    assert np.array_equal(np.isnan(lib), np.isnan(mine)) and np.isnan(mine).sum() == 2
    ok = ~np.isnan(lib)
    assert np.array_equal(lib[ok], mine[ok])
    assert mine[0x7e] == 448.0 and mine[0x38] == 1.0 and mine[0x01] == 2.0 ** -9 and mine[0xbc] == -1.5


def test_encode_is_the_inverse_on_codes_and_rounds_ties_to_even():
    codes = np.array([c for c in range(256) if c not in (0x7f, 0xff, 0x80)], np.uint8)   # (-0 encodes as 0x80 too)
    vals = orc.e4m3_decode(codes)
    assert np.array_equal(orc.e4m3_encode(vals), codes)
    # 1.0625 lies halfway between 1.0 (mantissa 000) and 1.125 (001): the even one; 1.1875 between
    # 1.125 (001) and 1.25 (010): the even one again
    assert orc.e4m3_encode([1.0625])[0] == 0x38 and orc.e4m3_encode([1.1875])[0] == 0x3a
    assert orc.e4m3_encode([1000.0])[0] == 0x7e and orc.e4m3_encode([-1000.0])[0] == 0xfe       # saturation
    assert orc.e4m3_encode([2.0 ** -10])[0] == 0x00 and orc.e4m3_encode([3 * 2.0 ** -10])[0] == 0x02   # subnormal ties


def test_encode_matches_the_library_conversion_on_random_values():
    import torch
    rng = np.random.default_rng(0)
    y = np.concatenate([rng.standard_normal(20000) * 100, rng.standard_normal(20000), rng.standard_normal(20000) * 0.01])
    y = y[np.abs(y) <= 448.0].astype(np.float32)
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = orc.e4m3_encode(y.astype(np.float64))
    zero = (lib & 0x7f) == 0                                  # the sign of a value rounded to zero is kept by both
    assert np.array_equal(lib[~zero], mine[~zero]) and np.array_equal(lib[zero] & 0x7f, mine[zero] & 0x7f)


def test_scale_rule_puts_the_maximum_in_the_top_binade_of_the_format():
    rng = np.random.default_rng(1)
    for amax in np.concatenate([10.0 ** rng.uniform(-20, 20, 200), [448.0, 448.0001, 224.0, 1.0, 2.0 ** -9]]):
        s = 2.0 ** orc.kv_scale_exponent(amax)
        assert 224.0 < amax / s <= 448.0
    assert orc.kv_scale_exponent(0.0) == 0


def test_store_and_load_round_trip_within_the_format_error():
    rng = np.random.default_rng(2)
    B, N, H, D = 2, 40, 3, 64
    k = rng.standard_normal((B, N, H, D)).astype(np.float32) * 0.09
    v = rng.standard_normal((B, N, H, D)).astype(np.float32)
    keep = np.stack([np.sort(rng.permutation(N)[:30]) for _ in range(B)]).astype(np.int32)
    n_keep = np.array([30, 11], np.int32)
    kq, vq, ks, vs = orc.rikv_store_e4m3(k, v, keep, n_keep)
    kd, vd = orc.rikv_load_e4m3(kq, vq, ks, vs, n_keep)
    for b in range(B):
        n = n_keep[b]
        for deq, full in ((kd, k), (vd, v)):
            want = full[b, keep[b, :n]].astype(np.float64)
            err = np.abs(deq[b, :n] - want)
            # half a unit in the last place of a 3-bit mantissa, relative to the element, or half a
            # subnormal step of the scaled format for elements far below the row maximum
            amax = np.max(np.abs(want), axis=-1, keepdims=True)
            assert np.all(err <= np.maximum(np.abs(want) * 2.0 ** -4, amax / 224.0 * 2.0 ** -10))
            assert np.all(np.max(np.abs(deq[b, :n]), axis=-1) <= np.max(np.abs(want), axis=-1) * (1 + 2.0 ** -4))
        assert np.all(np.isnan(kd[b, n:])) and np.all(kq[b, n:] == 0)
