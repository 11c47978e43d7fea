"""The C-ABI library loads without a GPU, exports every symbol the header declares, validates
arguments on the host, and its host-only entry points agree with the oracle (CPU only)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_symbols():
    text = open(os.path.join(ROOT, "include", "regione.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(regione_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2510_25590_b200 import build
    build.build()
    lib = binding.load()
    names = _header_symbols()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.SIGNATURES) == names          # the binding covers exactly the header
    assert binding.version() >= 100
    assert binding.status_string(binding.UNSUPPORTED) == "REGIONE_UNSUPPORTED"


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(binding.RegionEError):
        binding.load(str(tmp_path / "nope.so"))


def test_argument_validation_happens_on_the_host():
    lib = binding.load()
    null = None
    t1 = (ctypes.c_float * 1)(0.5)
    assert lib.regione_partition(null, null, null, 1, 8, 16, t1, 0, 0.9, null, null, null, null, null,
                                 null, null, null) == binding.INVALID_ARG
    fake = ctypes.c_void_p(4096)
    assert lib.regione_partition(fake, fake, fake, 1, 8, 12, t1, 0, 0.9, fake, fake, fake, fake, fake,
                                 null, null, null) == binding.UNSUPPORTED         # C % 8 != 0
    assert lib.regione_partition(fake, fake, fake, 1, 8, 16, t1, 7, 0.9, fake, fake, fake, fake, fake,
                                 null, null, null) == binding.INVALID_ARG         # unknown metric
    assert lib.regione_partition(fake, fake, fake, 1, 8, 16, null, 0, 0.9, fake, fake, fake, fake, fake,
                                 null, null, null) == binding.INVALID_ARG         # no per-request times
    # one request may hold at most 2^20 tokens
    assert lib.regione_partition(fake, fake, fake, 1, (1 << 20) + 1, 16, t1, 0, 0.9, fake, fake, fake, fake,
                                 fake, null, null, null) == binding.UNSUPPORTED
    odd = ctypes.c_void_p(4100)
    assert lib.regione_gather(odd, fake, fake, 1, 4, 4, 4, 32, fake, null, null) == binding.INVALID_ARG
    assert lib.regione_gather(fake, fake, fake, 1, 4, 4, 4, 24, fake, null, null) == binding.UNSUPPORTED
    assert lib.regione_scatter(fake, fake, fake, 1, 8, 4, 8, 32, fake, null, null) == binding.INVALID_ARG
    assert lib.regione_rikv_store(fake, fake, fake, fake, 1, 8, 8, 3, 3, fake, fake, null, null) \
        == binding.UNSUPPORTED
    # the producer of fresh Q / K / V rows: head sizes 64 and 128, a known pair layout, tables required
    assert lib.regione_fresh_qkv(fake, fake, fake, fake, fake, 1, 8, 4, 2, 96, 0, null, null, 1e-6, fake, fake, 0,
                                 fake, fake, fake, null, null) == binding.UNSUPPORTED
    assert lib.regione_fresh_qkv(fake, fake, fake, fake, fake, 1, 8, 4, 2, 64, 0, null, null, 1e-6, fake, fake, 2,
                                 fake, fake, fake, null, null) == binding.INVALID_ARG
    assert lib.regione_fresh_qkv(fake, fake, fake, fake, fake, 1, 8, 4, 2, 64, 0, null, null, 1e-6, null, fake, 0,
                                 fake, fake, fake, null, null) == binding.INVALID_ARG
    assert lib.regione_fresh_qkv(fake, fake, fake, fake, fake, 1, 8, 4, 2, 64, 1, odd, null, 1e-6, fake, fake, 0,
                                 fake, fake, fake, null, null) == binding.INVALID_ARG
    assert lib.regione_fresh_qkv(fake, fake, fake, fake, fake, 1, 8, 0, 2, 64, 1, null, null, 1e-6, fake, fake, 1,
                                 fake, fake, fake, null, null) == binding.OK          # nothing to do
    # the 8-bit cache: head sizes 64 and 128 only, 16-byte aligned buffers, counts required
    assert lib.regione_rikv_store_e4m3(fake, fake, fake, fake, 1, 8, 8, 3, 96, fake, fake, fake, fake, null,
                                       null) == binding.UNSUPPORTED
    assert lib.regione_rikv_store_e4m3(fake, fake, fake, null, 1, 8, 8, 3, 64, fake, fake, fake, fake, null,
                                       null) == binding.INVALID_ARG
    assert lib.regione_rikv_store_e4m3(fake, fake, fake, fake, 1, 8, 8, 3, 64, odd, fake, fake, fake, null,
                                       null) == binding.INVALID_ARG
    assert lib.regione_rikv_store_e4m3(fake, fake, fake, fake, 0, 8, 8, 3, 64, fake, fake, fake, fake, null,
                                       null) == binding.OK                        # nothing to do
    assert lib.regione_rikv_load_e4m3(fake, fake, fake, fake, fake, 1, 8, 3, 32, fake, fake, null, null) \
        == binding.UNSUPPORTED
    assert lib.regione_rikv_load_e4m3(fake, fake, null, fake, fake, 1, 8, 3, 128, fake, fake, null, null) \
        == binding.INVALID_ARG
    assert lib.regione_rikv_load_e4m3(fake, fake, fake, fake, fake, 1, 0, 3, 128, fake, fake, null, null) \
        == binding.OK
    assert lib.regione_region_attention(fake, fake, fake, fake, fake, fake, fake, fake, 1, 8, 8, 8, 2, 96,
                                        0.0, fake, null, 0, null, null) == binding.UNSUPPORTED
    assert lib.regione_region_attention(fake, null, null, fake, fake, fake, fake, fake, 1, 8, 8, 8, 2, 64,
                                        0.0, fake, null, 0, null, null) == binding.INVALID_ARG
    assert lib.regione_velocity_decay(fake, t1, t1, fake, null, fake, 1, 8, 10, null, null) \
        == binding.UNSUPPORTED
    assert lib.regione_velocity_decay(fake, null, t1, fake, null, fake, 1, 8, 16, null, null) \
        == binding.INVALID_ARG
    assert lib.regione_merge(fake, fake, null, fake, t1, 1, 8, 4, 16, fake, null, null) \
        == binding.INVALID_ARG
    assert lib.regione_merge(fake, fake, fake, fake, null, 1, 8, 4, 16, fake, null, null) \
        == binding.INVALID_ARG
    assert lib.regione_crosscheck_region_attention(fake, fake, fake, fake, fake, fake, fake, fake, 1, 8, 8, 8,
                                                   2, 96, 0.0, fake, null, null) == binding.UNSUPPORTED
    assert lib.regione_selftest_bounded_wait(0, null, null, null) == binding.INVALID_ARG
    assert lib.regione_selftest_bounded_wait(10 ** 9, null, null, null) == binding.INVALID_ARG
    assert lib.regione_mask_open_close(fake, 1, 200, 200, ctypes.c_void_p(8192), fake, fake, fake, fake,
                                       null, null) == binding.UNSUPPORTED
    assert lib.regione_region_attention_workspace(1, 128, 128, 128, 4, 96) == 0


def test_avd_step_matches_oracle():
    T = 28
    ts = np.arange(T + 1) / T
    g = 0.9 + 0.1 * np.random.default_rng(5).random(T + 1)
    for delta in (-1.0, 0.02, 0.04, 0.1, 1.0):
        p_lib = p_orc = 1.0
        for j in range(21, 2, -1):
            dt = ts[j + 1] - ts[j]
            p_lib, r_lib = binding.avd_step(p_lib, dt, g[j], delta)
            p_orc, r_orc = orc.avd_step(p_orc, dt, g[j], delta)
            assert r_lib == r_orc and abs(p_lib - p_orc) < 1e-15
    with pytest.raises(binding.RegionEError):
        binding._check(binding.load().regione_avd_step(None, 0.1, 1.0, 0.1, None), "avd")
