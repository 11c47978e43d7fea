"""regione_region_attention_static: the attention entry point that needs no workspace.

Some users of this library cannot allocate device memory at the call site (a server whose arena
already owns all of HBM, a step loop that must avoid the device-wide stall of cudaMalloc), so the
library carries a fixed scratch array for the split-KV partials.  This file checks, through the
C ABI, that the variant gives the same result as the ordinary entry point and as the fp64 oracle,
twice in a row with different inputs (the scratch keeps the first call's contents), and that an
oversized shape is refused.  It is named to be collected last.
"""
import ctypes

import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, dev_i32, host_f64
from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _case(seed, B, nq, nf, nc, H, D):
    rng = np.random.default_rng(seed)
    mk = lambda n: synth.bf16_round(rng.standard_normal((B, n, H, D), dtype=np.float32))
    return mk(nq), mk(nf), mk(nf), mk(nc), mk(nc)


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    import torch
    B, nq, nf, nc, H, D = 2, 300, 290, 2000, 4, 128
    ws_bytes = binding.region_attention_workspace(B, nq, nf, nc, H, D)
    assert ws_bytes > 0, "shape must use split-KV, otherwise no scratch is exercised"
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    n_q, n_f, n_c = dev_i32([nq, nq - 41]), dev_i32([nf, 17]), dev_i32([nc, nc - 333])
    counts = (np.array([nq, nq - 41]), np.array([nf, 17]), np.array([nc, nc - 333]))
    for call, seed in enumerate((11, 12)):
        host = _case(seed, B, nq, nf, nc, H, D)
        q, kf, vf, kc, vc = (dev_bf16(a) for a in host)
        want = torch.full(q.shape, -3.0, dtype=torch.bfloat16, device="cuda")
        got = torch.full(q.shape, -3.0, dtype=torch.bfloat16, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.region_attention(q, kf, vf, kc, vc, n_q, n_f, n_c, want, workspace=ws, dev_status=st)
        binding.region_attention_static(q, kf, vf, kc, vc, n_q, n_f, n_c, got, dev_status=st)
        torch.cuda.synchronize()
        assert int(st[0]) == 0
        w, g = host_f64(want), host_f64(got)
        assert np.array_equal(g[0, nq:], w[0, nq:]) and np.array_equal(g[1, nq - 41:], w[1, nq - 41:])
        assert_close(g[0, :nq], w[0, :nq], f"call {call}, request 0")
        assert_close(g[1, :nq - 41], w[1, :nq - 41], f"call {call}, request 1")
        # and against the fp64 oracle directly, every live row
        ref = orc.region_attention(*host, *counts)
        assert_close(g[0, :nq], ref[0, :nq], f"call {call}, request 0 vs oracle")
        assert_close(g[1, :nq - 41], ref[1, :nq - 41], f"call {call}, request 1 vs oracle")


def test_static_scratch_variant_refuses_shapes_beyond_its_array():
    lib = binding.load()
    B, nq, nf, nc, H, D = 1, 4096, 4096, 4352, 24, 128
    assert binding.region_attention_workspace(B, nq, nf, nc, H, D) > (64 << 20)
    fake = ctypes.c_void_p(4096)
    rc = lib.regione_region_attention_static(fake, fake, fake, fake, fake, fake, fake, fake, B, nq, nf, nc,
                                             H, D, 0.0, fake, None, None)
    assert rc == binding.WORKSPACE_TOO_SMALL
