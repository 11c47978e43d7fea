"""Helpers shared by the GPU parity tests: buffer conversion and error measures."""
import numpy as np

from paper_2510_25590_b200 import synth

MAX_ABS_TOL = 2e-2     # tolerance stated for attention and latent outputs
REL_RMS_TOL = 5e-3


def dev_bf16(x):
    """bf16-representable float32 numpy array -> torch bf16 CUDA tensor with the same values."""
    import torch
    bits = synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32)).reshape(np.shape(x))
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def host_f64(t):
    """torch tensor (any dtype) -> float64 / native numpy array on the host."""
    import torch
    if t.dtype == torch.bfloat16:
        bits = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        return synth.bf16_bits_to_f32(bits).reshape(tuple(t.shape)).astype(np.float64)
    return t.cpu().numpy()


def dev_i32(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def errors(got, want):
    """(max-abs error, relative RMS error) over the entries where `want` is finite."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    ok = np.isfinite(want)
    d = got[ok] - want[ok]
    if d.size == 0:
        return 0.0, 0.0
    rms = np.sqrt(np.mean(want[ok] ** 2))
    return float(np.max(np.abs(d))) if d.size else 0.0, float(np.sqrt(np.mean(d * d)) / rms) if d.size and rms > 0 else 0.0


def assert_close(got, want, what=""):
    assert np.all(np.isfinite(np.asarray(got)[np.isfinite(want)])), f"{what}: non-finite output"
    ma, rr = errors(got, want)
    assert ma <= MAX_ABS_TOL and rr <= REL_RMS_TOL, f"{what}: max-abs {ma:.3e}, rel-RMS {rr:.3e}"
    return ma, rr
