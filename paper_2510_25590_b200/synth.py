"""Seeded synthetic inputs shaped like the paper's three editors.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds none of the method's arithmetic: it only draws numbers,
rounds them to bf16-representable values and lays them out.  It imports
neither the oracle nor the CUDA binding.

The public image-editing suites the paper evaluates on are not reproduced
here; only the *shapes* are taken from the paper (Sec. 3, "Instruction-Based
Editing Model": roughly equal numbers of noise and instruction-image tokens,
far fewer prompt tokens) and from the three editors it accelerates.

Construction of the latents (flow-matching forward process, Preliminary
section, rectified-flow equation): a clean target ``X0`` and a noise sample
``X1`` give ``x_t = (1 - t) X0 + t X1`` and the straight-line velocity
``v = X1 - X0``.  On planted *unedited* tokens ``X0`` is the reference latent
plus a tiny perturbation; on planted *edited* tokens ``X0`` is unrelated to
(slightly anti-correlated with) the reference and the velocity carries a
small extra curvature term.

All floating-point arrays returned are float32 arrays whose values are
exactly representable in bfloat16, so the fp64 oracle and the bf16 GPU path
consume identical numbers.
"""
from __future__ import annotations

import heapq
import math
from dataclasses import dataclass, field

import numpy as np

# ----------------------------------------------------------------------------
# bf16 helpers (storage format only)
# ----------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float32 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float32 array whose every value is bf16-representable (RNE)."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x)).reshape(np.shape(x))


def rng_for(config: int, stream: int) -> np.random.Generator:
    """Counter-based generator (Philox) keyed by ``1000*config + stream``."""
    return np.random.Generator(np.random.Philox(key=1000 * int(config) + int(stream)))


# ----------------------------------------------------------------------------
# workload table
# ----------------------------------------------------------------------------


@dataclass(frozen=True)
class Workload:
    """Shape of one benchmark / parity configuration."""

    config: int
    name: str
    grid: tuple          # latent grid (rows, cols); N = rows*cols image tokens
    n_ref: int           # reference-image ("instruction") tokens
    n_text: int          # prompt tokens
    heads: int
    head_dim: int
    channels: int = 16   # latent channels per token
    batch: int = 1
    mask_kind: str = "rect"     # rect | ellipses | blobs | blob1
    ratios: tuple = (0.25,)     # edit-mask ratio(s)
    metric: str = "cosine"      # cosine | l2
    threshold: float = 0.88
    qkv_std: float = 1.0
    t_partition: float = 22.0 / 28.0   # time at which the partition runs (after 6 of 28 steps)
    extra: dict = field(default_factory=dict)

    @property
    def n_img(self) -> int:
        return self.grid[0] * self.grid[1]

    @property
    def n_full(self) -> int:
        return self.n_text + self.n_img + self.n_ref


WORKLOADS = {
    1: Workload(1, "tiny", (32, 32), 1024, 64, 4, 64, mask_kind="rect", ratios=(0.25,),
                threshold=0.88, qkv_std=1.0),
    2: Workload(2, "flux_kontext_shaped", (64, 64), 4096, 512, 24, 128, mask_kind="ellipses",
                ratios=(0.20,), threshold=0.93, qkv_std=1.0 / math.sqrt(128.0)),
    3: Workload(3, "qwen_image_edit_shaped", (64, 64), 4096, 256, 24, 128, mask_kind="blobs",
                ratios=(0.05, 0.10, 0.25, 0.50, 1.00), threshold=0.80,
                qkv_std=1.0 / math.sqrt(128.0)),
    4: Workload(4, "step1x_edit_shaped_loop", (64, 64), 4096, 256, 24, 128, mask_kind="ellipses",
                ratios=(0.20,), metric="l2", threshold=0.1, qkv_std=1.0 / math.sqrt(128.0),
                extra=dict(hidden=3072, blocks=8, steps=28, mlp_ratio=4)),
    5: Workload(5, "large_resolution_stress", (96, 96), 9216, 512, 24, 128, batch=4,
                mask_kind="blob1", ratios=(0.15,), threshold=0.88,
                qkv_std=1.0 / math.sqrt(128.0)),
}


def scaled_workload(base: Workload, *, grid=None, n_ref=None, n_text=None, heads=None,
                    head_dim=None, batch=None, channels=None) -> Workload:
    """A smaller (or larger) copy of a workload, used by tests that need oracle-sized cases."""
    g = tuple(grid) if grid is not None else base.grid
    return Workload(base.config, base.name + "_scaled", g,
                    n_ref if n_ref is not None else g[0] * g[1],
                    n_text if n_text is not None else base.n_text,
                    heads if heads is not None else base.heads,
                    head_dim if head_dim is not None else base.head_dim,
                    channels if channels is not None else base.channels,
                    batch if batch is not None else base.batch,
                    base.mask_kind, base.ratios, base.metric, base.threshold, base.qkv_std,
                    base.t_partition, dict(base.extra))


# ----------------------------------------------------------------------------
# planted edit masks (1 = edited)
# ----------------------------------------------------------------------------


def mask_rectangle(rng, grid, ratio) -> np.ndarray:
    """One axis-aligned rectangle covering ``ratio`` of the grid at a seeded offset."""
    rows, cols = grid
    target = int(round(ratio * rows * cols))
    h = max(1, int(round(math.sqrt(target * rows / cols))))
    h = min(h, rows)
    w = min(cols, max(1, int(round(target / h))))
    r0 = int(rng.integers(0, rows - h + 1))
    c0 = int(rng.integers(0, cols - w + 1))
    m = np.zeros((rows, cols), dtype=np.uint8)
    m[r0:r0 + h, c0:c0 + w] = 1
    return m.reshape(-1)


def _top_k_mask(fieldv: np.ndarray, k: int) -> np.ndarray:
    """Mask of the k largest entries (ties broken by index, so the count is exact)."""
    flat = fieldv.reshape(-1)
    m = np.zeros(flat.shape[0], dtype=np.uint8)
    if k > 0:
        order = np.argsort(-flat, kind="stable")
        m[order[:k]] = 1
    return m


def mask_ellipses(rng, grid, ratio, count=2) -> np.ndarray:
    """``count`` seeded ellipses; the union covers exactly round(ratio*N) tokens.

    Each ellipse contributes a smooth "inside-ness" field; the union field is
    thresholded by quantile so the total is exact.
    """
    rows, cols = grid
    yy, xx = np.meshgrid(np.arange(rows, dtype=np.float64), np.arange(cols, dtype=np.float64),
                         indexing="ij")
    best = np.full((rows, cols), -np.inf)
    for _ in range(count):
        cy = rng.uniform(0.25, 0.75) * rows
        cx = rng.uniform(0.25, 0.75) * cols
        ay = rng.uniform(0.6, 1.4)
        ax = rng.uniform(0.6, 1.4)
        th = rng.uniform(0.0, math.pi)
        dy, dx = yy - cy, xx - cx
        u = (math.cos(th) * dx + math.sin(th) * dy) / ax
        w = (-math.sin(th) * dx + math.cos(th) * dy) / ay
        best = np.maximum(best, -(u * u + w * w))
    return _top_k_mask(best, int(round(ratio * rows * cols)))


def _smooth_noise(rng, grid, sigma) -> np.ndarray:
    from scipy.ndimage import gaussian_filter
    return gaussian_filter(rng.standard_normal(grid), sigma=sigma, mode="wrap")


def mask_blobs(rng, grid, ratio, sigma=3.0) -> np.ndarray:
    """Random blobs: smoothed noise thresholded by quantile to hit the ratio exactly."""
    rows, cols = grid
    return _top_k_mask(_smooth_noise(rng, grid, sigma), int(round(ratio * rows * cols)))


def mask_single_blob(rng, grid, ratio, sigma=4.0) -> np.ndarray:
    """One connected irregular blob of exactly round(ratio*N) tokens.

    Grown from the maximum of a smoothed noise field by always adding the
    4-neighbour frontier pixel with the largest field value.
    """
    rows, cols = grid
    target = int(round(ratio * rows * cols))
    f = _smooth_noise(rng, grid, sigma)
    m = np.zeros((rows, cols), dtype=np.uint8)
    if target == 0:
        return m.reshape(-1)
    r, c = np.unravel_index(int(np.argmax(f)), f.shape)
    heap = [(-f[r, c], int(r), int(c))]
    seen = np.zeros((rows, cols), dtype=bool)
    seen[r, c] = True
    filled = 0
    while heap and filled < target:
        _, r, c = heapq.heappop(heap)
        m[r, c] = 1
        filled += 1
        for dr, dc in ((1, 0), (-1, 0), (0, 1), (0, -1)):
            rr, cc = r + dr, c + dc
            if 0 <= rr < rows and 0 <= cc < cols and not seen[rr, cc]:
                seen[rr, cc] = True
                heapq.heappush(heap, (-f[rr, cc], rr, cc))
    return m.reshape(-1)


def planted_mask(kind: str, rng, grid, ratio) -> np.ndarray:
    if ratio >= 1.0:
        return np.ones(grid[0] * grid[1], dtype=np.uint8)
    if ratio <= 0.0:
        return np.zeros(grid[0] * grid[1], dtype=np.uint8)
    if kind == "rect":
        return mask_rectangle(rng, grid, ratio)
    if kind == "ellipses":
        return mask_ellipses(rng, grid, ratio)
    if kind == "blobs":
        return mask_blobs(rng, grid, ratio)
    if kind == "blob1":
        return mask_single_blob(rng, grid, ratio)
    raise ValueError(kind)


# ----------------------------------------------------------------------------
# latents for the partition / decay / merge path
# ----------------------------------------------------------------------------


def make_latents(wl: Workload, ratio: float | None = None, *, stream: int = 0,
                 t: float | None = None, curvature: float = 0.05, eps: float = 0.005):
    """Latents with a planted edit mask.

    Returns a dict with float32 (bf16-representable) arrays ``x_t``, ``v``,
    ``ref`` of shape [B, N, C], the planted ``mask`` uint8 [B, N], and ``t``.
    """
    ratio = wl.ratios[0] if ratio is None else ratio
    t = wl.t_partition if t is None else float(t)
    B, N, C = wl.batch, wl.n_img, wl.channels
    x_t = np.empty((B, N, C), np.float32)
    v = np.empty((B, N, C), np.float32)
    ref = np.empty((B, N, C), np.float32)
    mask = np.empty((B, N), np.uint8)
    for b in range(B):
        rng = rng_for(wl.config, 100 * stream + b)
        mrng = rng_for(wl.config, 100 * stream + 50 + b)
        m = planted_mask(wl.mask_kind, mrng, wl.grid, ratio)
        r = rng.standard_normal((N, C))
        noise = rng.standard_normal((N, C))
        z = rng.standard_normal((N, C))
        small = rng.standard_normal((N, C))
        curve = rng.standard_normal((N, C))
        a = 0.3
        x0_unedited = r + eps * small
        x0_edited = math.sqrt(1.0 - a * a) * z - a * r
        e = m.astype(bool)[:, None]
        x0 = np.where(e, x0_edited, x0_unedited)
        vel = noise - x0 + np.where(e, curvature * curve, 0.0)
        x_t[b] = bf16_round(((1.0 - t) * x0 + t * noise).astype(np.float32))
        v[b] = bf16_round(vel.astype(np.float32))
        ref[b] = bf16_round(r.astype(np.float32))
        mask[b] = m
    return dict(x_t=x_t, v=v, ref=ref, mask=mask, t=t)


# ----------------------------------------------------------------------------
# Q/K/V for one attention layer, generated at full joint length
# ----------------------------------------------------------------------------


def make_qkv_full(wl: Workload, *, stream: int = 0, std: float | None = None):
    """Q, K, V over the joint sequence [text | image | reference], [B, n_full, H, D]."""
    std = wl.qkv_std if std is None else std
    shape = (wl.batch, wl.n_full, wl.heads, wl.head_dim)
    out = {}
    for i, name in enumerate(("q", "k", "v")):
        rng = rng_for(wl.config, 100 * stream + 10 + i)
        out[name] = bf16_round((rng.standard_normal(shape, dtype=np.float32) * np.float32(std)))
    return out


# ----------------------------------------------------------------------------
# sampler schedule inputs
# ----------------------------------------------------------------------------


def uniform_timesteps(T: int = 28) -> np.ndarray:
    """t_i = i / T for i = 0..T (t_T = 1, t_0 = 0)."""
    return np.arange(T + 1, dtype=np.float64) / float(T)


def gamma_table(T: int = 28, kind: str = "ones", seed: int = 7) -> np.ndarray:
    """Timestep-aware correction gamma_{t_i}, i = 0..T.

    The paper fits it on sampled data and does not print it; benchmarks use
    either all ones or a seeded table in [0.90, 1.00].
    """
    if kind == "ones":
        return np.ones(T + 1, dtype=np.float64)
    rng = np.random.Generator(np.random.Philox(key=seed))
    return 0.90 + 0.10 * rng.random(T + 1)


# ----------------------------------------------------------------------------
# random weights of the stand-in transformer stack of the sampler-loop configuration
# ----------------------------------------------------------------------------


def rope_tables(n_pos: int, head_dim: int, base: float = 10000.0):
    """cos / sin [n_pos, head_dim / 2] float32 of the angles position * base^(-2i / head_dim)."""
    inv = base ** (-np.arange(head_dim // 2, dtype=np.float64) * 2.0 / head_dim)
    th = np.arange(n_pos, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)


def mmdit_weight_shapes(hidden: int, head_dim: int, channels: int, n_text: int, blocks: int, mlp_ratio: int = 4):
    """Name -> (shape, standard deviation, mean) of every tensor of the stand-in stack (two weight sets
    per block: index 0 for the text rows, 1 for the image and reference rows)."""
    hd, m = hidden, mlp_ratio * hidden
    sh = {"text_emb": ((n_text, hd), 1.0, 0.0), "w_in": ((channels, hd), channels ** -0.5, 0.0),
          "b_in": ((hd,), 0.1, 0.0), "ref_emb": ((hd,), 0.5, 0.0), "t_a": ((hd,), 1.0, 0.0), "t_b": ((hd,), 1.0, 0.0),
          "w_out": ((hd, channels), hd ** -0.5, 0.0)}
    for l in range(blocks):
        sh[f"qn{l}"] = ((head_dim,), 0.1, 1.0)
        sh[f"kn{l}"] = ((head_dim,), 0.1, 1.0)
        for s in range(2):
            sh[f"mod{l}_{s}"] = ((hd, 6 * hd), 0.5 * hd ** -0.5, 0.0)
            sh[f"qkv{l}_{s}"] = ((hd, 3 * hd), hd ** -0.5, 0.0)
            sh[f"o{l}_{s}"] = ((hd, hd), hd ** -0.5, 0.0)
            sh[f"fc1_{l}_{s}"] = ((hd, m), hd ** -0.5, 0.0)
            sh[f"fc2_{l}_{s}"] = ((m, hd), m ** -0.5, 0.0)
    return sh


def make_mmdit_weights(hidden: int, head_dim: int, channels: int, n_text: int, blocks: int, mlp_ratio: int = 4,
                       seed: int = 0):
    """Seeded bf16-representable float32 weights of the stand-in stack (host arrays: test sizes)."""
    rng = np.random.default_rng(seed)
    out = {}
    for name, (shape, std, mean) in mmdit_weight_shapes(hidden, head_dim, channels, n_text, blocks, mlp_ratio).items():
        out[name] = bf16_round((mean + std * rng.standard_normal(shape, dtype=np.float32)).astype(np.float32))
    return out
