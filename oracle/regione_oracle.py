"""fp64 CPU oracle for the region-aware denoising step (RegionE, arXiv 2510.25590).

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this file;
only tests, the smoke check and the benchmark's CPU-baseline leg use it.  It
shares no code with the CUDA path and imports nothing from it.

Every function is the plain definition the paper gives, evaluated in float64
with numpy, without blocking, fusion or reordering.  Inputs are arrays whose
values are already bf16-representable (the caller widens them); outputs stay
float64.  Index outputs are int32.

Pins (see tests, marker "not gpu"): straight-line identity, Euler invariance,
planted-mask recovery, index invariants, scatter(gather) round trip, plain
copy for the identity keep list, brute-force loops on tiny shapes, agreement
with a library softmax-attention, split/permutation invariance, uniform-key
mean, dominant-key selection, the E4M3 code table against a library's and its round trip,
the RMS normalisation against a library's and the rotary embedding's relative-position property,
the row-membership counts and partition-of-the-sequence
property, the gamma = 1 closed form of the appendix, planted
decay corrections for the gamma fit, and the zero-edit / full-edit merge cases.
Every function has such a pin.  Two of them implement a *reading* where the paper
leaves the operator open, and are pinned as operators only, not against the paper:
``open_close`` (3x3 structuring element, opening then closing) and ``gamma_fit``
(mean of per-sample norm ratios): for those two choices, parity unpinned.  ``rms_norm``, ``rope`` and
``fresh_qkv`` state operations the paper does not define at all (the editors' own normalisation and
rotary embedding of Q and K): pinned against a library routine and the rotation's textbook
properties, parity unpinned against the paper.  The 8-bit cache functions likewise follow the
published number format, not the paper.
"""
from __future__ import annotations

import numpy as np

COSINE = 0
L2 = 1


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# ----------------------------------------------------------------------------
# Adaptive Region Partition
# ----------------------------------------------------------------------------


def one_step_estimate(x_t, t, v):
    """One-step clean estimate: X_hat_0 = X_t - v * (t - 0).

    One-step estimation equation of the Adaptive Region Partition paragraph
    with t_f = 0; Algorithm 1, the line computing X_hat_0.
    """
    return _f64(x_t) - float(t) * _f64(v)


def token_score(x0_hat, ref, metric):
    """One score per token, reduced over that token's channels.

    metric COSINE: cosine similarity between the estimate and the instruction
    (reference) latent, one value per token (Adaptive Region Partition
    paragraph).  A zero denominator is clamped at 1e-12.
    metric L2: Euclidean distance over the channels (not squared, not averaged).
    """
    a, r = _f64(x0_hat), _f64(ref)
    if metric == COSINE:
        dot = np.sum(a * r, axis=-1)
        den = np.sqrt(np.sum(a * a, axis=-1)) * np.sqrt(np.sum(r * r, axis=-1))
        return dot / np.maximum(den, 1e-12)
    if metric == L2:
        d = a - r
        return np.sqrt(np.sum(d * d, axis=-1))
    raise ValueError("metric")


def edit_mask(score, metric, threshold):
    """mask = 1 (edited) unless the token is similar enough to the reference.

    Cosine: the paper calls a token unedited iff similarity > eta (strict), so
    it is edited iff s <= eta.  L2: edited iff distance > tau, unedited iff
    distance <= tau.
    """
    s = _f64(score)
    thr = float(threshold)
    if metric == COSINE:
        return (s <= thr).astype(np.uint8)
    if metric == L2:
        return (s > thr).astype(np.uint8)
    raise ValueError("metric")


def compact_indices(mask):
    """E_index, U_index (ascending token ids), slot and count for one request.

    Algorithm 1: E_index / U_index used by X[E_index], X[U_index].  A plain
    sequential loop; ``slot[n]`` is the position of token n in ``edit_idx`` or -1.
    Entries of edit_idx past n_edit and of keep_idx past N - n_edit are -1 here
    (the GPU leaves them untouched; tests compare the live prefix only).
    """
    m = np.asarray(mask).astype(bool)
    N = m.shape[0]
    edit_idx = np.full(N, -1, np.int32)
    keep_idx = np.full(N, -1, np.int32)
    slot = np.full(N, -1, np.int32)
    ne = 0
    nk = 0
    for n in range(N):
        if m[n]:
            edit_idx[ne] = n
            slot[n] = ne
            ne += 1
        else:
            keep_idx[nk] = n
            nk += 1
    return edit_idx, keep_idx, slot, ne


def partition(x_t, v, ref, t, metric, threshold):
    """Adaptive Region Partition without the morphological clean-up.

    x_t, v, ref: [B, N, C].  Returns dict(score [B,N] f64, mask u8 [B,N],
    edit_idx, keep_idx, slot int32 [B,N], n_edit int32 [B]).
    """
    x_t, v, ref = _f64(x_t), _f64(v), _f64(ref)
    B, N, _ = x_t.shape
    score = token_score(one_step_estimate(x_t, t, v), ref, metric)
    mask = edit_mask(score, metric, threshold)
    edit_idx = np.empty((B, N), np.int32)
    keep_idx = np.empty((B, N), np.int32)
    slot = np.empty((B, N), np.int32)
    n_edit = np.empty(B, np.int32)
    for b in range(B):
        edit_idx[b], keep_idx[b], slot[b], n_edit[b] = compact_indices(mask[b])
    return dict(score=score, mask=mask, edit_idx=edit_idx, keep_idx=keep_idx, slot=slot,
                n_edit=n_edit)


# ----------------------------------------------------------------------------
# Morphological opening + closing of the edited mask (ARP clean-up step)
# ----------------------------------------------------------------------------


def _erode3(m):
    """3x3 binary erosion; neighbours outside the grid are ignored."""
    rows, cols = m.shape
    out = np.ones_like(m)
    for dr in (-1, 0, 1):
        for dc in (-1, 0, 1):
            for r in range(rows):
                for c in range(cols):
                    rr, cc = r + dr, c + dc
                    if 0 <= rr < rows and 0 <= cc < cols and not m[rr, cc]:
                        out[r, c] = 0
    return out


def _dilate3(m):
    """3x3 binary dilation; neighbours outside the grid are ignored."""
    rows, cols = m.shape
    out = np.zeros_like(m)
    for dr in (-1, 0, 1):
        for dc in (-1, 0, 1):
            for r in range(rows):
                for c in range(cols):
                    rr, cc = r + dr, c + dc
                    if 0 <= rr < rows and 0 <= cc < cols and m[rr, cc]:
                        out[r, c] = 1
    return out


def open_close(mask, grid):
    """Opening (erode, dilate) then closing (dilate, erode) of the edited mask.

    The Adaptive Region Partition paragraph cleans the mask with a morphological
    opening and closing; the structuring element is not given: a 3x3 square on the
    rows x cols token grid is used, out-of-grid neighbours ignored.
    """
    m = np.asarray(mask).astype(np.uint8).reshape(grid)
    m = _dilate3(_erode3(m))
    m = _erode3(_dilate3(m))
    return m.reshape(-1)


# ----------------------------------------------------------------------------
# Token gather / scatter, RIKV cache store
# ----------------------------------------------------------------------------


def gather(src, idx, n):
    """dst[b, j] = src[b, idx[b, j]] for j < n[b]  (X^E = X[E_index]; Algorithm 1).

    Rows j >= n[b] of the result are NaN (unspecified on the GPU).
    """
    src = np.asarray(src)
    idx = np.asarray(idx)
    B = src.shape[0]
    cap = idx.shape[1]
    dst = np.full((B, cap) + src.shape[2:], np.nan, dtype=np.float64)
    for b in range(B):
        for j in range(int(n[b])):
            dst[b, j] = src[b, idx[b, j]]
    return dst


def scatter(dst, src, idx, n):
    """dst[b, idx[b, j]] = src[b, j] for j < n[b]; other rows of dst unchanged.

    The re-gathering of region results by spatial position (end of the
    Adaptive Velocity Decay Cache paragraph; Algorithm 1, the gather line).
    """
    out = np.array(dst, dtype=np.float64, copy=True)
    for b in range(out.shape[0]):
        for j in range(int(n[b])):
            out[b, idx[b, j]] = src[b, j]
    return out


def rikv_store(k_full, v_full, keep_rows, n_keep):
    """K^C, V^C: the retained rows of the last full step's K and V.

    Stabilization Stage paragraph (K and V of every attention layer are kept at
    the last full step), refreshed at forced steps.  k_full, v_full: [B, n_full, H, D];
    keep_rows [B, cap]; returns (k_cache, v_cache) [B, cap, H, D], NaN past n_keep[b].
    """
    return gather(k_full, keep_rows, n_keep), gather(v_full, keep_rows, n_keep)


# ----------------------------------------------------------------------------
# 8-bit (E4M3) variant of the cache.  The paper keeps the cache in the model's precision; this is
# the storage variant of the library, stated here from the published format: 1 sign bit, 4 exponent
# bits (bias 7), 3 mantissa bits, exponent field 0 = subnormal, largest finite value 448, no
# infinities (sign.1111.111 is NaN).
# ----------------------------------------------------------------------------


def e4m3_decode(code):
    """Value of an E4M3 code (uint8 array) in float64; the two NaN codes give NaN."""
    c = np.asarray(code).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 15
    m = c & 7
    mag = np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7.0))
    return np.where((e == 15) & (m == 7), np.nan, sign * mag)


def e4m3_encode(y):
    """Nearest E4M3 code of each value (ties to the even mantissa), magnitudes above 448 saturate
    at 448.  A plain search over the 127 non-negative finite codes, no bit tricks."""
    y = _f64(y)
    grid = e4m3_decode(np.arange(127, dtype=np.uint8))          # 0 .. 448, ascending
    a = np.minimum(np.abs(y), 448.0)
    hi = np.searchsorted(grid, a, side="left")                   # first code with value >= a
    hi = np.minimum(hi, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - grid[lo], grid[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))   # tie: the code with an even last bit
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(y), code | 0x80, code).astype(np.uint8)


def kv_scale_exponent(amax):
    """k of the power-of-two scale 2^k of one (row, head): the smallest k with amax / 2^k <= 448
    (k = 0 for amax = 0, k >= -100)."""
    amax = float(amax)
    if not amax > 0.0:
        return 0
    k = -200
    while amax / 2.0 ** k > 448.0:
        k += 1
    return max(k, -100)


def rikv_store_e4m3(k_full, v_full, keep_rows, n_keep):
    """The retained rows of K and V as E4M3 codes with one scale per (row, head).

    Returns (k_codes, v_codes uint8 [B, cap, H, D], k_scale, v_scale float64 [B, cap, H]); entries past
    n_keep[b] are 0 / NaN."""
    outs = []
    for full in (k_full, v_full):
        full = _f64(full)
        B, _, H, D = full.shape
        cap = np.shape(keep_rows)[1]
        codes = np.zeros((B, cap, H, D), np.uint8)
        scale = np.full((B, cap, H), np.nan)
        for b in range(B):
            for j in range(int(n_keep[b])):
                row = full[b, keep_rows[b][j]]
                for h in range(H):
                    s = 2.0 ** kv_scale_exponent(np.max(np.abs(row[h])))
                    scale[b, j, h] = s
                    codes[b, j, h] = e4m3_encode(row[h] / s)
        outs.append((codes, scale))
    return outs[0][0], outs[1][0], outs[0][1], outs[1][1]


def rikv_load_e4m3(k_codes, v_codes, k_scale, v_scale, n_keep):
    """The cache the attention sees: code value times the row-and-head scale (NaN past n_keep[b])."""
    res = []
    for codes, scale in ((k_codes, k_scale), (v_codes, v_scale)):
        out = e4m3_decode(codes) * np.asarray(scale, np.float64)[..., None]
        for b in range(out.shape[0]):
            out[b, int(n_keep[b]):] = np.nan
        res.append(out)
    return res[0], res[1]


# ----------------------------------------------------------------------------
# Producer of the fresh Q / K / V rows of a region step: gather, per-head RMS normalisation of Q and
# K, rotary position embedding at the rows' own positions in the joint sequence.  The paper does not
# state these two operations (it treats the attention layer of the editors it accelerates as given);
# the editors apply them to Q and K of every attention layer, and what the method adds is that a
# recomputed token keeps its position (Sec. 4 "Region-Aware Generation": the region's tokens are
# gathered and later put back by spatial position), so the row index of the gather is also the
# position of the rotation.  Definitions, from their publications:
#   RMS normalisation   y = x / sqrt(mean(x^2) + eps) * w                     (per row and head, over D)
#   rotary embedding    (a, b) -> (a cos t - b sin t, a sin t + b cos t)      for each of the D/2 pairs,
#     pair i = elements (2i, 2i+1) ("interleaved") or (i, i + D/2) ("half"), angle t = theta[pos, i]
# ----------------------------------------------------------------------------

ROPE_INTERLEAVED = 0
ROPE_HALF = 1


def rms_norm(x, weight=None, eps=1e-6):
    """x / sqrt(mean(x^2 over the last axis) + eps), times `weight` [D] if given."""
    x = _f64(x)
    y = x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return y if weight is None else y * _f64(weight)


def rope(x, cos, sin, layout):
    """Rotates the D/2 pairs of the last axis of x [..., D] by the angles whose cosines and sines are
    cos, sin [..., D/2] (broadcast against x's leading axes)."""
    x = _f64(x)
    D = x.shape[-1]
    cos, sin = _f64(cos), _f64(sin)
    out = np.empty_like(x)
    for i in range(D // 2):
        ia, ib = (2 * i, 2 * i + 1) if layout == ROPE_INTERLEAVED else (i, i + D // 2)
        a, b = x[..., ia], x[..., ib]
        out[..., ia] = a * cos[..., i] - b * sin[..., i]
        out[..., ib] = a * sin[..., i] + b * cos[..., i]
    return out


def fresh_qkv(q_src, k_src, v_src, idx, n, q_weight, k_weight, eps, cos, sin, layout, src_compact=False):
    """Row j < n[b] of the result: source row idx[b, j] of Q, K, V [B, N, H, D] (or, with src_compact,
    source row j of [B, cap, H, D]); Q and K normalised per head and rotated by the angles of
    position idx[b, j] (cos, sin: [positions, D/2]); V copied.  NaN past n[b]."""
    q_src, k_src, v_src = _f64(q_src), _f64(k_src), _f64(v_src)
    B, _, H, D = q_src.shape
    cap = np.shape(idx)[1]
    q = np.full((B, cap, H, D), np.nan)
    k = np.full((B, cap, H, D), np.nan)
    v = np.full((B, cap, H, D), np.nan)
    for b in range(B):
        for j in range(int(n[b])):
            pos = int(idx[b][j])
            r = j if src_compact else pos
            for h in range(H):
                q[b, j, h] = rope(rms_norm(q_src[b, r, h], q_weight, eps), cos[pos], sin[pos], layout)
                k[b, j, h] = rope(rms_norm(k_src[b, r, h], k_weight, eps), cos[pos], sin[pos], layout)
            v[b, j] = v_src[b, r]
    return q, k, v


# ----------------------------------------------------------------------------
# Which rows of the joint sequence are recomputed and which come from the cache
# ----------------------------------------------------------------------------


def region_rows(mask, n_text, n_ref, membership="edited_queries"):
    """Row lists into the joint sequence [text | image | reference] for one request.

    Region-Aware Generation paragraph, the attention equation: the recomputed
    tokens supply the queries and the fresh keys / values, every other token is
    served from the Region-Instruction KV cache.
      ``paper``          : Q = [Q_P, Q_E], fresh = [P, E], cache = [U, I] (the equation as printed:
                           prompt and edited tokens are recomputed; unedited and instruction-image
                           tokens are cached).
      ``edited_queries`` : only the edited image tokens are recomputed; prompt, unedited and
                           instruction-image tokens all come from the cache.
    Inside each group rows ascend, and groups are concatenated in joint-sequence order.
    Returns dict(query, fresh, cache) of int32 arrays.
    """
    m = np.asarray(mask).astype(bool).reshape(-1)
    n_img = m.shape[0]
    query, cache = [], []
    recompute_text = {"paper": True, "edited_queries": False}[membership]
    for row in range(n_text + n_img + n_ref):
        if row < n_text:
            recomputed = recompute_text
        elif row < n_text + n_img:
            recomputed = bool(m[row - n_text])
        else:
            recomputed = False
        (query if recomputed else cache).append(row)
    q = np.asarray(query, np.int32)
    return dict(query=q, fresh=q.copy(), cache=np.asarray(cache, np.int32))


# ----------------------------------------------------------------------------
# Region attention with the Region-Instruction KV cache
# ----------------------------------------------------------------------------


def region_attention(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, scale=None):
    """softmax(Q [K_fresh, K_cache]^T / sqrt(d)) [V_fresh, V_cache].

    The attention equation of the Region-Aware Generation paragraph: queries of
    the recomputed tokens against the concatenation of their own fresh keys
    and the cached keys of everything else.  The concatenation is written out
    literally.  q [B, Nq, H, D]; k/v fresh [B, Nf, H, D]; cache [B, Nc, H, D];
    counts per batch entry.  Rows q >= n_q[b] of the result are NaN.  With no
    key at all the result row is zero.
    """
    q = _f64(q)
    B, Nq, H, D = q.shape
    s = (1.0 / np.sqrt(D)) if scale is None or scale <= 0 else float(scale)
    out = np.full((B, Nq, H, D), np.nan)
    for b in range(B):
        nq, nf, nc = int(n_q[b]), int(n_fresh[b]), int(n_cache[b])
        if nq == 0:
            continue
        if nf + nc == 0:
            out[b, :nq] = 0.0
            continue
        K = np.concatenate([_f64(k_fresh[b, :nf]), _f64(k_cache[b, :nc])], axis=0)
        V = np.concatenate([_f64(v_fresh[b, :nf]), _f64(v_cache[b, :nc])], axis=0)
        for h in range(H):
            logits = (q[b, :nq, h, :] @ K[:, h, :].T) * s
            logits = logits - logits.max(axis=1, keepdims=True)
            p = np.exp(logits)
            p = p / p.sum(axis=1, keepdims=True)
            out[b, :nq, h, :] = p @ V[:, h, :]
    return out


def region_attention_rows(q, k_fresh, v_fresh, k_cache, v_cache, n_fresh, n_cache, samples,
                          scale=None):
    """Same definition, evaluated only at sampled (b, q_row, h) triples.

    Returns [len(samples), D].  Used for parity at sizes where the full oracle
    would take too long.
    """
    D = np.shape(q)[-1]
    s = (1.0 / np.sqrt(D)) if scale is None or scale <= 0 else float(scale)
    res = np.empty((len(samples), D))
    for i, (b, r, h) in enumerate(samples):
        nf, nc = int(n_fresh[b]), int(n_cache[b])
        K = np.concatenate([_f64(k_fresh[b, :nf, h]), _f64(k_cache[b, :nc, h])], axis=0)
        V = np.concatenate([_f64(v_fresh[b, :nf, h]), _f64(v_cache[b, :nc, h])], axis=0)
        logits = (K @ _f64(q[b, r, h])) * s
        logits = logits - logits.max()
        p = np.exp(logits)
        p = p / p.sum()
        res[i] = p @ V
    return res


# ----------------------------------------------------------------------------
# Adaptive Velocity Decay cache
# ----------------------------------------------------------------------------


def decay_factor(dt, gamma):
    """(1 - dt) * gamma: the per-step decay of the velocity norm (decay-factor equation)."""
    return (1.0 - float(dt)) * float(gamma)


def avd_step(running_product, dt, gamma, delta):
    """One step of the AVDCache criterion.

    Criterion = 1 - prod (1 - dt) * gamma accumulated since the cached step
    (criterion equation).  Returns (new_product, reuse).  If the criterion
    exceeds delta the DiT is recomputed: the cache is refreshed and the product
    restarts at 1.  Otherwise the cached velocity times the product is used.
    """
    p = float(running_product) * decay_factor(dt, gamma)
    if 1.0 - p > float(delta):
        return 1.0, False
    return p, True


def avd_schedule(timesteps, gammas, delta, first, last):
    """Decisions for region steps j = first, first-1, ..., last (descending step index).

    The first step of a run always computes (empty cache).  Returns a list of
    (j, reuse, scale) with scale the factor applied to the cached velocity.
    ``timesteps[i]`` = t_i, increasing in i; the step at index j advances from
    t_j to t_{j-1}; its decay factor uses dt = t_{j+1} - t_j and gamma_{t_j}.
    """
    out = []
    prod = 1.0
    have_cache = False
    for j in range(first, last - 1, -1):
        if not have_cache:
            out.append((j, False, 1.0))
            have_cache = True
            prod = 1.0
            continue
        prod, reuse = avd_step(prod, timesteps[j + 1] - timesteps[j], gammas[j], delta)
        out.append((j, reuse, prod if reuse else 1.0))
    return out


def gamma_fit(v, dt):
    """gamma_{t_i} from sampled velocities (decay-factor equation solved for gamma).

    v [S, T1, n] (index i+1 = the earlier step), dt [T1-1].  Per sample the ratio
    ||v_i|| / ||v_{i+1}||, averaged over the samples, divided by the solver factor (1 - dt_i).
    The paper only says gamma is fitted on sampled data; the mean of ratios is this reading.
    Returns (norms [S, T1], gamma [T1-1]).
    """
    v = _f64(v)
    norms = np.sqrt(np.sum(v * v, axis=-1))
    ratio = norms[:, :-1] / norms[:, 1:]
    return norms, ratio.mean(axis=0) / (1.0 - _f64(dt))


def velocity_decay(v_in, scale, dt, x_e, n_edit):
    """v^E = scale * v_in;  X^E_{t_{j-1}} = X^E_{t_j} - dt * v^E  (Euler sampler equation).

    ``scale`` is the accumulated decay product when the cached velocity is
    reused and 1 on a recomputed step.  Rows >= n_edit[b] are returned unchanged.
    Returns (x_e_new, v_used).
    """
    v_in, x_e = _f64(v_in), _f64(x_e)
    v_used = float(scale) * v_in
    x_new = np.array(x_e, copy=True)
    for b in range(x_e.shape[0]):
        ne = int(n_edit[b])
        x_new[b, :ne] = x_e[b, :ne] - float(dt) * v_used[b, :ne]
    return x_new, v_used


# ----------------------------------------------------------------------------
# Merge of the two regions
# ----------------------------------------------------------------------------


def merge(x_full, v_last_full, x_e, slot, dt_unedited):
    """Full image tokens after a run of region steps.

    Edited tokens come from the iterated X^E (by slot); unedited tokens are the
    one-step prediction X^U - v^U * dt with the last full step's velocity
    (one-step estimation equation; Algorithm 1, the two lines before and after
    the inner loop).
    """
    x_full, v_last_full, x_e = _f64(x_full), _f64(v_last_full), _f64(x_e)
    B, N, _ = x_full.shape
    out = np.empty_like(x_full)
    for b in range(B):
        for n in range(N):
            j = int(slot[b, n])
            if j >= 0:
                out[b, n] = x_e[b, j]
            else:
                out[b, n] = x_full[b, n] - float(dt_unedited) * v_last_full[b, n]
    return out


# ----------------------------------------------------------------------------
# Stage schedule (host control flow of Algorithm 1)
# ----------------------------------------------------------------------------


def stage_schedule(T=28, t_st=6, forced=(16,), t_sm=2):
    """Step kinds for steps T, T-1, ..., 1.

    Stabilization: steps T .. T-t_st+1 are full; the last of them stores K/V.
    Bounds [T-t_st, *forced, t_sm-1].  For each consecutive (prev, next):
    region steps prev .. next+2, a merge, then one full step at next+1 that
    refreshes the cache.  Steps below the last bound are full smooth steps.
    Returns a list of (step_index, kind) with kind in {"full", "full_store",
    "region"}; a merge precedes every "full_store" that follows region steps.
    """
    kinds = []
    for i in range(T, T - t_st, -1):
        kinds.append((i, "full_store" if i == T - t_st + 1 else "full"))
    bounds = [T - t_st] + list(forced) + [t_sm - 1]
    for prev, nxt in zip(bounds[:-1], bounds[1:]):
        for j in range(prev, nxt + 1, -1):
            kinds.append((j, "region"))
        kinds.append((nxt + 1, "full_store"))
    for i in range(bounds[-1], 0, -1):
        kinds.append((i, "full"))
    return kinds
