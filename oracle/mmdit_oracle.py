"""fp64 statement of the stand-in transformer stack of the sampler-loop configuration, run the
region-aware way (Sec. 4: full steps that save K and V of every attention layer, region steps that
recompute only the region's rows against that cache).

TEST INFRASTRUCTURE ONLY (same rules as regione_oracle): shares no code with the CUDA path.

The stack is scaffold: random weights, no training, not from the paper (its editors' weights are
not available).  What follows the paper is how it is *run*: at a full step every row of the joint
sequence [text | image | reference] goes through every block and the blocks' K and V (as they
enter the softmax) are kept; at a region step only the recomputed rows go through the blocks, and
in every block their queries attend over [their own fresh K, V | the kept K, V of all other rows]
(the attention equation of "Region-Aware Generation"), through ``regione_oracle.region_attention``.
Its velocity is blended with a planted region so that the partition has something to find: outside
the planted mask the velocity is the straight line to the reference latent.

A block (weights index s = 0 for text rows, 1 for image and reference rows; all plain definitions):
    (shift1, scale1, gate1, shift2, scale2, gate2) = c(t) @ mod_s,   c(t) = tanh(t * t_a + t_b)
    a = LN(h) * (1 + scale1) + shift1;  q, k, v = split(a @ qkv_s) into heads
    q, k <- rotary(rms_norm(., qn / kn), angles of the row's position)
    h += gate1 * (attention(q, k, v) @ o_s);  m = LN(h) * (1 + scale2) + shift2
    h += gate2 * (gelu_tanh(m @ fc1_s) @ fc2_s)
and the velocity of the image tokens is LN(h_image) @ w_out.
"""
from __future__ import annotations

import numpy as np

from oracle import regione_oracle as orc


def _ln(x):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + 1e-6)


def _gelu_tanh(x):
    return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))


class MMDiTOracle:
    def __init__(self, weights, n_text, n_img, n_ref, heads, head_dim, blocks, cos, sin, ref, planted,
                 membership="paper"):
        self.w = {k: np.asarray(v, np.float64) for k, v in weights.items()}
        self.n_text, self.n_img, self.n_ref = n_text, n_img, n_ref
        self.H, self.D, self.L = heads, head_dim, blocks
        self.cos, self.sin = np.asarray(cos, np.float64), np.asarray(sin, np.float64)
        self.ref = np.asarray(ref, np.float64)             # [1, n_img, C]
        self.planted = np.asarray(planted).astype(bool)    # [1, n_img]
        self.membership = membership
        self.k_full = [None] * blocks                      # K, V of every row at the last full step
        self.v_full = [None] * blocks
        self.stream = np.concatenate([np.zeros(n_text, int), np.ones(n_img + n_ref, int)])

    # ---- pieces ---------------------------------------------------------------------------
    def _embed(self, x_rows, which):
        w = self.w
        if which == "text":
            return w["text_emb"].copy()
        h = x_rows @ w["w_in"] + w["b_in"]
        return h + w["ref_emb"] if which == "ref" else h

    def _per_stream(self, x, streams, name):
        """Row-wise x @ W_s with the weight set of each row's stream."""
        out = None
        for s in (0, 1):
            sel = streams == s
            if not sel.any():
                continue
            y = x[sel] @ self.w[f"{name}_{s}"]
            if out is None:
                out = np.zeros((x.shape[0], y.shape[1]))
            out[sel] = y
        return out

    def _mods(self, t, l, streams):
        c = np.tanh(t * self.w["t_a"] + self.w["t_b"])
        m = np.stack([c @ self.w[f"mod{l}_{s}"] for s in (0, 1)])[streams]      # [rows, 6 * hidden]
        return np.split(m, 6, axis=-1)

    def _blocks(self, h, t, positions, streams, attend):
        """h [rows, hidden] through all blocks; attend(l, q, k, v) -> o, all [rows, H, D]."""
        H, D = self.H, self.D
        for l in range(self.L):
            sh1, sc1, g1, sh2, sc2, g2 = self._mods(t, l, streams)
            a = _ln(h) * (1.0 + sc1) + sh1
            qkv = self._per_stream(a, streams, f"qkv{l}")
            q, k, v = (z.reshape(-1, H, D) for z in np.split(qkv, 3, axis=-1))
            cs, sn = self.cos[positions][:, None, :], self.sin[positions][:, None, :]
            q = orc.rope(orc.rms_norm(q, self.w[f"qn{l}"], 1e-6), cs, sn, orc.ROPE_INTERLEAVED)
            k = orc.rope(orc.rms_norm(k, self.w[f"kn{l}"], 1e-6), cs, sn, orc.ROPE_INTERLEAVED)
            o = attend(l, q, k, v).reshape(-1, H * D)
            h = h + g1 * self._per_stream(o, streams, f"o{l}")
            m = _ln(h) * (1.0 + sc2) + sh2
            h = h + g2 * self._per_stream(_gelu_tanh(self._per_stream(m, streams, f"fc1_{l}")), streams, f"fc2_{l}")
        return h

    def _blend(self, v_net, x_rows, ref_rows, planted_rows, t):
        return np.where(planted_rows[:, None], v_net, (x_rows - ref_rows) / t)

    # ---- the two calls of the loop ----------------------------------------------------------
    def full(self, x, t):
        """Velocity of all image tokens [1, n_img, C]; K and V of every block are kept."""
        x = np.asarray(x, np.float64)
        h = np.concatenate([self._embed(None, "text"), self._embed(x[0], "img"), self._embed(self.ref[0], "ref")])
        n = h.shape[0]

        def attend(l, q, k, v):
            self.k_full[l], self.v_full[l] = k[None], v[None]
            return orc.region_attention(q[None], k[None], v[None], k[None, :0], v[None, :0], [n], [n], [0])[0]

        h = self._blocks(h, t, np.arange(n), self.stream, attend)
        v_net = _ln(h[self.n_text:self.n_text + self.n_img]) @ self.w["w_out"]
        return self._blend(v_net, x[0], self.ref[0], self.planted[0], t)[None]

    def region(self, x_e, t, edit_idx, n_edit):
        """Velocity of the edited tokens [1, cap, C] (rows past n_edit zero): only the recomputed rows go
        through the blocks; the other rows' K and V come from the last full step."""
        x_e = np.asarray(x_e, np.float64)
        ne = int(n_edit[0])
        mask = np.zeros(self.n_img, np.uint8)
        mask[np.asarray(edit_idx[0][:ne], int)] = 1
        rows = orc.region_rows(mask, self.n_text, self.n_ref, "paper" if self.membership == "paper" else "edited_queries")
        qr, cr = rows["query"], rows["cache"]
        nq, nc = len(qr), len(cr)
        with_text = self.membership == "paper"
        h = self._embed(x_e[0, :ne], "img")
        if with_text:
            h = np.concatenate([self._embed(None, "text"), h])
        streams = self.stream[qr]

        def attend(l, q, k, v):
            kc, vc = orc.rikv_store(self.k_full[l], self.v_full[l], cr[None], [nc])
            return orc.region_attention(q[None], k[None], v[None], kc, vc, [nq], [nq], [nc])[0]

        h = self._blocks(h, t, qr, streams, attend)
        v_net = _ln(h[-ne:] if ne else h[:0]) @ self.w["w_out"]
        e = np.asarray(edit_idx[0][:ne], int)
        out = np.zeros_like(x_e)
        out[0, :ne] = self._blend(v_net, x_e[0, :ne], self.ref[0, e], self.planted[0, e], t)
        return out
