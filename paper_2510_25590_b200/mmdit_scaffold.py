"""Stand-in transformer stack for the sampler-loop configuration (8 random blocks in the benchmark),
run the region-aware way.  Scaffold around the library, not part of it: the paper's editors and their
weights are not available, so the blocks' dense projections, normalisations and activations are
plain torch operations on random weights (library GEMMs), while everything the method is about goes
through the C-ABI: the rotary / RMS-normalised Q, K, V rows (``fresh_qkv``), the attention of a full
step (``region_attention`` with no cache), the Region-Instruction KV cache of every block
(``rikv_store``) and the region step's attention over [fresh | cached] keys (``region_attention``).

It offers the two callbacks the sampler loop (``loop.RegionELoop``) asks of a velocity model:

    full(x, t, store)                 every row of [text | image | reference] through every block; with
                                      ``store`` the blocks' K and V are kept (Sec. 4, "Stabilization Stage")
    region(x_e, t, edit_idx, n_edit)  only the recomputed rows (edited tokens, plus the text rows under the
                                      attention equation as printed) through every block, their queries
                                      attending over their own fresh K, V and the kept K, V of all other rows

Outside a planted mask the velocity is replaced by the straight line to the reference latent, so that
the Adaptive Region Partition has a region to find in a stack that was never trained.  One request
(batch 1); the block definition is stated in the oracle's counterpart of this file.
"""
from __future__ import annotations

from . import binding


class MMDiTScaffold:
    def __init__(self, weights, n_text, n_img, n_ref, heads, head_dim, blocks, cos, sin, ref, planted,
                 membership=binding.ROWS_PAPER):
        import torch
        self.w = weights                                   # name -> bf16 CUDA tensor
        self.n_text, self.n_img, self.n_ref = n_text, n_img, n_ref
        self.n_full = n_text + n_img + n_ref
        self.H, self.D, self.L, self.hidden = heads, head_dim, blocks, heads * head_dim
        self.cos, self.sin, self.ref, self.planted = cos, sin, ref, planted
        self.membership = membership
        self.loop = None
        dev, i32, bf = ref.device, torch.int32, torch.bfloat16
        n, H, D = self.n_full, heads, head_dim
        buf = lambda rows: torch.empty((1, rows, H, D), dtype=bf, device=dev)
        self.k_full = [buf(n) for _ in range(blocks)]       # K, V of every row at the last storing step
        self.v_full = [buf(n) for _ in range(blocks)]
        self.k_cache = [buf(n) for _ in range(blocks)]      # the rows a region step does not recompute
        self.v_cache = [buf(n) for _ in range(blocks)]
        self.scratch = [buf(n) for _ in range(5)]
        self.all_rows = torch.arange(n, dtype=i32, device=dev).view(1, n)
        self.n_all = torch.tensor([n], dtype=i32, device=dev)
        self.zero = torch.zeros(1, dtype=i32, device=dev)
        self.query_rows = torch.zeros((1, n), dtype=i32, device=dev)
        self.cache_rows = torch.zeros((1, n), dtype=i32, device=dev)
        self.n_query, self.n_cache = torch.zeros(1, dtype=i32, device=dev), torch.zeros(1, dtype=i32, device=dev)
        self.dev_status = torch.zeros(1, dtype=i32, device=dev)
        ws = binding.region_attention_workspace(1, n, n, n, H, D)
        self.workspace = torch.empty(max(ws, 256), dtype=torch.uint8, device=dev)
        self._stale = True                                   # row lists / compacted caches need rebuilding
        self._nq = 0
        self.library_launches = 0

    def bind(self, loop):
        """The loop whose partition lists (keep_idx) the region steps read."""
        self.loop = loop
        return self

    # ---- torch pieces (scaffold) ----------------------------------------------------------
    def _ln(self, h):
        import torch
        return torch.nn.functional.layer_norm(h.float(), (self.hidden,), eps=1e-6)

    def _mm(self, a, name, n_text_rows):
        """Rows [text | others] times the weight set of their stream."""
        import torch
        w0, w1 = self.w[f"{name}_0"], self.w[f"{name}_1"]
        if n_text_rows == 0:
            return a @ w1
        return torch.cat([a[:n_text_rows] @ w0, a[n_text_rows:] @ w1])

    def _mods(self, t, l, n_text_rows, rows):
        import torch
        c = torch.tanh(t * self.w["t_a"].float() + self.w["t_b"].float()).to(torch.bfloat16)[None]
        m = [(c @ self.w[f"mod{l}_{s}"]).float() for s in (0, 1)]               # [1, 6 * hidden] per stream
        full = torch.cat([m[0].expand(n_text_rows, -1), m[1].expand(rows - n_text_rows, -1)])
        return full.chunk(6, dim=-1)

    def _blocks(self, h, t, positions, n_rows_dev, n_text_rows, attend, keep_kv):
        import torch
        bf = torch.bfloat16
        rows, H, D, hd = h.shape[0], self.H, self.D, self.hidden
        q_s, k_s, v_s, q_d, o_d = self.scratch              # each [1, rows, H, D]
        for l in range(self.L):
            sh1, sc1, g1, sh2, sc2, g2 = self._mods(t, l, n_text_rows, rows)
            a = (self._ln(h) * (1.0 + sc1) + sh1).to(bf)
            wq = lambda s: self.w[f"qkv{l}_{s}"]
            for j, dst in enumerate((q_s, k_s, v_s)):            # three projections, each into its own buffer
                out = dst.view(-1, hd)[:rows]
                if n_text_rows:
                    torch.matmul(a[:n_text_rows], wq(0)[:, j * hd:(j + 1) * hd], out=out[:n_text_rows])
                torch.matmul(a[n_text_rows:], wq(1)[:, j * hd:(j + 1) * hd], out=out[n_text_rows:])
            k_d, v_d = (self.k_full[l], self.v_full[l]) if keep_kv else (self._tmp("_ktmp", rows), self._tmp("_vtmp", rows))
            binding.fresh_qkv(q_s, k_s, v_s, positions, n_rows_dev,
                              self.w[f"qn{l}"], self.w[f"kn{l}"], 1e-6, self.cos, self.sin, binding.ROPE_INTERLEAVED,
                              q_d, k_d, v_d, src_compact=True, dev_status=self.dev_status)
            self.library_launches += 1
            attend(l, q_d, k_d, v_d, o_d)
            o = o_d.view(-1, hd)[:rows]
            h = (h.float() + g1 * self._mm(o, f"o{l}", n_text_rows).float()).to(bf)
            m = (self._ln(h) * (1.0 + sc2) + sh2).to(bf)
            u = torch.nn.functional.gelu(self._mm(m, f"fc1_{l}", n_text_rows), approximate="tanh")
            h = (h.float() + g2 * self._mm(u, f"fc2_{l}", n_text_rows).float()).to(bf)
        return h

    def _tmp(self, name, rows):
        import torch
        t = getattr(self, name, None)
        if t is None or t.shape[1] != rows:
            t = torch.empty((1, rows, self.H, self.D), dtype=torch.bfloat16, device=self.ref.device)
            setattr(self, name, t)
        return t

    def _blend(self, v_net, x_rows, ref_rows, planted_rows, t):
        import torch
        line = ((x_rows.float() - ref_rows.float()) / t).to(torch.bfloat16)
        return torch.where(planted_rows[:, None], v_net, line)

    # ---- the two calls of the loop ----------------------------------------------------------
    def full(self, x, t, store):
        import torch
        if isinstance(t, (list, tuple)):
            t, store = t[0], store[0]
        w = self.w
        emb = lambda z: z[0] @ w["w_in"] + w["b_in"]
        h = torch.cat([w["text_emb"], emb(x), emb(self.ref) + w["ref_emb"]])

        def attend(l, q, k, v, o):
            binding.region_attention(q, k, v, None, None, self.n_all, self.n_all, self.zero, o,
                                     workspace=self.workspace, dev_status=self.dev_status)
            self.library_launches += 2

        # (the scratch buffers span the whole sequence here, so no slicing copies happen)
        h = self._blocks(h, float(t), self.all_rows, self.n_all, self.n_text, attend, keep_kv=bool(store))
        if store:
            self._stale = True
        v_net = (self._ln(h[self.n_text:self.n_text + self.n_img]).to(torch.bfloat16) @ w["w_out"])
        return self._blend(v_net, x[0], self.ref[0], self.planted[0], float(t))[None]

    def _refresh_lists_and_caches(self, edit_idx, n_edit):
        lp = self.loop
        binding.region_rows(edit_idx, lp.keep_idx, n_edit, self.n_text, self.n_ref, self.membership,
                            self.query_rows, self.n_query, self.cache_rows, self.n_cache, dev_status=self.dev_status)
        for l in range(self.L):
            binding.rikv_store(self.k_full[l], self.v_full[l], self.cache_rows, self.n_cache, self.k_cache[l],
                               self.v_cache[l], dev_status=self.dev_status)
        self.library_launches += 1 + self.L
        self._nq = int(self.n_query.item())                  # one host read per run of region steps: the GEMM sizes
        self._stale = False

    def region(self, x_e, t, edit_idx, n_edit):
        import torch
        if isinstance(t, (list, tuple)):
            t = t[0]
        if self._stale:
            self._refresh_lists_and_caches(edit_idx, n_edit)
        w, nq = self.w, self._nq
        with_text = self.membership == binding.ROWS_PAPER
        nt = self.n_text if with_text else 0
        ne = nq - nt
        h = x_e[0, :ne] @ w["w_in"] + w["b_in"]
        if with_text:
            h = torch.cat([w["text_emb"], h])
        positions = self.query_rows[:, :nq].contiguous()

        def attend(l, q, k, v, o):
            binding.region_attention(q, k, v, self.k_cache[l], self.v_cache[l], self.n_query, self.n_query,
                                     self.n_cache, o, workspace=self.workspace, dev_status=self.dev_status)
            self.library_launches += 2

        h = self._blocks_compact(h, float(t), positions, nt, attend)
        v_net = (self._ln(h[nt:]).to(torch.bfloat16) @ w["w_out"])
        e = edit_idx[0, :ne].long()
        out = torch.zeros_like(x_e)
        out[0, :ne] = self._blend(v_net, x_e[0, :ne], self.ref[0, e], self.planted[0, e], float(t))
        return out

    def _blocks_compact(self, h, t, positions, n_text_rows, attend):
        """The same blocks over a compact set of rows (own buffers of that size)."""
        rows = h.shape[0]
        saved = self.scratch
        self.scratch = [self._tmp(f"_c{i}", rows) for i in range(5)]
        try:
            return self._blocks(h, t, positions, self.n_query, n_text_rows, attend, keep_kv=False)
        finally:
            self.scratch = saved
