"""One region-aware denoising step for one attention layer, as a fixed sequence of C-ABI calls.

This is call sequencing and buffer ownership only (torch tensors are device
buffers): every operation runs in the library's kernels.  The sequence follows
Algorithm 1 of the paper for one layer:

  partition with the joint-sequence row lists (one launch) -> two independent branches, joined
  before the step returns:
    attention branch: RIKV store -> gather Q/K/V of the recomputed rows (one launch) ->
                      region attention writing its rows back at their joint-sequence positions
    latent branch   : gather X^E, v^E (one launch) -> velocity decay + Euler update -> merge with
                      the one-step-predicted unedited tokens (on a side stream)

No step needs a host round trip: per-request counts stay in device memory.
Capacities are host integers chosen by the caller (``plan_capacity`` reads the
edited-token count back once, outside any timed region).
"""
from __future__ import annotations

from dataclasses import dataclass

from . import binding


@dataclass
class StepShapes:
    B: int
    N: int          # image tokens
    n_text: int
    n_ref: int
    C: int          # latent channels
    H: int
    D: int
    ne_cap: int     # capacity for edited tokens (rows of X^E)
    metric: int = binding.METRIC_COSINE
    threshold: float = 0.9
    membership: int = binding.ROWS_EDITED_QUERIES

    @property
    def n_full(self):
        return self.n_text + self.N + self.n_ref

    @property
    def q_cap(self):
        return self.ne_cap + (self.n_text if self.membership == binding.ROWS_PAPER else 0)

    @property
    def c_cap(self):
        return self.n_full          # the cache can never hold more than the joint sequence


def plan_capacity(x_t, v, ref, t, metric, threshold, round_to=128):
    """Runs the partition once and returns max_b n_edit[b] rounded up (one host read-back)."""
    import torch
    B, N, _ = x_t.shape
    dev = x_t.device
    mask = torch.empty((B, N), dtype=torch.uint8, device=dev)
    e, k, s = (torch.empty((B, N), dtype=torch.int32, device=dev) for _ in range(3))
    ne = torch.empty(B, dtype=torch.int32, device=dev)
    binding.partition(x_t, v, ref, t, metric, threshold, mask, e, k, s, ne)
    m = int(ne.max().item())
    return max(round_to, (m + round_to - 1) // round_to * round_to)


class RegionStep:
    """Owns the intermediate buffers of one step and launches its kernels in order."""

    def __init__(self, shp: StepShapes, device="cuda"):
        import torch
        self.shp = shp
        B, N, C, H, D = shp.B, shp.N, shp.C, shp.H, shp.D
        i32, bf = torch.int32, torch.bfloat16
        z = lambda *s, dt=bf: torch.zeros(s, dtype=dt, device=device)
        self.mask = z(B, N, dt=torch.uint8)
        self.edit_idx, self.keep_idx, self.slot = z(B, N, dt=i32), z(B, N, dt=i32), z(B, N, dt=i32)
        self.n_edit, self.n_q, self.n_cache = z(B, dt=i32), z(B, dt=i32), z(B, dt=i32)
        self.query_rows, self.cache_rows = z(B, shp.q_cap, dt=i32), z(B, shp.c_cap, dt=i32)
        self.x_e, self.v_e, self.v_avd = z(B, shp.ne_cap, C), z(B, shp.ne_cap, C), z(B, shp.ne_cap, C)
        self.k_cache, self.v_cache = z(B, shp.c_cap, H, D), z(B, shp.c_cap, H, D)
        self.q_e, self.k_fresh, self.v_fresh = (z(B, shp.q_cap, H, D) for _ in range(3))
        self.o_e = z(B, shp.q_cap, H, D)
        self.o_full = z(B, shp.n_full, H, D)
        self.x_out = z(B, N, C)
        self.dev_status = z(1, dt=i32)
        ws = binding.region_attention_workspace(B, shp.q_cap, shp.q_cap, shp.c_cap, H, D)
        self.workspace = torch.empty(max(ws, 256), dtype=torch.uint8, device=device)
        self.launches = 0
        self._side = torch.cuda.Stream(device=device)
        self._fork, self._join = torch.cuda.Event(), torch.cuda.Event()
        self.attention_events = None      # optional (start, stop) pair recorded around the attention

    def run(self, x_t, v, ref, q_full, k_full, v_full, t, scale, dt, dt_unedited, stream=None,
            store_cache=True):
        """One region-aware step.  ``store_cache=False`` leaves the cache as the last storing call wrote
        it (Algorithm 1 refreshes it at full steps only; valid while the partition is unchanged)."""
        import torch
        s = self.shp
        st = self.dev_status
        b = binding
        b.partition_rows(x_t, v, ref, t, s.metric, s.threshold, self.mask, self.edit_idx,
                         self.keep_idx, self.slot, self.n_edit, s.n_text, s.n_ref, s.membership,
                         self.query_rows, self.n_q, self.cache_rows, self.n_cache, dev_status=st,
                         stream=stream)
        # Two independent branches hang off the partition: the latent branch (gather of X^E and v,
        # velocity decay, merge: small latency-bound kernels) and the attention branch (cache store,
        # gather of Q/K/V, attention, scatter).  The latent branch runs on a side stream so that it
        # falls into the shadow of the cache store; both join before the step returns.
        main = torch.cuda.current_stream() if stream is None else stream
        self._fork.record(main)
        self._side.wait_event(self._fork)
        side = self._side
        b.gather_multi([x_t, v], self.edit_idx, self.n_edit, [self.x_e, self.v_e], dev_status=st,
                       stream=side)
        b.velocity_decay(self.v_e, scale, dt, self.x_e, self.n_edit, v_cache_out=self.v_avd,
                         dev_status=st, stream=side)
        b.merge(x_t, v, self.x_e, self.slot, dt_unedited, self.x_out, dev_status=st, stream=side)
        self._join.record(side)
        if store_cache:
            b.rikv_store(k_full, v_full, self.cache_rows, self.n_cache, self.k_cache, self.v_cache,
                         dev_status=st, stream=stream)
        b.gather_multi([q_full, k_full, v_full], self.query_rows, self.n_q,
                       [self.q_e, self.k_fresh, self.v_fresh], dev_status=st, stream=stream)
        if self.attention_events is not None:
            self.attention_events[0].record(stream)
        # the attention rows go straight to their positions in the joint sequence (o_full)
        b.region_attention_scatter(self.q_e, self.k_fresh, self.v_fresh, self.k_cache, self.v_cache,
                                   self.n_q, self.n_q, self.n_cache, self.o_full, self.query_rows,
                                   workspace=self.workspace, dev_status=st, stream=stream)
        if self.attention_events is not None:
            self.attention_events[1].record(stream)
        main.wait_event(self._join)
        self.launches += 8 if store_cache else 7     # kernels launched (the attention call launches two)
        return self.x_out
