"""Host control flow of the region-aware sampler (Algorithm 1 of the paper) over the C-ABI calls.

The loop owns the latent state and sequences library calls; it performs no arithmetic itself.
What it needs from outside is the velocity model (the DiT of the paper, a stand-in in tests):

    model.full(x, t, store)            -> v            velocity of all N image tokens at time t
                                                        (``store`` = this step refreshes the RIKV cache)
    model.region(x_e, t, edit_idx, n_edit) -> v_e      velocity of the edited tokens only

Both take and return bf16 CUDA tensors.  Everything else is a library call: the Euler update of a
full step and of a region step (``velocity_decay``), the partition after the stabilization steps,
the gather of X^E, the AVDCache criterion (``avd_step``, host scalar), the decayed cached velocity,
and the merge with the one-step-predicted unedited tokens at the end of every run of region steps.

Schedule (``kinds``): one character per sampling step, 'F' = full step, 'R' = region step, in the
order the sampler takes them (time decreasing).  ``paper_schedule`` and ``alternating_schedule``
build the two schedules the tests and the benchmark use.
"""
from __future__ import annotations

from dataclasses import dataclass, field

from . import binding


def paper_schedule(T=28, t_st=6, forced=(16,), t_sm=2):
    """Stage schedule of the paper's implementation details, steps indexed T .. 1.

    Stabilization: steps T .. T-t_st+1 full.  Bounds [T-t_st, *forced, t_sm-1]; for consecutive
    (prev, next): region steps prev .. next+2, then one full step at next+1 (cache refresh).  The
    steps below the last bound are full smooth steps.  Returns (kinds, partition_after) where
    partition_after is the number of steps taken before the partition.
    """
    kinds = ["F"] * t_st
    bounds = [T - t_st] + list(forced) + [t_sm - 1]
    for prev, nxt in zip(bounds[:-1], bounds[1:]):
        kinds += ["R"] * (prev - nxt - 1) + ["F"]
    kinds += ["F"] * bounds[-1]
    assert len(kinds) == T, len(kinds)
    return "".join(kinds), t_st


def alternating_schedule(T=28, first_full=6, refresh_every=5, last_full=2):
    """Steps k = 1 .. T: full steps 1 .. first_full, then every ``refresh_every``-th step and the last
    ``last_full`` + 1 steps; the rest are region steps."""
    kinds = []
    for k in range(1, T + 1):
        full = k <= first_full or k > T - last_full - 1 or (k - first_full) % refresh_every == 0
        kinds.append("F" if full else "R")
    return "".join(kinds), first_full


@dataclass
class LoopConfig:
    kinds: str                       # 'F' / 'R' per step
    partition_after: int             # partition runs after this many steps
    timesteps: list                  # t before step k, k = 0 .. T, decreasing; timesteps[T] = end time
    gammas: list                     # timestep-aware decay correction per step
    delta: float                     # AVDCache threshold
    metric: int = binding.METRIC_COSINE
    threshold: float = 0.9


@dataclass
class LoopTrace:
    """What happened, for tests and reports."""
    steps: list = field(default_factory=list)        # (k, kind, 'full' | 'compute' | 'reuse', scale)
    model_full_calls: int = 0
    model_region_calls: int = 0
    launches: int = 0


class RegionELoop:
    """Buffers and call sequence of one edit (a batch of B independent requests sharing the schedule)."""

    def __init__(self, B, N, C, cfg: LoopConfig, device="cuda"):
        import torch
        self.B, self.N, self.C, self.cfg = B, N, C, cfg
        i32, bf = torch.int32, torch.bfloat16
        z = lambda *s, dt=bf: torch.zeros(s, dtype=dt, device=device)
        self.mask = z(B, N, dt=torch.uint8)
        self.edit_idx, self.keep_idx, self.slot = z(B, N, dt=i32), z(B, N, dt=i32), z(B, N, dt=i32)
        self.n_edit = z(B, dt=i32)
        self.n_all = torch.full((B,), N, dtype=i32, device=device)
        self.x_e, self.v_cache = z(B, N, C), z(B, N, C)      # capacity N: no host read-back needed
        self.x_run_start, self.v_last_full = z(B, N, C), z(B, N, C)
        self.dev_status = z(1, dt=i32)
        self.hook = None             # optional callable(event: str, k: int, tensors: dict)

    @staticmethod
    def _copy(dst, src, stream):
        """Device-to-device copy ordered on the same stream as the library calls around it."""
        import torch
        if stream is None:
            dst.copy_(src)
        else:
            with torch.cuda.stream(stream):
                dst.copy_(src)

    def _emit(self, event, k, **tensors):
        if self.hook is not None:
            self.hook(event, k, tensors)

    def run(self, x, ref, model, stream=None):
        """Runs all steps on ``x`` [B, N, C] bf16 (updated in place); returns (x, trace)."""
        cfg, b, st = self.cfg, binding, self.dev_status
        ts = cfg.timesteps
        tr = LoopTrace()
        partitioned = False
        in_run = False
        t_run = None
        product, have_cache = 1.0, False
        for k, kind in enumerate(cfg.kinds):
            t_cur, t_next = float(ts[k]), float(ts[k + 1])
            dt = t_cur - t_next
            if kind == "F":
                if in_run:
                    # end of a run of region steps: edited tokens from X^E, unedited tokens by one
                    # step of the last full velocity over the whole run
                    self._emit("merge_in", k, x=self.x_run_start, v=self.v_last_full, x_e=self.x_e,
                               slot=self.slot, dt_unedited=t_run - t_cur)
                    b.merge(self.x_run_start, self.v_last_full, self.x_e, self.slot, t_run - t_cur, x,
                            dev_status=st, stream=stream)
                    self._emit("merge_out", k, x=x)
                    tr.launches += 1
                    in_run = False
                v = model.full(x, t_cur, partitioned or k + 1 == cfg.partition_after)
                tr.model_full_calls += 1
                self._copy(self.v_last_full, v, stream)
                self._emit("euler_in", k, x=x, v=v, dt=dt)
                b.velocity_decay(v, 1.0, dt, x, self.n_all, dev_status=st, stream=stream)
                self._emit("euler_out", k, x=x)
                tr.launches += 1
                tr.steps.append((k, kind, "full", 1.0))
                if k + 1 == cfg.partition_after:
                    self._emit("partition_in", k, x=x, v=v, ref=ref, t=t_next)
                    b.partition(x, v, ref, t_next, cfg.metric, cfg.threshold, self.mask, self.edit_idx,
                                self.keep_idx, self.slot, self.n_edit, dev_status=st, stream=stream)
                    self._emit("partition_out", k, mask=self.mask, edit_idx=self.edit_idx, slot=self.slot,
                               n_edit=self.n_edit)
                    tr.launches += 1
                    partitioned = True
                continue
            # ---- region step ----
            if not partitioned:
                raise binding.RegionEError("a region step was scheduled before the partition")
            if not in_run:
                self._copy(self.x_run_start, x, stream)
                b.gather(x, self.edit_idx, self.n_edit, self.x_e, dev_status=st, stream=stream)
                tr.launches += 1
                in_run, t_run = True, t_cur
                product, have_cache = 1.0, False
            reuse = False
            if have_cache:
                product, reuse = b.avd_step(product, float(ts[k - 1]) - t_cur, float(cfg.gammas[k]), cfg.delta)
            if reuse:
                self._emit("decay_in", k, v=self.v_cache, x_e=self.x_e, scale=product, dt=dt, n_edit=self.n_edit)
                b.velocity_decay(self.v_cache, product, dt, self.x_e, self.n_edit, dev_status=st, stream=stream)
                tr.steps.append((k, kind, "reuse", product))
            else:
                v_e = model.region(self.x_e, t_cur, self.edit_idx, self.n_edit)
                tr.model_region_calls += 1
                self._emit("decay_in", k, v=v_e, x_e=self.x_e, scale=1.0, dt=dt, n_edit=self.n_edit)
                b.velocity_decay(v_e, 1.0, dt, self.x_e, self.n_edit, v_cache_out=self.v_cache,
                                 dev_status=st, stream=stream)
                product, have_cache = 1.0, True
                tr.steps.append((k, kind, "compute", 1.0))
            self._emit("decay_out", k, x_e=self.x_e)
            tr.launches += 1
        if in_run:
            t_end = float(ts[len(cfg.kinds)])
            self._emit("merge_in", len(cfg.kinds), x=self.x_run_start, v=self.v_last_full, x_e=self.x_e,
                       slot=self.slot, dt_unedited=t_run - t_end)
            b.merge(self.x_run_start, self.v_last_full, self.x_e, self.slot, t_run - t_end, x,
                    dev_status=st, stream=stream)
            self._emit("merge_out", len(cfg.kinds), x=x)
            tr.launches += 1
        return x, tr
