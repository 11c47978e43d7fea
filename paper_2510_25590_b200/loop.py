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

Requests of one batch need not be at the same step (a request that joined the batch later, or the
conditional / unconditional pair of one guided request, which is simply two batch entries).  With
``offsets`` request b takes its step k at tick ``offsets[b] + k``; at every tick the Euler updates of
all requests share their launches, each request with its own time, step length and decay product,
and a request that has nothing to do in a launch sits it out (NaN scalar, see the header).  The
calls that happen once per run of region steps (partition, gather of X^E, merge) are made per
request on its slice of the batch.

When the requests of a tick differ in time the model callbacks receive lists:
    model.full(x, [t_b or None], [store_b])          None = request b is not at a full step
    model.region(x_e, [t_b or None], edit_idx, n_edit)
and must return a value for every batch entry (entries with None are ignored).
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
    steps: list = field(default_factory=list)        # request 0: (k, kind, 'full' | 'compute' | 'reuse', scale)
    per_request: list = field(default_factory=list)  # the same list for every request
    model_full_calls: int = 0
    model_region_calls: int = 0
    launches: int = 0


@dataclass
class _RequestState:
    partitioned: bool = False
    in_run: bool = False
    t_run: float = 0.0
    product: float = 1.0
    have_cache: bool = False


_NAN = float("nan")


class RegionELoop:
    """Buffers and call sequence of one edit (a batch of B independent requests; same schedule,
    optionally shifted against each other by ``offsets``)."""

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

    def run(self, x, ref, model, stream=None, offsets=None):
        """Runs all steps on ``x`` [B, N, C] bf16 (updated in place); returns (x, trace).

        ``offsets`` [B]: request b takes step k at tick offsets[b] + k (default: all zero)."""
        cfg, b, st = self.cfg, binding, self.dev_status
        ts, T, B = cfg.timesteps, len(cfg.kinds), self.B
        offsets = [0] * B if offsets is None else [int(o) for o in offsets]
        if len(offsets) != B or min(offsets) < 0:
            raise binding.RegionEError("offsets must hold one non-negative tick per request")
        uniform = len(set(offsets)) == 1
        tr = LoopTrace(per_request=[[] for _ in range(B)])
        state = [_RequestState() for _ in range(B)]
        sl = lambda t_, r: t_[r:r + 1]                     # request r's slice of a batch tensor

        def merge_request(r, k, t_to):
            # end of a run of region steps: edited tokens from X^E, unedited tokens by one step of
            # the last full velocity over the whole run
            s_ = state[r]
            self._emit("merge_in", k, r=r, x=sl(self.x_run_start, r), v=sl(self.v_last_full, r),
                       x_e=sl(self.x_e, r), slot=sl(self.slot, r), dt_unedited=s_.t_run - t_to)
            b.merge(sl(self.x_run_start, r), sl(self.v_last_full, r), sl(self.x_e, r), sl(self.slot, r),
                    s_.t_run - t_to, sl(x, r), dev_status=st, stream=stream)
            self._emit("merge_out", k, r=r, x=sl(x, r))
            tr.launches += 1
            s_.in_run = False

        for tick in range(T + max(offsets)):
            ks = [tick - o if 0 <= tick - o < T else None for o in offsets]     # step of each request
            full = [r for r in range(B) if ks[r] is not None and cfg.kinds[ks[r]] == "F"]
            region = [r for r in range(B) if ks[r] is not None and cfg.kinds[ks[r]] == "R"]
            t_cur = [float(ts[k]) if k is not None else None for k in ks]
            dt = [float(ts[k]) - float(ts[k + 1]) if k is not None else None for k in ks]
            k0 = ks[0] if uniform else tick

            # ---- full steps ----
            if full:
                for r in full:
                    if state[r].in_run:
                        merge_request(r, ks[r], t_cur[r])
                store = [ks[r] is not None and (state[r].partitioned or ks[r] + 1 == cfg.partition_after)
                         for r in range(B)]
                if uniform:
                    v = model.full(x, t_cur[0], store[0])
                else:
                    v = model.full(x, [t_cur[r] if r in full else None for r in range(B)], store)
                tr.model_full_calls += 1
                if len(full) == B:
                    self._copy(self.v_last_full, v, stream)
                else:
                    for r in full:
                        self._copy(sl(self.v_last_full, r), sl(v, r), stream)
                dts = [dt[r] if r in full else _NAN for r in range(B)]
                self._emit("euler_in", k0, x=x, v=v, dt=dts, active=full)
                b.velocity_decay(v, 1.0, dts, x, self.n_all, dev_status=st, stream=stream)
                self._emit("euler_out", k0, x=x, active=full)
                tr.launches += 1
                part = [r for r in full if ks[r] + 1 == cfg.partition_after]
                if part:
                    t_part = [float(ts[ks[r] + 1]) if r in part else _NAN for r in range(B)]
                    self._emit("partition_in", k0, x=x, v=v, ref=ref, t=t_part, active=part)
                    b.partition(x, v, ref, t_part, cfg.metric, cfg.threshold, self.mask, self.edit_idx,
                                self.keep_idx, self.slot, self.n_edit, dev_status=st, stream=stream)
                    self._emit("partition_out", k0, mask=self.mask, edit_idx=self.edit_idx, slot=self.slot,
                               n_edit=self.n_edit, active=part)
                    tr.launches += 1
                    for r in part:
                        state[r].partitioned = True
                for r in full:
                    tr.per_request[r].append((ks[r], "F", "full", 1.0))

            # ---- region steps ----
            if region:
                reuse, compute = [], []
                for r in region:
                    s_ = state[r]
                    if not s_.partitioned:
                        raise binding.RegionEError("a region step was scheduled before the partition")
                    if not s_.in_run:
                        self._copy(sl(self.x_run_start, r), sl(x, r), stream)
                        b.gather(sl(x, r), sl(self.edit_idx, r), sl(self.n_edit, r), sl(self.x_e, r),
                                 dev_status=st, stream=stream)
                        tr.launches += 1
                        s_.in_run, s_.t_run = True, t_cur[r]
                        s_.product, s_.have_cache = 1.0, False
                    again = False
                    if s_.have_cache:
                        k = ks[r]
                        s_.product, again = b.avd_step(s_.product, float(ts[k - 1]) - t_cur[r],
                                                       float(cfg.gammas[k]), cfg.delta)
                    (reuse if again else compute).append(r)
                if reuse:
                    scale = [state[r].product if r in reuse else _NAN for r in range(B)]
                    dts = [dt[r] if r in reuse else _NAN for r in range(B)]
                    self._emit("decay_in", k0, v=self.v_cache, x_e=self.x_e, scale=scale, dt=dts,
                               n_edit=self.n_edit, active=reuse)
                    b.velocity_decay(self.v_cache, scale, dts, self.x_e, self.n_edit, dev_status=st,
                                     stream=stream)
                    self._emit("decay_out", k0, x_e=self.x_e, active=reuse)
                    tr.launches += 1
                    for r in reuse:
                        tr.per_request[r].append((ks[r], "R", "reuse", state[r].product))
                if compute:
                    if uniform:
                        v_e = model.region(self.x_e, t_cur[0], self.edit_idx, self.n_edit)
                    else:
                        v_e = model.region(self.x_e, [t_cur[r] if r in compute else None for r in range(B)],
                                           self.edit_idx, self.n_edit)
                    tr.model_region_calls += 1
                    scale = [1.0 if r in compute else _NAN for r in range(B)]
                    dts = [dt[r] if r in compute else _NAN for r in range(B)]
                    self._emit("decay_in", k0, v=v_e, x_e=self.x_e, scale=scale, dt=dts, n_edit=self.n_edit,
                               active=compute)
                    b.velocity_decay(v_e, scale, dts, self.x_e, self.n_edit, v_cache_out=self.v_cache,
                                     dev_status=st, stream=stream)
                    self._emit("decay_out", k0, x_e=self.x_e, active=compute)
                    tr.launches += 1
                    for r in compute:
                        state[r].product, state[r].have_cache = 1.0, True
                        tr.per_request[r].append((ks[r], "R", "compute", 1.0))

            # a request whose last step was a region step ends with the merge
            for r in range(B):
                if ks[r] == T - 1 and state[r].in_run:
                    merge_request(r, T, float(ts[T]))
        tr.steps = tr.per_request[0]
        return x, tr
