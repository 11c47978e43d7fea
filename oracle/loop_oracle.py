"""fp64 statement of the whole sampler loop (Algorithm 1) on top of regione_oracle.

TEST INFRASTRUCTURE ONLY (same rules as regione_oracle): shares no code with the CUDA path.

The loop of Algorithm 1 in the reading the design notes list: the schedule is a string of step
kinds ('F' full, 'R' region); the Adaptive Region Partition runs once, after ``partition_after``
steps, on the post-update latent and the latest full velocity; every run of region steps starts by
taking X^E = X[E_index], keeps the unedited tokens frozen, and ends (at the next full step, or at
the end) with the merge: edited tokens from X^E, unedited tokens one-step predicted over the whole
run with the last full velocity.  Inside a run the AVDCache criterion decides between calling the
model on the edited tokens and reusing the cached velocity times the accumulated decay; the Euler
update applies in both cases.  The first region step of a run always computes.
"""
from __future__ import annotations

import numpy as np

from oracle import regione_oracle as orc


def run_loop(x, ref, model, kinds, partition_after, timesteps, gammas, delta, metric, threshold):
    """x, ref: [B, N, C] float64.  model.full(x, t) -> v [B, N, C]; model.region(x_e, t, edit_idx,
    n_edit) -> v_e [B, cap, C].  Returns dict(x, partition, log) with log = list of
    (k, kind, what, scale)."""
    x = np.array(x, dtype=np.float64, copy=True)
    part = None
    log = []
    in_run = False
    for k, kind in enumerate(kinds):
        t_cur, t_next = float(timesteps[k]), float(timesteps[k + 1])
        dt = t_cur - t_next
        if kind == "F":
            if in_run:
                x = orc.merge(x_start, v_last, x_e, part["slot"], t_run - t_cur)
                in_run = False
            v = np.asarray(model.full(x, t_cur), dtype=np.float64)
            v_last = v
            x = x - dt * v                      # Euler sampler equation
            log.append((k, kind, "full", 1.0))
            if k + 1 == partition_after:
                part = orc.partition(x, v, ref, t_next, metric, threshold)
            continue
        if not in_run:
            x_start = x.copy()
            x_e = orc.gather(x, part["edit_idx"], part["n_edit"])
            in_run, t_run = True, t_cur
            product, cache = 1.0, None
        reuse = False
        if cache is not None:
            product, reuse = orc.avd_step(product, float(timesteps[k - 1]) - t_cur, float(gammas[k]), delta)
        if reuse:
            x_e, _ = orc.velocity_decay(cache, product, dt, x_e, part["n_edit"])
            log.append((k, kind, "reuse", product))
        else:
            v_e = np.asarray(model.region(x_e, t_cur, part["edit_idx"], part["n_edit"]), dtype=np.float64)
            x_e, _ = orc.velocity_decay(v_e, 1.0, dt, x_e, part["n_edit"])
            cache, product = v_e, 1.0
            log.append((k, kind, "compute", 1.0))
    if in_run:
        x = orc.merge(x_start, v_last, x_e, part["slot"], t_run - float(timesteps[len(kinds)]))
    return dict(x=x, partition=part, log=log)


class StraightLineModel:
    """Velocity of the rectified flow toward a fixed target X0*: v(x, t) = (x - X0*) / t, the exact
    velocity X1 - X0 of the straight path through x at time t (Preliminary section)."""

    def __init__(self, target):
        self.target = np.asarray(target, dtype=np.float64)

    def full(self, x, t):
        return (np.asarray(x, np.float64) - self.target) / t

    def region(self, x_e, t, edit_idx, n_edit):
        x_e = np.asarray(x_e, np.float64)
        out = np.zeros_like(x_e)
        for b in range(x_e.shape[0]):
            ne = int(n_edit[b])
            out[b, :ne] = (x_e[b, :ne] - self.target[b, edit_idx[b, :ne]]) / t
        return out
