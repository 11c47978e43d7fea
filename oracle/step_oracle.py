"""The whole region-aware step for one attention layer, as a chain of oracle calls (fp64).

TEST INFRASTRUCTURE ONLY (same rules as regione_oracle).  Mirrors Algorithm 1 for one layer:
partition, gather, cache store, region attention, scatter, velocity decay + Euler, merge.
``wl`` is only read for its shape fields (batch, n_text, n_ref, metric, threshold); nothing of the
product package is imported.

Pins (marker "not gpu", tests/test_oracle_step.py): a zero-edit mask gives x - dt_U * v on every token
and an all-zero attention output; a full mask under the paper's membership with no reference tokens
reduces the attention rows to a library softmax attention; the counts of the tiny configuration;
edited tokens of the merged latent equal X^E after the Euler step and unedited ones lie on the
straight line; the cache holds exactly the rows the membership rule names.
"""
from __future__ import annotations

import numpy as np

from oracle import regione_oracle as orc


def region_step(wl, lat, qkv, t, scale, dt, dt_unedited, membership="edited_queries", heads=None):
    """Returns a dict of every intermediate the GPU step also produces.

    ``heads`` restricts the attention to a subset of heads (used to bound the CPU-baseline
    timing); all other stages always run at full size.
    """
    metric = orc.COSINE if wl.metric == "cosine" else orc.L2
    B = wl.batch
    p = orc.partition(lat["x_t"], lat["v"], lat["ref"], t, metric, wl.threshold)
    rows = [orc.region_rows(p["mask"][b], wl.n_text, wl.n_ref, membership) for b in range(B)]
    nq = np.array([len(r["query"]) for r in rows], np.int32)
    nc = np.array([len(r["cache"]) for r in rows], np.int32)
    q_cap, c_cap = max(1, int(nq.max())), max(1, int(nc.max()))
    qrows = np.zeros((B, q_cap), np.int32)
    crows = np.zeros((B, c_cap), np.int32)
    for b in range(B):
        qrows[b, :nq[b]] = rows[b]["query"]
        crows[b, :nc[b]] = rows[b]["cache"]
    x_e = orc.gather(lat["x_t"], p["edit_idx"], p["n_edit"])
    v_e = orc.gather(lat["v"], p["edit_idx"], p["n_edit"])
    hs = slice(None) if heads is None else slice(0, heads)
    qf, kf, vf = qkv["q"][:, :, hs], qkv["k"][:, :, hs], qkv["v"][:, :, hs]
    k_cache, v_cache = orc.rikv_store(kf, vf, crows, nc)
    q_e = orc.gather(qf, qrows, nq)
    k_fresh = orc.gather(kf, qrows, nq)
    v_fresh = orc.gather(vf, qrows, nq)
    o_e = orc.region_attention(q_e, k_fresh, v_fresh, k_cache, v_cache, nq, nq, nc)
    o_full = orc.scatter(np.zeros(qf.shape), o_e, qrows, nq)
    x_e_new, _ = orc.velocity_decay(v_e, scale, dt, x_e, p["n_edit"])
    x_out = orc.merge(lat["x_t"], lat["v"], x_e_new, p["slot"], dt_unedited)
    return dict(partition=p, query_rows=qrows, cache_rows=crows, n_q=nq, n_cache=nc, x_e=x_e_new,
                v_e=v_e, k_cache=k_cache, v_cache=v_cache, o_e=o_e, o_full=o_full, x_out=x_out)
