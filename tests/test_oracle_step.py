"""Pins for the oracle's row-membership rule and for the chained step oracle (CPU only).

None of these re-evaluates the oracle's own formulas: they compare against closed forms, against
a library softmax attention, against counts the configurations fix, and against independently
built index sets.
"""
import numpy as np
import pytest

from oracle import regione_oracle as orc
from oracle import step_oracle
from paper_2510_25590_b200 import synth


def _small(cfg, **kw):
    return synth.scaled_workload(synth.WORKLOADS[cfg], **kw)


# ---- region_rows: which joint-sequence rows are recomputed, which are cached -----------------


@pytest.mark.parametrize("membership", ["edited_queries", "paper"])
def test_row_lists_partition_the_joint_sequence(membership):
    rng = np.random.default_rng(3)
    n_text, n_img, n_ref = 7, 50, 13
    mask = (rng.random(n_img) < 0.3).astype(np.uint8)
    r = orc.region_rows(mask, n_text, n_ref, membership)
    both = np.concatenate([r["query"], r["cache"]])
    assert np.array_equal(np.sort(both), np.arange(n_text + n_img + n_ref))       # every row exactly once
    assert np.all(np.diff(r["query"]) > 0) and np.all(np.diff(r["cache"]) > 0)    # ascending
    assert np.array_equal(r["fresh"], r["query"])
    # built independently with set arithmetic on the joint positions
    edited = set((n_text + np.flatnonzero(mask)).tolist())
    text = set(range(n_text))
    want_q = edited | text if membership == "paper" else edited
    assert set(r["query"].tolist()) == want_q
    # reference rows are never recomputed; text rows only under the attention equation as printed
    assert set(range(n_text + n_img, n_text + n_img + n_ref)) <= set(r["cache"].tolist())
    assert (text <= set(r["query"].tolist())) == (membership == "paper" or n_text == 0)


def test_row_counts_of_the_tiny_configuration():
    wl = synth.WORKLOADS[1]
    mask = synth.make_latents(wl)["mask"][0]
    r = orc.region_rows(mask, wl.n_text, wl.n_ref, "edited_queries")
    assert len(r["query"]) == 256 and len(r["cache"]) == 64 + 1024 + 768 == 1856
    r = orc.region_rows(mask, wl.n_text, wl.n_ref, "paper")
    assert len(r["query"]) == 64 + 256 and len(r["cache"]) == 768 + 1024


def test_row_lists_of_the_all_and_nothing_masks():
    r = orc.region_rows(np.zeros(9, np.uint8), 2, 4, "edited_queries")
    assert len(r["query"]) == 0 and np.array_equal(r["cache"], np.arange(15))
    r = orc.region_rows(np.ones(9, np.uint8), 2, 4, "paper")
    assert np.array_equal(r["query"], np.arange(11)) and np.array_equal(r["cache"], np.arange(11, 15))


# ---- region_step: the chain -------------------------------------------------------------------


def _inputs(wl, ratio=None):
    return synth.make_latents(wl, ratio), synth.make_qkv_full(wl)


def test_zero_edit_mask_gives_the_one_step_prediction_everywhere_and_no_attention_rows():
    wl = _small(2, grid=(8, 8), n_text=5, heads=2)
    lat, qkv = _inputs(wl, ratio=0.0)
    dt_u = 5.0 / 28.0
    res = step_oracle.region_step(wl, lat, qkv, lat["t"], 0.9, 1.0 / 28.0, dt_u)
    assert int(res["partition"]["n_edit"][0]) == 0 and int(res["n_q"][0]) == 0
    # closed form, written with the inputs only (one-step estimation equation on every token)
    want = lat["x_t"].astype(np.float64) - dt_u * lat["v"].astype(np.float64)
    assert np.array_equal(res["x_out"], want)
    assert np.all(res["o_full"] == 0.0)
    assert int(res["n_cache"][0]) == wl.n_full


def test_full_mask_with_paper_membership_and_no_reference_is_library_attention():
    import torch
    wl = _small(3, grid=(6, 6), n_text=4, heads=2, n_ref=0)
    lat, qkv = _inputs(wl, ratio=1.0)
    res = step_oracle.region_step(wl, lat, qkv, lat["t"], 1.0, 1.0 / 28.0, 0.1, membership="paper")
    assert int(res["n_q"][0]) == wl.n_full and int(res["n_cache"][0]) == 0
    tq, tk, tv = (torch.from_numpy(qkv[k].astype(np.float64)).permute(0, 2, 1, 3) for k in ("q", "k", "v"))
    sdpa = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    assert np.allclose(res["o_full"], sdpa, rtol=1e-10, atol=1e-12)
    assert np.allclose(res["o_e"][0], sdpa[0], rtol=1e-10, atol=1e-12)


def test_full_mask_edited_queries_attend_over_every_row_of_the_sequence():
    # permutation / split invariance at the level of the chain: with every image token edited the
    # keys are [edited | text, reference], i.e. the whole joint sequence, so each image row equals
    # the library attention of that row over all keys
    import torch
    wl = _small(3, grid=(5, 5), n_text=3, heads=2, n_ref=6)
    lat, qkv = _inputs(wl, ratio=1.0)
    res = step_oracle.region_step(wl, lat, qkv, lat["t"], 1.0, 1.0 / 28.0, 0.1)
    tq, tk, tv = (torch.from_numpy(qkv[k].astype(np.float64)).permute(0, 2, 1, 3) for k in ("q", "k", "v"))
    sdpa = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    img = slice(wl.n_text, wl.n_text + wl.n_img)
    assert np.allclose(res["o_full"][:, img], sdpa[:, img], rtol=1e-10, atol=1e-12)
    assert np.all(res["o_full"][:, :wl.n_text] == 0) and np.all(res["o_full"][:, wl.n_text + wl.n_img:] == 0)


def test_counts_and_cache_contents_of_the_tiny_configuration():
    wl = synth.WORKLOADS[1]
    lat, qkv = _inputs(wl)
    res = step_oracle.region_step(wl, lat, qkv, lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0, heads=1)
    assert int(res["n_q"][0]) == 256 and int(res["n_cache"][0]) == 1856
    assert np.array_equal(res["partition"]["mask"], lat["mask"])                 # planted mask recovered
    # the cache holds text, unedited image and reference rows of the full K / V, in sequence order
    planted = lat["mask"][0].astype(bool)
    rows = np.concatenate([np.arange(wl.n_text), wl.n_text + np.flatnonzero(~planted),
                           wl.n_text + wl.n_img + np.arange(wl.n_ref)])
    assert np.array_equal(res["k_cache"][0, :1856], qkv["k"][0, rows, :1].astype(np.float64))
    assert np.array_equal(res["v_cache"][0, :1856], qkv["v"][0, rows, :1].astype(np.float64))


def test_merged_latent_takes_edited_tokens_from_the_euler_step_and_unedited_from_the_straight_line():
    wl = _small(2, grid=(12, 12), n_text=6, heads=1)
    lat, qkv = _inputs(wl)
    t, scale, dt, dt_u = lat["t"], 0.75, 2.0 / 28.0, 6.0 / 28.0
    res = step_oracle.region_step(wl, lat, qkv, t, scale, dt, dt_u)
    x, v = lat["x_t"].astype(np.float64), lat["v"].astype(np.float64)
    planted = lat["mask"][0].astype(bool)
    assert planted.sum() > 0 and (~planted).sum() > 0
    # edited tokens: Euler step with the decayed velocity (scale and dt both matter: a swapped or
    # dropped factor changes these values)
    assert np.allclose(res["x_out"][0, planted], x[0, planted] - dt * scale * v[0, planted], rtol=0, atol=1e-15)
    # unedited tokens: one step of length dt_u, not dt, and no decay factor
    assert np.allclose(res["x_out"][0, ~planted], x[0, ~planted] - dt_u * v[0, ~planted], rtol=0, atol=1e-15)
    # and they land on the straight line of the rectified flow: x(t - dt_u) = x0 + (t - dt_u) (x1 - x0)
    # where the generator's unedited tokens have v = x1 - x0 exactly up to bf16 rounding of its outputs
    x0_hat = x[0, ~planted] - t * v[0, ~planted]
    on_line = x0_hat + (t - dt_u) * v[0, ~planted]
    assert np.allclose(res["x_out"][0, ~planted], on_line, rtol=0, atol=1e-12)
    # X^E rows are in ascending token order
    ne = int(res["partition"]["n_edit"][0])
    assert np.allclose(res["x_e"][0, :ne], res["x_out"][0, planted], rtol=0, atol=0)


def test_attention_rows_land_at_their_joint_sequence_positions():
    wl = _small(5, grid=(8, 8), n_text=4, heads=2, batch=2)
    lat, qkv = _inputs(wl)
    res = step_oracle.region_step(wl, lat, qkv, lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0)
    for b in range(wl.batch):
        planted = lat["mask"][b].astype(bool)
        rows = wl.n_text + np.flatnonzero(planted)
        nq = int(res["n_q"][b])
        assert nq == len(rows) and np.array_equal(res["query_rows"][b, :nq], rows)
        assert np.array_equal(res["o_full"][b, rows], res["o_e"][b, :nq])
        others = np.setdiff1d(np.arange(wl.n_full), rows)
        assert np.all(res["o_full"][b, others] == 0.0)
        # one sampled row against a direct evaluation over the whole sequence (keys in any order)
        r = rows[len(rows) // 2]
        for h in range(wl.heads):
            lg = qkv["k"][b, :, h].astype(np.float64) @ qkv["q"][b, r, h].astype(np.float64) / np.sqrt(wl.head_dim)
            p = np.exp(lg - lg.max()); p /= p.sum()
            assert np.allclose(res["o_full"][b, r, h], p @ qkv["v"][b, :, h].astype(np.float64), rtol=1e-9, atol=1e-12)
