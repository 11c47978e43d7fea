"""GPU parity of the fused producer of fresh Q / K / V rows (gather + per-head RMS normalisation + rotary
embedding) against the fp64 oracle, and of the region attention fed by it."""
import numpy as np
import pytest

from gpu_util import assert_close, dev_bf16, dev_i32, host_f64
from oracle import regione_oracle as orc
from paper_2510_25590_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _tables(n_pos, D, seed):
    """cos / sin of seeded angles: textbook frequencies times the position, plus a per-position offset so
    that no two positions share a row of the table."""
    rng = np.random.default_rng(seed)
    inv = 10000.0 ** (-np.arange(D // 2, dtype=np.float64) * 2.0 / D)
    th = np.arange(n_pos, dtype=np.float64)[:, None] * inv[None, :] + rng.uniform(0, 0.5, (n_pos, 1))
    return np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)


def _run(q, k, v, idx, n, wq, wk, eps, cos, sin, layout, src_compact=False):
    import torch
    B, _, H, D = q.shape
    cap = idx.shape[1]
    outs = [torch.full((B, cap, H, D), -3.0, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.fresh_qkv(dev_bf16(q), dev_bf16(k), dev_bf16(v), dev_i32(idx), dev_i32(n),
                      None if wq is None else dev_bf16(wq), None if wk is None else dev_bf16(wk), eps,
                      torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda(), layout, *outs,
                      src_compact=src_compact, dev_status=st)
    torch.cuda.synchronize()
    return outs, int(st[0])


@pytest.mark.parametrize("layout", [binding.ROPE_INTERLEAVED, binding.ROPE_HALF])
@pytest.mark.parametrize("D,H,weights", [(128, 24, True), (64, 3, True), (128, 5, False), (64, 4, False)])
def test_fresh_rows_match_the_oracle(D, H, weights, layout):
    rng = np.random.default_rng(D + H + layout)
    B, N, cap = 2, 300, 150
    q, k, v = (synth.bf16_round((rng.standard_normal((B, N, H, D), dtype=np.float32) * np.float32(s)))
               for s in (0.09, 2.5, 1.0))
    k[0, 17, 0] = 0.0                                        # an all-zero row and head stays zero (eps keeps it finite)
    wq = synth.bf16_round(1.0 + 0.2 * rng.standard_normal(D, dtype=np.float32)) if weights else None
    wk = synth.bf16_round(1.0 + 0.2 * rng.standard_normal(D, dtype=np.float32)) if weights else None
    idx = np.stack([rng.permutation(N)[:cap] for _ in range(B)]).astype(np.int32)     # any order, not ascending
    idx[0, 0] = 17; idx[0, 1] = 0; idx[1, 0] = N - 1
    n = np.array([cap, 37], np.int32)
    cos, sin = _tables(N, D, 3)
    (gq, gk, gv), status = _run(q, k, v, idx, n, wq, wk, 1e-6, cos, sin, layout)
    assert status == 0
    wantq, wantk, wantv = orc.fresh_qkv(q, k, v, idx, n, wq, wk, np.float32(1e-6), cos, sin, layout)
    for b in range(B):
        m = n[b]
        for got, want in ((gq, wantq), (gk, wantk)):
            g, w = host_f64(got)[b, :m], want[b, :m]
            # fp32 arithmetic and one rounding to bf16 (half a unit in the 8th significant bit)
            assert np.all(np.abs(g - w) <= np.abs(w) * 2.0 ** -8 * 1.02 + 1e-6)
            assert_close(g, w, "normalised and rotated rows")
            assert np.all(host_f64(got)[b, m:] == -3.0)                               # tail untouched
        assert np.array_equal(host_f64(gv)[b, :m], wantv[b, :m])                      # V: a copy, bit-exact
        assert np.all(host_f64(gv)[b, m:] == -3.0)
    assert np.all(host_f64(gk)[0, 0, 0] == 0.0)


@pytest.mark.parametrize("layout", [binding.ROPE_INTERLEAVED, binding.ROPE_HALF])
def test_rows_that_are_already_gathered_take_their_position_from_the_index(layout):
    """A region step projects Q, K, V for the recomputed rows only: the sources hold row j at j, the index
    list names the position whose angles rotate it.  Same result as gathering from the whole sequence."""
    rng = np.random.default_rng(11 + layout)
    B, N, cap, H, D = 2, 200, 60, 3, 128
    q, k, v = (synth.bf16_round(rng.standard_normal((B, N, H, D), dtype=np.float32)) for _ in range(3))
    idx = np.stack([np.sort(rng.permutation(N)[:cap]) for _ in range(B)]).astype(np.int32)
    n = np.array([cap, 41], np.int32)
    cos, sin = _tables(N, D, 4)
    take = lambda a: np.stack([a[b, idx[b]] for b in range(B)])
    (cq, ck, cv), st1 = _run(take(q), take(k), take(v), idx, n, None, None, 1e-6, cos, sin, layout, src_compact=True)
    (gq, gk, gv), st2 = _run(q, k, v, idx, n, None, None, 1e-6, cos, sin, layout)
    assert st1 == 0 and st2 == 0
    import torch
    for a, b_ in ((cq, gq), (ck, gk), (cv, gv)):
        assert torch.equal(a.view(torch.int16), b_.view(torch.int16))           # bit-identical to the gathering form
    want = orc.fresh_qkv(take(q), take(k), take(v), idx, n, None, None, np.float32(1e-6), cos, sin, layout, src_compact=True)
    for b in range(B):
        assert_close(host_f64(cq)[b, :n[b]], want[0][b, :n[b]], "compact source")


def test_attention_over_produced_rows_matches_the_oracle_chain():
    """The producer feeding the region attention: fresh rows normalised and rotated at their positions,
    the cache holding the other rows normalised and rotated at theirs (as a full step leaves them),
    against the oracle's producer followed by the oracle's attention."""
    import torch
    wl = synth.scaled_workload(synth.WORKLOADS[2], grid=(24, 24), n_text=70, heads=4)
    mask = synth.make_latents(wl)["mask"][0]
    qkv = synth.make_qkv_full(wl, std=1.0)
    rows = orc.region_rows(mask, wl.n_text, wl.n_ref, "edited_queries")
    nq, nc, D = len(rows["query"]), len(rows["cache"]), wl.head_dim
    cos, sin = _tables(wl.n_full, D, 5)
    rng = np.random.default_rng(9)
    wq = synth.bf16_round(1.0 + 0.1 * rng.standard_normal(D, dtype=np.float32))
    wk = synth.bf16_round(1.0 + 0.1 * rng.standard_normal(D, dtype=np.float32))
    layout = binding.ROPE_INTERLEAVED
    both = np.zeros((1, max(nq, nc)), np.int32)
    idx_q = both.copy(); idx_q[0, :nq] = rows["query"]
    idx_c = both.copy(); idx_c[0, :nc] = rows["cache"]
    (fq, fk, fv), s1 = _run(qkv["q"], qkv["k"], qkv["v"], idx_q, np.array([nq], np.int32), wq, wk, 1e-6, cos, sin, layout)
    (_, ck, cv), s2 = _run(qkv["q"], qkv["k"], qkv["v"], idx_c, np.array([nc], np.int32), wq, wk, 1e-6, cos, sin, layout)
    assert s1 == 0 and s2 == 0
    out = torch.full(fq.shape, -3.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    cap = fq.shape[1]
    ws = torch.empty(max(binding.region_attention_workspace(1, cap, cap, cap, wl.heads, D), 256), dtype=torch.uint8, device="cuda")
    binding.region_attention(fq, fk, fv, ck, cv, dev_i32([nq]), dev_i32([nq]), dev_i32([nc]), out, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    # the oracle chain on the bf16 values the producer wrote (its own rounding is checked above)
    want = orc.region_attention(host_f64(fq), host_f64(fk), host_f64(fv), host_f64(ck), host_f64(cv), [nq], [nq], [nc])
    assert_close(host_f64(out)[0, :nq], want[0, :nq], "attention over produced rows")
    # and end to end from the oracle's own producer, within the looser bound two bf16 roundings of Q and K allow
    oq, ok_, ov = orc.fresh_qkv(qkv["q"], qkv["k"], qkv["v"], idx_q, [nq], wq, wk, np.float32(1e-6), cos, sin, layout)
    _, oc, ocv = orc.fresh_qkv(qkv["q"], qkv["k"], qkv["v"], idx_c, [nc], wq, wk, np.float32(1e-6), cos, sin, layout)
    want2 = orc.region_attention(oq, ok_, ov, oc, ocv, [nq], [nq], [nc])
    d = host_f64(out)[0, :nq] - want2[0, :nq]
    rel = np.sqrt(np.mean(d * d)) / np.sqrt(np.mean(want2[0, :nq] ** 2))
    print(f"end-to-end rel-RMS against the unrounded producer: {rel:.3e}")
    assert rel < 3e-2


def test_bad_arguments_and_indices():
    import torch
    rng = np.random.default_rng(2)
    q, k, v = (synth.bf16_round(rng.standard_normal((1, 20, 2, 64), dtype=np.float32)) for _ in range(3))
    cos, sin = _tables(20, 64, 1)
    idx = np.array([[3, 25, 5]], np.int32)
    (gq, _, gv), status = _run(q, k, v, idx, np.array([3], np.int32), None, None, 1e-6, cos, sin, binding.ROPE_HALF)
    assert status == binding.DEV_BOUNDS
    assert np.all(host_f64(gq)[0, 1] == -3.0) and np.all(host_f64(gv)[0, 2] == v[0, 5])
    with pytest.raises(binding.RegionEError):
        _run(q, k, v, idx, np.array([3], np.int32), None, None, 1e-6, cos, sin, 7)
