"""ctypes binding over the C ABI of ``libregione.so`` (see ``include/regione.h``).

Argument marshalling only: every function takes torch CUDA tensors (used purely
as device buffers), checks dtype / contiguity, and forwards raw pointers and
sizes to the entry point of the same name.  There is no fallback of any kind:
if the shared library is missing or a call fails, a ``RegionEError`` is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_double, c_float, c_int, c_int64, c_longlong, c_size_t, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libregione.so")

OK, INVALID_ARG, UNSUPPORTED, CUDA_ERROR, WORKSPACE_TOO_SMALL = 0, 1, 2, 3, 4
DEV_OK, DEV_TIMEOUT, DEV_BOUNDS = 0, 5, 6
METRIC_COSINE, METRIC_L2 = 0, 1
ROWS_EDITED_QUERIES, ROWS_PAPER = 0, 1
ROPE_INTERLEAVED, ROPE_HALF = 0, 1

# every symbol include/regione.h declares: name -> (restype, argtypes)
_P = c_void_p
SIGNATURES = {
    "regione_version": (c_int, []),
    "regione_status_string": (c_char_p, [c_int]),
    "regione_partition": (c_int, [_P, _P, _P, c_int, c_int, c_int, _P, c_int, c_float,
                                  _P, _P, _P, _P, _P, _P, _P, _P]),
    "regione_partition_rows": (c_int, [_P, _P, _P, c_int, c_int, c_int, _P, c_int, c_float,
                                       _P, _P, _P, _P, _P, _P, c_int, c_int, c_int,
                                       _P, _P, c_int, _P, _P, c_int, _P, _P]),
    "regione_mask_open_close": (c_int, [_P, c_int, c_int, c_int, _P, _P, _P, _P, _P, _P, _P]),
    "regione_region_rows": (c_int, [_P, _P, _P, c_int, c_int, c_int, c_int, c_int,
                                    _P, _P, c_int, _P, _P, c_int, _P, _P]),
    "regione_gather": (c_int, [_P, _P, _P, c_int, c_int64, c_int64, c_int64, c_int64, _P, _P, _P]),
    "regione_gather_multi": (c_int, [_P, _P, c_int, _P, _P, c_int, c_int64, c_int64, c_int64, c_int64, _P, _P]),
    "regione_scatter": (c_int, [_P, _P, _P, c_int, c_int64, c_int64, c_int64, c_int64, _P, _P, _P]),
    "regione_rikv_store": (c_int, [_P, _P, _P, _P, c_int, c_int, c_int, c_int, c_int, _P, _P, _P, _P]),
    "regione_rikv_store_e4m3": (c_int, [_P, _P, _P, _P, c_int, c_int, c_int, c_int, c_int, _P, _P, _P, _P, _P, _P]),
    "regione_rikv_load_e4m3": (c_int, [_P, _P, _P, _P, _P, c_int, c_int, c_int, c_int, _P, _P, _P, _P]),
    "regione_fresh_qkv": (c_int, [_P] * 5 + [c_int] * 6 + [_P, _P, c_float, _P, _P, c_int, _P, _P, _P, _P, _P]),
    "regione_region_attention_workspace": (c_size_t, [c_int] * 6),
    "regione_region_attention": (c_int, [_P] * 8 + [c_int] * 6 + [c_float, _P, _P, c_size_t, _P, _P]),
    "regione_region_attention_scatter": (c_int, [_P] * 8 + [c_int] * 6 + [c_float, _P, c_int, _P, _P, c_size_t, _P, _P]),
    "regione_full_attention_store_workspace": (c_size_t, [c_int] * 4),
    "regione_full_attention_store": (c_int, [_P] * 4 + [c_int] * 4 + [c_float, _P, _P, c_int, _P, _P, _P, _P,
                                             c_size_t, _P, _P]),
    "regione_region_attention_static": (c_int, [_P] * 8 + [c_int] * 6 + [c_float, _P, _P, _P]),
    "regione_avd_step": (c_int, [POINTER(c_double), c_double, c_double, c_double, POINTER(c_int)]),
    "regione_gamma_fit": (c_int, [_P, c_int, c_int, c_int64, _P, _P, _P, _P]),
    "regione_velocity_decay": (c_int, [_P, _P, _P, _P, _P, _P, c_int, c_int, c_int, _P, _P]),
    "regione_merge": (c_int, [_P, _P, _P, _P, _P, c_int, c_int, c_int, c_int, _P, _P, _P]),
    "regione_crosscheck_region_attention": (c_int, [_P] * 8 + [c_int] * 6 + [c_float, _P, _P, _P]),
    "regione_selftest_bounded_wait": (c_int, [c_longlong, _P, _P, _P]),
}


class RegionEError(RuntimeError):
    pass


_lib = None


def load(path: str | None = None) -> ctypes.CDLL:
    """Loads libregione.so (once) and declares every entry point.  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RegionEError(
            f"{p} not found: build it with `python -m paper_2510_25590_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(p)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    if path is None:
        _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().regione_status_string(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != OK:
        raise RegionEError(f"{what} failed: {status_string(code)} ({code})")


def _torch():
    import torch
    return torch


def _ptr(t, dtype=None, name="tensor"):
    if t is None:
        return None
    torch = _torch()
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise RegionEError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise RegionEError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise RegionEError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return c_void_p(t.data_ptr())


def _stream(stream=None):
    torch = _torch()
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _per_request(value, B, name):
    """A sampler scalar for the batch: one number (shared by every request) or B numbers (each
    request at its own sampler step) -> a host float array of length B."""
    try:
        vals = [float(value)] * B
    except (TypeError, ValueError):
        vals = [float(x) for x in value]
        if len(vals) != B:
            raise RegionEError(f"{name} must be one number or {B} numbers, got {len(vals)}")
    return (c_float * max(B, 1))(*vals)


def version() -> int:
    return load().regione_version()


def partition(x_t, v, ref, t, metric, threshold, mask, edit_idx, keep_idx, slot, n_edit,
              score=None, dev_status=None, stream=None):
    torch = _torch()
    B, N, C = x_t.shape
    bf = torch.bfloat16
    _check(load().regione_partition(
        _ptr(x_t, bf, "x_t"), _ptr(v, bf, "v"), _ptr(ref, bf, "ref"), B, N, C, _per_request(t, B, "t"),
        int(metric),
        float(threshold), _ptr(mask, torch.uint8, "mask"), _ptr(edit_idx, torch.int32, "edit_idx"),
        _ptr(keep_idx, torch.int32, "keep_idx"), _ptr(slot, torch.int32, "slot"),
        _ptr(n_edit, torch.int32, "n_edit"), _ptr(score, torch.float32, "score"),
        _ptr(dev_status, torch.int32, "dev_status"), _stream(stream)), "regione_partition")


def partition_rows(x_t, v, ref, t, metric, threshold, mask, edit_idx, keep_idx, slot, n_edit,
                   n_text, n_ref, membership, query_rows, n_query, cache_rows, n_cache,
                   score=None, dev_status=None, stream=None):
    """``partition`` and ``region_rows`` in one launch."""
    torch = _torch()
    B, N, C = x_t.shape
    bf, i32 = torch.bfloat16, torch.int32
    _check(load().regione_partition_rows(
        _ptr(x_t, bf, "x_t"), _ptr(v, bf, "v"), _ptr(ref, bf, "ref"), B, N, C, _per_request(t, B, "t"),
        int(metric),
        float(threshold), _ptr(mask, torch.uint8, "mask"), _ptr(edit_idx, i32, "edit_idx"),
        _ptr(keep_idx, i32, "keep_idx"), _ptr(slot, i32, "slot"), _ptr(n_edit, i32, "n_edit"),
        _ptr(score, torch.float32, "score"), int(n_text), int(n_ref), int(membership),
        _ptr(query_rows, i32), _ptr(n_query, i32), query_rows.shape[1],
        _ptr(cache_rows, i32), _ptr(n_cache, i32), cache_rows.shape[1],
        _ptr(dev_status, i32, "dev_status"), _stream(stream)), "regione_partition_rows")


def mask_open_close(mask_in, rows, cols, mask_out, edit_idx, keep_idx, slot, n_edit,
                    dev_status=None, stream=None):
    torch = _torch()
    B = mask_in.shape[0]
    _check(load().regione_mask_open_close(
        _ptr(mask_in, torch.uint8, "mask_in"), B, int(rows), int(cols),
        _ptr(mask_out, torch.uint8, "mask_out"), _ptr(edit_idx, torch.int32), _ptr(keep_idx, torch.int32),
        _ptr(slot, torch.int32), _ptr(n_edit, torch.int32), _ptr(dev_status, torch.int32),
        _stream(stream)), "regione_mask_open_close")


def region_rows(edit_idx, keep_idx, n_edit, n_text, n_ref, membership, query_rows, n_query,
                cache_rows, n_cache, dev_status=None, stream=None):
    torch = _torch()
    B, N = edit_idx.shape
    i32 = torch.int32
    _check(load().regione_region_rows(
        _ptr(edit_idx, i32), _ptr(keep_idx, i32), _ptr(n_edit, i32), B, N, int(n_text), int(n_ref),
        int(membership), _ptr(query_rows, i32), _ptr(n_query, i32), query_rows.shape[1],
        _ptr(cache_rows, i32), _ptr(n_cache, i32), cache_rows.shape[1], _ptr(dev_status, i32),
        _stream(stream)), "regione_region_rows")


def _row_bytes(t):
    rb = t.element_size()
    for d in t.shape[2:]:
        rb *= d
    return rb


def gather(src, idx, n, dst, dev_status=None, stream=None):
    """dst[b, j] = src[b, idx[b, j]], j < n[b].  src [B, rows, ...], dst [B, cap, ...]."""
    torch = _torch()
    B = src.shape[0]
    _check(load().regione_gather(
        _ptr(src, None, "src"), _ptr(idx, torch.int32, "idx"), _ptr(n, torch.int32, "n"), B,
        src.shape[1], idx.shape[1], dst.shape[1], _row_bytes(src), _ptr(dst, src.dtype, "dst"),
        _ptr(dev_status, torch.int32), _stream(stream)), "regione_gather")


def gather_multi(srcs, idx, n, dsts, dev_status=None, stream=None):
    """dsts[i][b, j] = srcs[i][b, idx[b, j]] for up to 4 same-shaped tensors, one launch."""
    torch = _torch()
    k = len(srcs)
    if k != len(dsts) or not 1 <= k <= 4:
        raise RegionEError("gather_multi takes 1 to 4 (src, dst) pairs")
    for s_, d_ in zip(srcs, dsts):
        if s_.shape != srcs[0].shape or d_.shape != dsts[0].shape or s_.dtype != d_.dtype:
            raise RegionEError("gather_multi: tensors must share shape and dtype")
    sp = (c_void_p * k)(*[_ptr(t, None, "src").value for t in srcs])
    dp = (c_void_p * k)(*[_ptr(t, None, "dst").value for t in dsts])
    _check(load().regione_gather_multi(
        sp, dp, k, _ptr(idx, torch.int32, "idx"), _ptr(n, torch.int32, "n"), srcs[0].shape[0],
        srcs[0].shape[1], idx.shape[1], dsts[0].shape[1], _row_bytes(srcs[0]),
        _ptr(dev_status, torch.int32), _stream(stream)), "regione_gather_multi")


def scatter(src, idx, n, dst, dev_status=None, stream=None):
    """dst[b, idx[b, j]] = src[b, j], j < n[b].  src [B, cap, ...], dst [B, rows, ...]."""
    torch = _torch()
    B = src.shape[0]
    _check(load().regione_scatter(
        _ptr(src, None, "src"), _ptr(idx, torch.int32, "idx"), _ptr(n, torch.int32, "n"), B,
        src.shape[1], idx.shape[1], dst.shape[1], _row_bytes(src), _ptr(dst, src.dtype, "dst"),
        _ptr(dev_status, torch.int32), _stream(stream)), "regione_scatter")


def rikv_store(k_full, v_full, keep_rows, n_keep, k_cache, v_cache, dev_status=None, stream=None):
    torch = _torch()
    bf = torch.bfloat16
    B, n_full, H, D = k_full.shape
    _check(load().regione_rikv_store(
        _ptr(k_full, bf, "k_full"), _ptr(v_full, bf, "v_full"), _ptr(keep_rows, torch.int32),
        _ptr(n_keep, torch.int32), B, n_full, k_cache.shape[1], H, D, _ptr(k_cache, bf, "k_cache"),
        _ptr(v_cache, bf, "v_cache"), _ptr(dev_status, torch.int32), _stream(stream)),
        "regione_rikv_store")


def rikv_store_e4m3(k_full, v_full, keep_rows, n_keep, k_q, v_q, k_scale, v_scale, dev_status=None, stream=None):
    """``rikv_store`` into an 8-bit (E4M3) cache with one power-of-two scale per (row, head)."""
    torch = _torch()
    bf = torch.bfloat16
    B, n_full, H, D = k_full.shape
    _check(load().regione_rikv_store_e4m3(
        _ptr(k_full, bf, "k_full"), _ptr(v_full, bf, "v_full"), _ptr(keep_rows, torch.int32),
        _ptr(n_keep, torch.int32), B, n_full, k_q.shape[1], H, D, _ptr(k_q, torch.uint8, "k_q"),
        _ptr(v_q, torch.uint8, "v_q"), _ptr(k_scale, torch.float32, "k_scale"),
        _ptr(v_scale, torch.float32, "v_scale"), _ptr(dev_status, torch.int32), _stream(stream)),
        "regione_rikv_store_e4m3")


def rikv_load_e4m3(k_q, v_q, k_scale, v_scale, n_keep, k_cache, v_cache, dev_status=None, stream=None):
    """Widens an 8-bit cache back to bf16 (exactly the quantised values) for the attention."""
    torch = _torch()
    bf = torch.bfloat16
    B, cap, H, D = k_q.shape
    _check(load().regione_rikv_load_e4m3(
        _ptr(k_q, torch.uint8, "k_q"), _ptr(v_q, torch.uint8, "v_q"), _ptr(k_scale, torch.float32, "k_scale"),
        _ptr(v_scale, torch.float32, "v_scale"), _ptr(n_keep, torch.int32), B, cap, H, D,
        _ptr(k_cache, bf, "k_cache"), _ptr(v_cache, bf, "v_cache"), _ptr(dev_status, torch.int32),
        _stream(stream)), "regione_rikv_load_e4m3")


def fresh_qkv(q_src, k_src, v_src, idx, n, q_weight, k_weight, eps, cos_table, sin_table, rope_layout,
              q_dst, k_dst, v_dst, src_compact=False, dev_status=None, stream=None):
    """Rows of Q, K, V of a region step with the per-head RMS normalisation and the rotary embedding of
    Q and K (angles of position idx[b, j]) in one pass.  ``src_compact``: the sources already hold the
    rows in order (row j), otherwise row idx[b, j] of the whole sequence is gathered."""
    torch = _torch()
    bf, f32 = torch.bfloat16, torch.float32
    B, src_rows, H, D = q_src.shape
    n_pos = cos_table.shape[0]
    if cos_table.shape != (n_pos, D // 2) or sin_table.shape != (n_pos, D // 2):
        raise RegionEError("cos_table and sin_table must be [positions, D / 2]")
    if (src_compact and src_rows != idx.shape[1]) or (not src_compact and src_rows != n_pos):
        raise RegionEError("source rows must match the index capacity (compact) or the table (gathered)")
    _check(load().regione_fresh_qkv(
        _ptr(q_src, bf, "q_src"), _ptr(k_src, bf, "k_src"), _ptr(v_src, bf, "v_src"), _ptr(idx, torch.int32),
        _ptr(n, torch.int32), B, n_pos, idx.shape[1], H, D, 1 if src_compact else 0,
        _ptr(q_weight, bf, "q_weight"), _ptr(k_weight, bf, "k_weight"), float(eps),
        _ptr(cos_table, f32, "cos_table"), _ptr(sin_table, f32, "sin_table"), int(rope_layout),
        _ptr(q_dst, bf, "q_dst"), _ptr(k_dst, bf, "k_dst"), _ptr(v_dst, bf, "v_dst"),
        _ptr(dev_status, torch.int32), _stream(stream)), "regione_fresh_qkv")


def region_attention_workspace(B, Nq_cap, Nf_cap, Nc_cap, H, D) -> int:
    return int(load().regione_region_attention_workspace(B, Nq_cap, Nf_cap, Nc_cap, H, D))


def region_attention(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, out,
                     softmax_scale=0.0, workspace=None, dev_status=None, stream=None):
    torch = _torch()
    bf = torch.bfloat16
    B, Nq_cap, H, D = q.shape
    Nf_cap = 0 if k_fresh is None else k_fresh.shape[1]
    Nc_cap = 0 if k_cache is None else k_cache.shape[1]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    i32 = torch.int32
    _check(load().regione_region_attention(
        _ptr(q, bf, "q"), _ptr(k_fresh, bf, "k_fresh"), _ptr(v_fresh, bf, "v_fresh"),
        _ptr(k_cache, bf, "k_cache"), _ptr(v_cache, bf, "v_cache"), _ptr(n_q, i32), _ptr(n_fresh, i32),
        _ptr(n_cache, i32), B, Nq_cap, Nf_cap, Nc_cap, H, D, float(softmax_scale), _ptr(out, bf, "out"),
        _ptr(workspace, None, "workspace"), ws_bytes, _ptr(dev_status, i32), _stream(stream)),
        "regione_region_attention")


def region_attention_scatter(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, out_full,
                             out_rows, softmax_scale=0.0, workspace=None, dev_status=None, stream=None):
    """``region_attention`` whose row i of request b lands in out_full[b, out_rows[b, i]]."""
    torch = _torch()
    bf = torch.bfloat16
    B, Nq_cap, H, D = q.shape
    Nf_cap = 0 if k_fresh is None else k_fresh.shape[1]
    Nc_cap = 0 if k_cache is None else k_cache.shape[1]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    i32 = torch.int32
    if out_rows.shape[0] != B or out_rows.shape[1] != Nq_cap:
        raise RegionEError("out_rows must be [B, Nq_cap]")
    _check(load().regione_region_attention_scatter(
        _ptr(q, bf, "q"), _ptr(k_fresh, bf, "k_fresh"), _ptr(v_fresh, bf, "v_fresh"),
        _ptr(k_cache, bf, "k_cache"), _ptr(v_cache, bf, "v_cache"), _ptr(n_q, i32), _ptr(n_fresh, i32),
        _ptr(n_cache, i32), B, Nq_cap, Nf_cap, Nc_cap, H, D, float(softmax_scale),
        _ptr(out_full, bf, "out_full"), out_full.shape[1], _ptr(out_rows, i32, "out_rows"),
        _ptr(workspace, None, "workspace"), ws_bytes, _ptr(dev_status, i32), _stream(stream)),
        "regione_region_attention_scatter")


def full_attention_store_workspace(B, N_cap, H, D) -> int:
    return int(load().regione_full_attention_store_workspace(B, N_cap, H, D))


def full_attention_store(q, k, v, n_rows, keep_rows, n_keep, k_cache, v_cache, out, softmax_scale=0.0,
                         workspace=None, dev_status=None, stream=None):
    """Plain joint attention over q / k / v that also writes rows ``keep_rows`` of k and v to the cache."""
    torch = _torch()
    bf, i32 = torch.bfloat16, torch.int32
    B, N_cap, H, D = q.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().regione_full_attention_store(
        _ptr(q, bf, "q"), _ptr(k, bf, "k"), _ptr(v, bf, "v"), _ptr(n_rows, i32, "n_rows"), B, N_cap, H, D,
        float(softmax_scale), _ptr(keep_rows, i32, "keep_rows"), _ptr(n_keep, i32, "n_keep"),
        keep_rows.shape[1], _ptr(k_cache, bf, "k_cache"), _ptr(v_cache, bf, "v_cache"), _ptr(out, bf, "out"),
        _ptr(workspace, None, "workspace"), ws_bytes, _ptr(dev_status, i32), _stream(stream)),
        "regione_full_attention_store")


def region_attention_static(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, out,
                            softmax_scale=0.0, dev_status=None, stream=None):
    """Region attention with the library's built-in 64 MiB scratch: no workspace, no allocation.

    For callers that cannot allocate device memory where they call (all of HBM already owned by
    an arena, or a loop that must not hit the device-wide synchronisation of cudaMalloc).  Calls
    on one device share the scratch, so do not let two of them overlap on the GPU.
    """
    torch = _torch()
    bf = torch.bfloat16
    B, Nq_cap, H, D = q.shape
    Nf_cap = 0 if k_fresh is None else k_fresh.shape[1]
    Nc_cap = 0 if k_cache is None else k_cache.shape[1]
    i32 = torch.int32
    _check(load().regione_region_attention_static(
        _ptr(q, bf, "q"), _ptr(k_fresh, bf, "k_fresh"), _ptr(v_fresh, bf, "v_fresh"),
        _ptr(k_cache, bf, "k_cache"), _ptr(v_cache, bf, "v_cache"), _ptr(n_q, i32), _ptr(n_fresh, i32),
        _ptr(n_cache, i32), B, Nq_cap, Nf_cap, Nc_cap, H, D, float(softmax_scale), _ptr(out, bf, "out"),
        _ptr(dev_status, i32), _stream(stream)), "regione_region_attention_static")


def crosscheck_region_attention(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, out,
                                softmax_scale=0.0, dev_status=None, stream=None):
    """The CUDA-core statement of the attention equation (test infrastructure, not a product path)."""
    torch = _torch()
    bf = torch.bfloat16
    B, Nq_cap, H, D = q.shape
    Nf_cap = 0 if k_fresh is None else k_fresh.shape[1]
    Nc_cap = 0 if k_cache is None else k_cache.shape[1]
    i32 = torch.int32
    _check(load().regione_crosscheck_region_attention(
        _ptr(q, bf, "q"), _ptr(k_fresh, bf, "k_fresh"), _ptr(v_fresh, bf, "v_fresh"),
        _ptr(k_cache, bf, "k_cache"), _ptr(v_cache, bf, "v_cache"), _ptr(n_q, i32), _ptr(n_fresh, i32),
        _ptr(n_cache, i32), B, Nq_cap, Nf_cap, Nc_cap, H, D, float(softmax_scale), _ptr(out, bf, "out"),
        _ptr(dev_status, i32), _stream(stream)), "regione_crosscheck_region_attention")


def selftest_bounded_wait(limit_cycles, dev_status, out=None, stream=None):
    """Lets one bounded wait expire on the device (see the header); ``out`` int64 [3], optional."""
    torch = _torch()
    _check(load().regione_selftest_bounded_wait(
        int(limit_cycles), _ptr(dev_status, torch.int32, "dev_status"), _ptr(out, torch.int64, "out"),
        _stream(stream)), "regione_selftest_bounded_wait")


def avd_step(running_product: float, dt: float, gamma: float, delta: float):
    """Returns (new_running_product, reuse)."""
    p = c_double(running_product)
    r = c_int(0)
    _check(load().regione_avd_step(ctypes.byref(p), dt, gamma, delta, ctypes.byref(r)),
           "regione_avd_step")
    return p.value, bool(r.value)


def gamma_fit(v, dt, norms, gamma, stream=None):
    """v [S, T1, n] bf16, dt [T1-1] f32 -> norms [S, T1], gamma [T1-1] (both f32, written)."""
    torch = _torch()
    S, T1, n = v.shape
    _check(load().regione_gamma_fit(
        _ptr(v, torch.bfloat16, "v"), S, T1, n, _ptr(dt, torch.float32, "dt"),
        _ptr(norms, torch.float32, "norms"), _ptr(gamma, torch.float32, "gamma"), _stream(stream)),
        "regione_gamma_fit")


def velocity_decay(v_in, scale, dt, x_e, n_edit, v_cache_out=None, dev_status=None, stream=None):
    torch = _torch()
    bf = torch.bfloat16
    B, Ne_cap, C = x_e.shape
    _check(load().regione_velocity_decay(
        _ptr(v_in, bf, "v_in"), _per_request(scale, B, "scale"), _per_request(dt, B, "dt"),
        _ptr(x_e, bf, "x_e"),
        _ptr(v_cache_out, bf, "v_cache_out"), _ptr(n_edit, torch.int32), B, Ne_cap, C,
        _ptr(dev_status, torch.int32), _stream(stream)), "regione_velocity_decay")


def merge(x_full, v_last_full, x_e, slot, dt_unedited, x_out, dev_status=None, stream=None):
    torch = _torch()
    bf = torch.bfloat16
    B, N, C = x_full.shape
    _check(load().regione_merge(
        _ptr(x_full, bf, "x_full"), _ptr(v_last_full, bf, "v_last_full"), _ptr(x_e, bf, "x_e"),
        _ptr(slot, torch.int32), _per_request(dt_unedited, B, "dt_unedited"), B, N,
        0 if x_e is None else x_e.shape[1], C,
        _ptr(x_out, bf, "x_out"), _ptr(dev_status, torch.int32), _stream(stream)), "regione_merge")
