/*
 * regione.h -- C ABI of libregione.so: the region-aware denoising step of a
 * flow-matching DiT image editor (RegionE, arXiv 2510.25590), as hand-written
 * CUDA kernels for sm_100a (NVIDIA B200).
 *
 * Conventions
 * -----------
 *  - Every function returns a regione_status.  Argument validation is done
 *    synchronously on the host; the work itself is enqueued on `stream`
 *    (a cudaStream_t passed as void*, NULL = default stream) and is
 *    asynchronous.  Nothing synchronises the device.
 *  - "dev" pointers are device memory owned by the caller; "host" values are
 *    plain scalars.  Unless a function says otherwise the library allocates
 *    nothing and keeps no state between calls.
 *  - bf16 tensors are passed as regione_bf16* (raw bfloat16 bit patterns),
 *    row-major with the last index contiguous.  All bf16 tensors must be
 *    16-byte aligned.  Arithmetic is fp32; results are rounded to bf16 with
 *    round-to-nearest-even.
 *  - Per-request counts (n_edit, n_q, ...) live in device memory as int32 so
 *    that no host round trip is needed between the partition and the calls
 *    that consume its output; capacities (*_cap) are host ints.
 *  - `dev_status` (nullable, device int32, caller zeroes it) receives
 *    REGIONE_DEV_BOUNDS or REGIONE_DEV_TIMEOUT if a kernel meets an index or
 *    count outside its capacity or a bounded wait runs out.  Kernels never
 *    trap: the offending access is skipped and the kernel ends normally.
 *  - Every kernel of the product entry points is launched with programmatic
 *    stream serialization and begins with a dependency wait: the order of work
 *    on `stream` is exactly that of ordinary launches (also under stream
 *    capture), only the launch of a kernel overlaps the tail of the kernel
 *    before it.  The two entry points of the "cross-check and self-test"
 *    section at the end are ordinary launches.
 *  - B is the number of independent edit requests in the batch.  Each request
 *    may sit at its own sampler step: the sampler scalars (t, dt, scale,
 *    dt_unedited) are host arrays of B floats, read during the call (the
 *    values travel to the kernels as launch parameters, 128 requests per
 *    launch; the arrays may be reused as soon as the call returns).  A request
 *    whose scalar is NaN (t for the partition, dt or scale for the velocity
 *    decay, dt_unedited for the merge) sits that call out: nothing of it is
 *    read or written.  This is how a batch whose requests are at different
 *    kinds of step shares one launch.
 *  - There is no CPU fallback: without a CUDA device every compute entry point
 *    returns REGIONE_CUDA_ERROR.
 */
#ifndef REGIONE_H_
#define REGIONE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t regione_bf16;

typedef enum {
    REGIONE_OK = 0,
    REGIONE_INVALID_ARG = 1,        /* null pointer, negative size, misaligned pointer */
    REGIONE_UNSUPPORTED = 2,        /* shape outside what the kernels implement */
    REGIONE_CUDA_ERROR = 3,         /* a CUDA runtime/driver call failed (launch, tensor map) */
    REGIONE_WORKSPACE_TOO_SMALL = 4
} regione_status;

enum { REGIONE_DEV_OK = 0, REGIONE_DEV_TIMEOUT = 5, REGIONE_DEV_BOUNDS = 6 };

enum { REGIONE_METRIC_COSINE = 0, REGIONE_METRIC_L2 = 1 };

/* membership of the joint sequence rows in one region-attention call */
enum { REGIONE_ROWS_EDITED_QUERIES = 0, REGIONE_ROWS_PAPER = 1 };
/* which elements of a head form a rotary pair: (2i, 2i+1) or (i, i + D/2) */
enum { REGIONE_ROPE_INTERLEAVED = 0, REGIONE_ROPE_HALF = 1 };

/* Library version (major*10000 + minor*100 + patch) and status names. */
int regione_version(void);
const char* regione_status_string(int status);

/*
 * Adaptive Region Partition (Sec. 4, "Adaptive Region Partition"; Algorithm 1,
 * the two lines computing X_hat_0 and E_index/U_index), without the
 * morphological clean-up.
 *
 * For every request b and token n:
 *     x0_hat[c] = x_t[b,n,c] - t * v[b,n,c]                (one-step estimate, t_f = 0)
 *     s = cos(x0_hat, ref[b,n,:])      (metric COSINE;  edited iff s <= threshold)
 *     s = || x0_hat - ref[b,n,:] ||_2  (metric L2;      edited iff s >  threshold)
 * and then, per request, the ascending index lists:
 *     edit_idx[b, 0..n_edit[b])      token ids with mask = 1
 *     keep_idx[b, 0..N-n_edit[b])    token ids with mask = 0
 *     slot[b,n] = position of n in edit_idx, or -1
 * A zero cosine denominator is clamped at 1e-12.
 *
 * x_t, v, ref : dev bf16 [B, N, C], C a multiple of 8 and <= 4096
 * t           : host f32 [B], the sampler time of each request
 * mask        : dev u8    [B, N]   (1 = edited)
 * edit_idx, keep_idx, slot : dev int32 [B, N]; entries of edit_idx / keep_idx past
 *               the live prefix are left untouched
 * n_edit      : dev int32 [B]
 * score       : dev f32   [B, N], nullable; receives s
 * Limits: 1 <= N <= 2^20 per request (REGIONE_UNSUPPORTED above), B <= 65535.
 * One kernel launch per 128 requests; a call of few long requests (N >= 32768, at most 18
 * requests) takes two per 128, the decisions and then the compaction, with the same results.
 */
int regione_partition(const regione_bf16* x_t, const regione_bf16* v, const regione_bf16* ref,
                      int B, int N, int C, const float* t, int metric, float threshold,
                      uint8_t* mask, int32_t* edit_idx, int32_t* keep_idx, int32_t* slot,
                      int32_t* n_edit, float* score, int32_t* dev_status, void* stream);

/*
 * regione_partition and regione_region_rows (below) in one call: the partition
 * of Sec. 4 "Adaptive Region Partition" that also writes the joint-sequence row
 * lists of the region-attention layer (Sec. 4 "Region-Aware Generation").  Same
 * arguments, layouts, limits and results as the two calls made one after the
 * other; the row lists are composed while the index lists are written, so the
 * launch of regione_region_rows and its pass over the lists are saved.
 */
int regione_partition_rows(const regione_bf16* x_t, const regione_bf16* v, const regione_bf16* ref,
                           int B, int N, int C, const float* t, int metric, float threshold,
                           uint8_t* mask, int32_t* edit_idx, int32_t* keep_idx, int32_t* slot,
                           int32_t* n_edit, float* score,
                           int n_text, int n_ref, int membership,
                           int32_t* query_rows, int32_t* n_query, int q_cap,
                           int32_t* cache_rows, int32_t* n_cache, int c_cap,
                           int32_t* dev_status, void* stream);

/*
 * Morphological opening then closing of the edited mask on the rows x cols token
 * grid (Sec. 4, "Adaptive Region Partition", the clean-up that makes the two
 * regions more contiguous; Algorithm 1 names an erosion and a dilation), followed
 * by the same compaction as regione_partition.  Structuring element 3x3; neighbours
 * outside the grid are ignored.  mask_in [B, rows*cols] -> mask_out and the index lists.
 * mask_in and mask_out may not alias.  rows*cols <= 16384.
 * dev_status is accepted for uniformity and never written: the kernel has no count
 * or index input that could be out of range on the device.
 */
int regione_mask_open_close(const uint8_t* mask_in, int B, int rows, int cols,
                            uint8_t* mask_out, int32_t* edit_idx, int32_t* keep_idx,
                            int32_t* slot, int32_t* n_edit, int32_t* dev_status, void* stream);

/*
 * Joint-sequence row lists for one region-attention layer, composed on the
 * device from the partition's output (Sec. 4, "Region-Aware Generation": which
 * tokens are recomputed and which come from the cache).  The joint sequence is
 * [text (n_text) | image (N) | reference (n_ref)].
 *   REGIONE_ROWS_EDITED_QUERIES: query_rows = n_text + edit_idx;
 *        cache_rows = text, n_text + keep_idx, reference   (ascending)
 *   REGIONE_ROWS_PAPER: query_rows = text, n_text + edit_idx;
 *        cache_rows = n_text + keep_idx, reference
 * query_rows : dev int32 [B, q_cap],  n_query dev int32 [B]
 * cache_rows : dev int32 [B, c_cap],  n_cache dev int32 [B]
 * Counts beyond a capacity are clamped and REGIONE_DEV_BOUNDS is recorded.
 */
int regione_region_rows(const int32_t* edit_idx, const int32_t* keep_idx, const int32_t* n_edit,
                        int B, int N, int n_text, int n_ref, int membership,
                        int32_t* query_rows, int32_t* n_query, int q_cap,
                        int32_t* cache_rows, int32_t* n_cache, int c_cap,
                        int32_t* dev_status, void* stream);

/*
 * Token gather (Algorithm 1: X^E = X[E_index], X^U = X[U_index]):
 *     dst[b, j, :] = src[b, idx[b, j], :]     for j < min(n[b], dst_rows_cap)
 * Rows are opaque byte strings of row_bytes (a multiple of 16) bytes.
 * src [B, src_rows, row_bytes], idx dev int32 [B, idx_stride], n dev int32 [B],
 * dst [B, dst_rows_cap, row_bytes].  Rows of dst past n[b] are left untouched.
 * An index outside [0, src_rows) is skipped and REGIONE_DEV_BOUNDS recorded.
 */
int regione_gather(const void* src, const int32_t* idx, const int32_t* n, int B,
                   int64_t src_rows, int64_t idx_stride, int64_t dst_rows_cap, int64_t row_bytes,
                   void* dst, int32_t* dev_status, void* stream);

/*
 * The same gather for up to 4 tensors of identical shape that share one index list, in one
 * launch (Algorithm 1 gathers X and v, and the recomputed rows of Q, K and V, with the same
 * E_index): dsts[i][b, j, :] = srcs[i][b, idx[b, j], :].
 * srcs, dsts : host arrays of n_tensors device pointers (1 <= n_tensors <= 4).
 */
int regione_gather_multi(const void* const* srcs, void* const* dsts, int n_tensors,
                         const int32_t* idx, const int32_t* n, int B, int64_t src_rows,
                         int64_t idx_stride, int64_t dst_rows_cap, int64_t row_bytes,
                         int32_t* dev_status, void* stream);

/*
 * Producer of a region step's fresh Q / K / V rows: the gather of the recomputed tokens' rows of Q,
 * K and V (Algorithm 1: the same E_index for all three) fused with the two operations the editors
 * apply to Q and K before attention, per-head RMS normalisation and rotary position embedding.  The
 * paper does not state those two (it takes the attention layer as given); what it fixes is that a
 * recomputed token keeps its place in the joint sequence (Sec. 4 "Region-Aware Generation": region
 * tokens are gathered and later put back by spatial position), so idx[b, j] is both the row that is
 * gathered and the position whose angles rotate it.
 *     y      = x / sqrt(mean_D(x^2) + eps) * weight          per row and head, fp32
 *     (a, b) -> (a cos t - b sin t, a sin t + b cos t)       for each of the D/2 pairs of y,
 *               t = angle i of position idx[b, j]; pair i = elements (2i, 2i+1)
 *               (REGIONE_ROPE_INTERLEAVED) or (i, i + D/2) (REGIONE_ROPE_HALF)
 *     q_dst[b, j, h, :] = rotate(norm(q_src[b, idx[b, j], h, :], q_weight)),  the same for K with
 *     k_weight;  v_dst[b, j] = v_src[b, idx[b, j]]             for j < n[b]; one rounding to bf16
 * src_compact = 0: q_src, k_src, v_src [B, N_src, H, D] bf16 hold the whole sequence and row idx[b, j]
 * is gathered (projections computed for every row, as in a full step or a synthetic layer);
 * src_compact = 1: they are [B, cap, H, D] and row j is read (projections computed for the recomputed
 * rows only, as a region step does); idx[b, j] is the position in both cases.  Source and
 * destination must not overlap.  idx dev int32 [B, cap]; n dev int32 [B];
 * q_weight, k_weight dev bf16 [D] or NULL (all ones); cos_table, sin_table dev fp32 [N_src, D/2]
 * (cosine and sine of the angles of every position: any frequency scheme, several axes included);
 * q_dst, k_dst, v_dst [B, cap, H, D].  D is 64 or 128; all buffers 16-byte aligned.
 * Rows past n[b] are left untouched; an index outside [0, N_src) is skipped and REGIONE_DEV_BOUNDS
 * recorded.  Nothing is allocated; the buffers stay the caller's.
 */
int regione_fresh_qkv(const regione_bf16* q_src, const regione_bf16* k_src, const regione_bf16* v_src,
                      const int32_t* idx, const int32_t* n, int B, int N_src, int cap, int H, int D,
                      int src_compact, const regione_bf16* q_weight, const regione_bf16* k_weight, float eps,
                      const float* cos_table, const float* sin_table, int rope_layout,
                      regione_bf16* q_dst, regione_bf16* k_dst, regione_bf16* v_dst,
                      int32_t* dev_status, void* stream);

/*
 * Token scatter, the inverse placement (Sec. 4, end of the AVDCache paragraph: the
 * region results are put back at their spatial positions; Algorithm 1, the
 * gather(...) line):
 *     dst[b, idx[b, j], :] = src[b, j, :]     for j < min(n[b], src_rows_cap)
 * Other rows of dst are left untouched.  idx must not repeat a row.
 */
int regione_scatter(const void* src, const int32_t* idx, const int32_t* n, int B,
                    int64_t src_rows_cap, int64_t idx_stride, int64_t dst_rows, int64_t row_bytes,
                    void* dst, int32_t* dev_status, void* stream);

/*
 * Region-Instruction KV cache store (Sec. 4, "Stabilization Stage": the Key and
 * Value of each attention layer are saved at the last full step; refreshed at
 * forced steps).  Compacts the retained rows of one layer's full K and V:
 *     k_cache[b, j, :, :] = k_full[b, keep_rows[b, j], :, :]   (same for V),  j < n_keep[b]
 * k_full, v_full [B, N_full, H, D] bf16; keep_rows dev int32 [B, Nc_cap];
 * k_cache, v_cache [B, Nc_cap, H, D].  H*D must be a multiple of 8.
 */
int regione_rikv_store(const regione_bf16* k_full, const regione_bf16* v_full,
                       const int32_t* keep_rows, const int32_t* n_keep,
                       int B, int N_full, int Nc_cap, int H, int D,
                       regione_bf16* k_cache, regione_bf16* v_cache,
                       int32_t* dev_status, void* stream);

/*
 * 8-bit variant of the Region-Instruction KV cache.  (Sec. 4 "Stabilization Stage" keeps K and V of
 * every attention layer from one full step to the next forced one; the paper keeps them in the
 * model's precision, so this storage format has no counterpart there.)  regione_rikv_store_e4m3 is
 * regione_rikv_store with the retained rows written as 8-bit floating point E4M3 (1 sign, 4 exponent,
 * 3 mantissa bits, bias 7, largest finite value 448, no infinities) and one power-of-two scale per
 * (row, head): half the bytes per cached layer.  regione_rikv_load_e4m3 widens such a cache back
 * to bf16 in front of a region step's attention:
 *     s = 2^k, k the smallest integer with max_d |x[b,row,h,d]| / 2^k <= 448   (k = 0 for an all-zero
 *         row and head; k >= -100)
 *     code = nearest E4M3 value of x / s, ties to the even mantissa
 *     k_cache[b,j,h,d] = value(code) * s        (exact in bf16: no second rounding)
 * k_full, v_full [B, N_full, H, D] bf16; keep_rows dev int32 [B, Nc_cap]; n_keep dev int32 [B];
 * k_q, v_q dev u8 [B, Nc_cap, H, D]; k_scale, v_scale dev f32 [B, Nc_cap, H];
 * k_cache, v_cache dev bf16 [B, Nc_cap, H, D].  Rows past n_keep[b] are left untouched by both.
 * D must be 64 or 128.  NaN elements are not preserved.
 */
int regione_rikv_store_e4m3(const regione_bf16* k_full, const regione_bf16* v_full,
                            const int32_t* keep_rows, const int32_t* n_keep,
                            int B, int N_full, int Nc_cap, int H, int D,
                            uint8_t* k_q, uint8_t* v_q, float* k_scale, float* v_scale,
                            int32_t* dev_status, void* stream);
int regione_rikv_load_e4m3(const uint8_t* k_q, const uint8_t* v_q, const float* k_scale,
                           const float* v_scale, const int32_t* n_keep,
                           int B, int Nc_cap, int H, int D,
                           regione_bf16* k_cache, regione_bf16* v_cache,
                           int32_t* dev_status, void* stream);

/*
 * Region attention with the Region-Instruction KV cache (Sec. 4, "Region-Aware
 * Generation", the attention equation):
 *     out[b,i,h,:] = sum_j softmax_j( scale * q[b,i,h,:] . k_j ) * v_j
 * with j running over the fresh rows 0..n_fresh[b) of (k_fresh, v_fresh) and the
 * cached rows 0..n_cache[b) of (k_cache, v_cache); the concatenation is never
 * materialised.  No mask, no positional encoding (the cache holds K as it
 * entered the softmax at the storing step).
 *
 * q, out          : dev bf16 [B, Nq_cap, H, D];  rows i >= n_q[b] are not written
 * k_fresh, v_fresh: dev bf16 [B, Nf_cap, H, D]
 * k_cache, v_cache: dev bf16 [B, Nc_cap, H, D]   (may be NULL when Nc_cap == 0)
 * n_q, n_fresh, n_cache : dev int32 [B]; values above the capacity are clamped and
 *                   REGIONE_DEV_BOUNDS recorded
 * softmax_scale   : <= 0 selects 1/sqrt(D)
 * workspace       : dev, 256-byte aligned, at least
 *                   regione_region_attention_workspace(...) bytes.  It holds the
 *                   partial results of (request, head, query-tile pair) items whose
 *                   key range was shared between thread blocks, and a small table
 *                   naming those items; its contents need not be initialised and
 *                   mean nothing after the call.
 * D must be 64 or 128.  bf16 inputs, fp32 accumulation, probabilities rounded
 * to bf16 before the second product.  With no key at all a row is zero.
 * The call enqueues two kernels (attention, then the merge of shared items; the
 * second is launched with programmatic stream serialization, i.e. it may become
 * resident while the first drains and waits for its completion on the device).
 */
size_t regione_region_attention_workspace(int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D);
int regione_region_attention(const regione_bf16* q,
                             const regione_bf16* k_fresh, const regione_bf16* v_fresh,
                             const regione_bf16* k_cache, const regione_bf16* v_cache,
                             const int32_t* n_q, const int32_t* n_fresh, const int32_t* n_cache,
                             int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D,
                             float softmax_scale, regione_bf16* out,
                             void* workspace, size_t workspace_bytes,
                             int32_t* dev_status, void* stream);

/*
 * regione_region_attention followed by regione_scatter of its rows, in the same
 * launches (Sec. 4: the attention rows of the recomputed tokens are put back at
 * their positions in the joint sequence): the result of query row i of request b
 * is written to out_full[b, out_rows[b, i], :, :] instead of out[b, i, :, :].
 *
 * out_full : dev bf16 [B, out_rows_cap, H, D]; rows not named by out_rows[b, 0..n_q[b])
 *            are left untouched
 * out_rows : dev int32 [B, Nq_cap]; an entry outside [0, out_rows_cap) drops that
 *            row and records REGIONE_DEV_BOUNDS
 * Everything else as regione_region_attention (same workspace query).
 */
int regione_region_attention_scatter(const regione_bf16* q,
                                     const regione_bf16* k_fresh, const regione_bf16* v_fresh,
                                     const regione_bf16* k_cache, const regione_bf16* v_cache,
                                     const int32_t* n_q, const int32_t* n_fresh, const int32_t* n_cache,
                                     int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D,
                                     float softmax_scale, regione_bf16* out_full, int out_rows_cap,
                                     const int32_t* out_rows,
                                     void* workspace, size_t workspace_bytes,
                                     int32_t* dev_status, void* stream);

/*
 * Full attention step that refreshes the Region-Instruction KV cache in passing (Sec. 4,
 * "Stabilization Stage": the last full step saves K and V of every attention layer; end of the
 * "Adaptive Velocity Decay Cache" paragraph: forced full-image steps update the cache; Algorithm 1,
 * the store flag f[0] of a full DiT call).  One call does what
 *     regione_region_attention(q, k, v, NULL, NULL, n_rows, n_rows, 0, ...)     (plain joint attention)
 *     regione_rikv_store(k, v, keep_rows, n_keep, ...)
 * do one after the other, bit for bit the same cache and the same output, but K and V are read from
 * device memory once: the attention kernel stages every K / V tile of a head in shared memory anyway,
 * and the thread block that walks the first query rows of a (request, head) writes the retained
 * rows of each tile from there to their slots in the cache.
 *
 * q, k, v, out : dev bf16 [B, N_cap, H, D];  n_rows dev int32 [B] live rows (queries = keys)
 * keep_rows    : dev int32 [B, Nc_cap], strictly ascending per request (as regione_region_rows
 *                and regione_partition_rows write them); n_keep dev int32 [B]
 * k_cache, v_cache : dev bf16 [B, Nc_cap, H, D]; rows past n_keep[b] are left untouched
 * An entry of keep_rows outside [0, n_rows[b]) or out of order is skipped and REGIONE_DEV_BOUNDS
 * recorded.  A request with n_rows[b] = 0 stores nothing.  Workspace: at least
 * regione_full_attention_store_workspace(...) bytes, 256-byte aligned (it equals the query of
 * regione_region_attention_workspace(B, N_cap, N_cap, 0, H, D)).  D must be 64 or 128.
 */
size_t regione_full_attention_store_workspace(int B, int N_cap, int H, int D);
int regione_full_attention_store(const regione_bf16* q, const regione_bf16* k, const regione_bf16* v,
                                 const int32_t* n_rows, int B, int N_cap, int H, int D,
                                 float softmax_scale,
                                 const int32_t* keep_rows, const int32_t* n_keep, int Nc_cap,
                                 regione_bf16* k_cache, regione_bf16* v_cache, regione_bf16* out,
                                 void* workspace, size_t workspace_bytes,
                                 int32_t* dev_status, void* stream);

/*
 * Region attention that brings its own scratch memory.  (The paper has no
 * counterpart: this entry point exists only for the way the library is deployed.)
 *
 * Same computation, arguments and limits as regione_region_attention, without the
 * workspace pair.  It is meant for callers that cannot obtain device memory at the
 * point of the call: an inference server that hands all of HBM to its own arena at
 * start-up so a later cudaMalloc fails, or a denoising loop that must not stall,
 * since cudaMalloc / cudaFree synchronise the whole device.  The split-KV partials
 * go to a 64 MiB array compiled into the library (device memory that every GPU
 * loading the library holds until the process ends); the call itself requests no
 * memory from the CUDA runtime or any other allocator.
 *
 *  - A shape whose partials would not fit, i.e.
 *    regione_region_attention_workspace(...) > 64 MiB, is refused with
 *    REGIONE_WORKSPACE_TOO_SMALL; nothing is launched.
 *  - The first call on each device looks the array's device address up (with that
 *    device current) and remembers it.  Make that first call outside any stream
 *    capture.  Under the CUDA runtime's lazy module loading that first use is also
 *    the moment the driver places the library's device image, array included, in
 *    device memory: make one warm-up call per device at start-up, BEFORE an arena
 *    takes the rest of HBM, or the warm-up itself fails with REGIONE_CUDA_ERROR.
 *  - All calls on a device share the one array and it keeps whatever the last call
 *    left in it.  Nothing in it needs clearing between calls, but two calls whose
 *    kernels overlap on the GPU (different streams) race on it: serialise them.
 */
int regione_region_attention_static(const regione_bf16* q,
                                    const regione_bf16* k_fresh, const regione_bf16* v_fresh,
                                    const regione_bf16* k_cache, const regione_bf16* v_cache,
                                    const int32_t* n_q, const int32_t* n_fresh, const int32_t* n_cache,
                                    int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D,
                                    float softmax_scale, regione_bf16* out,
                                    int32_t* dev_status, void* stream);

/*
 * One step of the AVDCache criterion (Sec. 4, "Adaptive Velocity Decay Cache",
 * the decay-factor and criterion equations).  Pure host arithmetic:
 *     p = *running_product * (1 - dt) * gamma
 *     if 1 - p > delta : *reuse = 0, *running_product = 1     (recompute, refresh the cache)
 *     else             : *reuse = 1, *running_product = p     (use cached velocity * p)
 */
int regione_avd_step(double* running_product, double dt, double gamma, double delta, int* reuse);

/*
 * Fit of the timestep-aware decay correction gamma (Sec. 4, "Adaptive Velocity Decay
 * Cache", decay-factor equation: ||v_{t_i}|| / ||v_{t_{i+1}}|| = (1 - dt_i) * gamma_{t_i};
 * the paper fits gamma on sampled data).  From the velocities of S
 * sampled trajectories at T1 consecutive steps:
 *     norms[s, i] = || v[s, i, :] ||_2
 *     gamma[i]    = mean_s( norms[s, i] / norms[s, i+1] ) / (1 - dt[i]),     i < T1 - 1
 * (index i+1 is the earlier, noisier step).  The paper does not say how it fits; the mean of
 * the per-sample ratios is this library's reading.
 * v : dev bf16 [S, T1, n], n a multiple of 8;  dt : dev f32 [T1-1];
 * norms : dev f32 [S, T1] (output);  gamma : dev f32 [T1-1] (output).
 */
int regione_gamma_fit(const regione_bf16* v, int S, int T1, int64_t n, const float* dt,
                      float* norms, float* gamma, void* stream);

/*
 * Decayed cached velocity and Euler update of the edited tokens (Sec. 4, the
 * case equation of the AVDCache; Sec. 3, the Euler sampler equation):
 *     v_use = scale[b] * v_in[b,j,:]
 *     x_e[b,j,:] <- x_e[b,j,:] - dt[b] * v_use             for j < n_edit[b]
 *     v_cache_out[b,j,:] <- v_in[b,j,:]   (if v_cache_out != NULL: a recomputed step
 *                                          refreshes the velocity cache)
 * scale[b] is the accumulated decay product on a reused step and 1 on a recomputed one.
 * v_in, x_e, v_cache_out : dev bf16 [B, Ne_cap, C], C a multiple of 8.
 * scale, dt : host f32 [B] (requests of one batch may sit at different sampler steps).
 */
int regione_velocity_decay(const regione_bf16* v_in, const float* scale, const float* dt, regione_bf16* x_e,
                           regione_bf16* v_cache_out, const int32_t* n_edit,
                           int B, int Ne_cap, int C, int32_t* dev_status, void* stream);

/*
 * Merge of the two regions at the end of a run of region steps (Sec. 4, one-step
 * estimation equation applied to the unedited tokens; Algorithm 1, the one-step
 * line before the inner loop and the gather line after it):
 *     x_out[b,n,:] = slot[b,n] >= 0 ? x_e[b, slot[b,n], :]
 *                                   : x_full[b,n,:] - dt_unedited[b] * v_last_full[b,n,:]
 * x_full, v_last_full, x_out : dev bf16 [B, N, C]; x_e [B, Ne_cap, C]; slot dev int32 [B, N];
 * dt_unedited host f32 [B].  x_out may alias x_full.  A slot >= Ne_cap is skipped and REGIONE_DEV_BOUNDS recorded.
 */
int regione_merge(const regione_bf16* x_full, const regione_bf16* v_last_full,
                  const regione_bf16* x_e, const int32_t* slot, const float* dt_unedited,
                  int B, int N, int Ne_cap, int C, regione_bf16* x_out,
                  int32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Cross-check and self-test entry points.  Test infrastructure that has to live inside the
 * library because it runs on the device; no product entry point above calls either of them,
 * and both are ordinary (not dependency-wait) launches.
 * ------------------------------------------------------------------------------------------ */

/*
 * The attention equation of Sec. 4 "Region-Aware Generation" once more, on the CUDA cores: one
 * warp per (request, head, query row), fp32 online softmax, no tensor cores, no shared plan.
 * Same arguments, layouts and results as regione_region_attention minus the workspace.  It is
 * orders of magnitude slower and exists so that tests can compare the tensor-core kernel with
 * an independent arithmetic path on the same device at sizes where the CPU oracle is slow.
 */
int regione_crosscheck_region_attention(const regione_bf16* q,
                                        const regione_bf16* k_fresh, const regione_bf16* v_fresh,
                                        const regione_bf16* k_cache, const regione_bf16* v_cache,
                                        const int32_t* n_q, const int32_t* n_fresh, const int32_t* n_cache,
                                        int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D,
                                        float softmax_scale, regione_bf16* out,
                                        int32_t* dev_status, void* stream);

/*
 * Lets a bounded wait run out, in the harmless form (the paper has no counterpart; this covers
 * the convention above that a wait that expires ends in REGIONE_DEV_TIMEOUT).  One thread of one
 * thread block waits, through the very routine the attention kernel's roles wait with, on a
 * barrier that nothing ever arrives on, with no copy and no tensor-core operation in flight.
 * After limit_cycles SM clock cycles (1 .. 10^8) the wait gives up, REGIONE_DEV_TIMEOUT is
 * recorded in dev_status and the kernel ends normally; the context stays usable.
 * out : dev int64 [3], nullable: {1 if the wait claimed completion (must be 0), cycles spent
 *       waiting, the abort flag the other roles would have seen (must be 1)}.
 */
int regione_selftest_bounded_wait(long long limit_cycles, int32_t* dev_status, long long* out,
                                  void* stream);

#ifdef __cplusplus
}
#endif
#endif /* REGIONE_H_ */
