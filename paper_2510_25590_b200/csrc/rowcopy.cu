// Indexed row copies: token gather / scatter (Algorithm 1: X[E_index] and the
// re-gathering by spatial position) and the Region-Instruction KV cache store
// (Sec. 4 "Stabilization Stage": K and V of every attention layer are saved).
//
// All three are pure HBM traffic.  Rows are byte strings whose length is a
// multiple of 16; a thread moves kUnroll 16-byte chunks that are blockDim
// apart, so a warp always touches 512 contiguous bytes per request, all loads
// of a thread are issued before its first store, and source data (read once)
// bypasses L1.
#include "common.cuh"

namespace regione {

constexpr int kCopyThreads = 256;
constexpr int kUnroll = 8;

struct RowCopyPair {
    const uint4* src;
    uint4* dst;
};

constexpr int kMaxPairs = 4;                 // tensors sharing one index list in one launch
struct RowCopyPairs {
    RowCopyPair p[kMaxPairs];
};

// GATHER: dst[b, j] = src[b, idx[b, j]];  !GATHER: dst[b, idx[b, j]] = src[b, j].
// `idx_rows` bounds the indexed side, `cap` the dense side.  blockIdx.z picks the tensor pair.
template <bool GATHER>
__global__ void __launch_bounds__(kCopyThreads)
row_copy_kernel(const RowCopyPairs pairs, const int32_t* __restrict__ idx,
                const int32_t* __restrict__ n, long long idx_rows, long long idx_stride,
                long long cap, int cpr, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int b = blockIdx.y;
    const RowCopyPair p = pairs.p[blockIdx.z];
    long long live = n[b];
    if (live < 0 || live > cap) {
        if (threadIdx.x == 0 && blockIdx.x == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        live = live < 0 ? 0 : cap;
    }
    // 32-bit chunk arithmetic: the host guarantees cap * cpr < 2^31.
    const unsigned total = (unsigned)live * (unsigned)cpr;
    const unsigned base = blockIdx.x * (unsigned)(kCopyThreads * kUnroll) + threadIdx.x;
    if (base >= total) return;
    const uint4* __restrict__ src = p.src + (size_t)b * (GATHER ? idx_rows : cap) * cpr;
    uint4* __restrict__ dst = p.dst + (size_t)b * (GATHER ? cap : idx_rows) * cpr;
    const int32_t* __restrict__ my_idx = idx + (size_t)b * idx_stride;

    // (row j, chunk c) of the first element; later elements advance by kCopyThreads chunks.
    unsigned j = base / (unsigned)cpr;
    unsigned c = base - j * (unsigned)cpr;
    const unsigned step_rows = (unsigned)kCopyThreads / (unsigned)cpr;
    const unsigned step_chunks = (unsigned)kCopyThreads - step_rows * (unsigned)cpr;

    uint4 val[kUnroll];
    long long to[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const unsigned e = base + (unsigned)u * kCopyThreads;
        to[u] = -1;
        if (e < total) {
            const long long r = my_idx[j];
            if (r < 0 || r >= idx_rows) {
                record_status(dev_status, REGIONE_DEV_BOUNDS);
            } else {
                const long long from = (GATHER ? r : (long long)j) * cpr + c;
                to[u] = (GATHER ? (long long)j : r) * cpr + c;
                val[u] = ld_stream128(src + from);
            }
        }
        j += step_rows;
        c += step_chunks;
        if (c >= (unsigned)cpr) { c -= (unsigned)cpr; ++j; }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
        if (to[u] >= 0) dst[to[u]] = val[u];
}

template <bool GATHER>
static int launch_row_copy(const RowCopyPairs& ps, int pairs, const int32_t* idx,
                           const int32_t* n, int B, long long idx_rows, long long idx_stride,
                           long long cap, long long row_bytes, int32_t* dev_status, void* stream) {
    const long long cpr = row_bytes / 16;
    const long long per_block = (long long)kCopyThreads * kUnroll;
    const long long blocks = (cap * cpr + per_block - 1) / per_block;
    if (cap * cpr + per_block >= 0x7fffffffLL) return REGIONE_UNSUPPORTED;
    dim3 grid((unsigned)blocks, (unsigned)B, (unsigned)pairs);
    return launch_status(launch_overlapped(row_copy_kernel<GATHER>, grid, dim3(kCopyThreads), 0,
                                           (cudaStream_t)stream, ps, idx, n, idx_rows, idx_stride,
                                           cap, (int)cpr, dev_status));
}

}  // namespace regione

using namespace regione;

static int check_rows(const void* src, const void* idx, const void* n, const void* dst, int B,
                      int64_t a, int64_t stride, int64_t c, int64_t row_bytes) {
    if (!src || !idx || !n || !dst) return REGIONE_INVALID_ARG;
    if (B < 0 || a < 0 || c < 0 || stride < 0 || row_bytes <= 0) return REGIONE_INVALID_ARG;
    if (!aligned16(src) || !aligned16(dst)) return REGIONE_INVALID_ARG;
    if (row_bytes % 16 != 0 || B > 65535) return REGIONE_UNSUPPORTED;
    return REGIONE_OK;
}

extern "C" int regione_gather(const void* src, const int32_t* idx, const int32_t* n, int B,
                              int64_t src_rows, int64_t idx_stride, int64_t dst_rows_cap,
                              int64_t row_bytes, void* dst, int32_t* dev_status, void* stream) {
    int s = check_rows(src, idx, n, dst, B, src_rows, idx_stride, dst_rows_cap, row_bytes);
    if (s != REGIONE_OK) return s;
    if (idx_stride < dst_rows_cap) return REGIONE_INVALID_ARG;
    if (B == 0 || dst_rows_cap == 0) return REGIONE_OK;
    RowCopyPairs ps = {};
    ps.p[0] = RowCopyPair{(const uint4*)src, (uint4*)dst};
    return launch_row_copy<true>(ps, 1, idx, n, B, src_rows, idx_stride, dst_rows_cap, row_bytes,
                                 dev_status, stream);
}

extern "C" int regione_scatter(const void* src, const int32_t* idx, const int32_t* n, int B,
                               int64_t src_rows_cap, int64_t idx_stride, int64_t dst_rows,
                               int64_t row_bytes, void* dst, int32_t* dev_status, void* stream) {
    int s = check_rows(src, idx, n, dst, B, dst_rows, idx_stride, src_rows_cap, row_bytes);
    if (s != REGIONE_OK) return s;
    if (idx_stride < src_rows_cap) return REGIONE_INVALID_ARG;
    if (B == 0 || src_rows_cap == 0) return REGIONE_OK;
    RowCopyPairs ps = {};
    ps.p[0] = RowCopyPair{(const uint4*)src, (uint4*)dst};
    return launch_row_copy<false>(ps, 1, idx, n, B, dst_rows, idx_stride, src_rows_cap, row_bytes,
                                  dev_status, stream);
}

extern "C" int regione_rikv_store(const regione_bf16* k_full, const regione_bf16* v_full,
                                  const int32_t* keep_rows, const int32_t* n_keep, int B,
                                  int N_full, int Nc_cap, int H, int D, regione_bf16* k_cache,
                                  regione_bf16* v_cache, int32_t* dev_status, void* stream) {
    if (!k_full || !v_full || !keep_rows || !n_keep || !k_cache || !v_cache)
        return REGIONE_INVALID_ARG;
    if (B < 0 || N_full < 0 || Nc_cap < 0 || H < 1 || D < 1) return REGIONE_INVALID_ARG;
    if (!aligned16(k_full) || !aligned16(v_full) || !aligned16(k_cache) || !aligned16(v_cache))
        return REGIONE_INVALID_ARG;
    const long long row_bytes = (long long)H * D * 2;
    if (row_bytes % 16 != 0 || B > 65535) return REGIONE_UNSUPPORTED;
    if (B == 0 || Nc_cap == 0) return REGIONE_OK;
    RowCopyPairs ps = {};
    ps.p[0] = RowCopyPair{(const uint4*)k_full, (uint4*)k_cache};
    ps.p[1] = RowCopyPair{(const uint4*)v_full, (uint4*)v_cache};
    return launch_row_copy<true>(ps, 2, keep_rows, n_keep, B, N_full, Nc_cap, Nc_cap, row_bytes,
                                 dev_status, stream);
}

extern "C" int regione_gather_multi(const void* const* srcs, void* const* dsts, int n_tensors,
                                    const int32_t* idx, const int32_t* n, int B, int64_t src_rows,
                                    int64_t idx_stride, int64_t dst_rows_cap, int64_t row_bytes,
                                    int32_t* dev_status, void* stream) {
    if (!srcs || !dsts || n_tensors < 1 || n_tensors > kMaxPairs) return REGIONE_INVALID_ARG;
    RowCopyPairs ps = {};
    for (int i = 0; i < n_tensors; ++i) {
        int s = check_rows(srcs[i], idx, n, dsts[i], B, src_rows, idx_stride, dst_rows_cap, row_bytes);
        if (s != REGIONE_OK) return s;
        ps.p[i] = RowCopyPair{(const uint4*)srcs[i], (uint4*)dsts[i]};
    }
    if (idx_stride < dst_rows_cap) return REGIONE_INVALID_ARG;
    if (B == 0 || dst_rows_cap == 0) return REGIONE_OK;
    return launch_row_copy<true>(ps, n_tensors, idx, n, B, src_rows, idx_stride, dst_rows_cap, row_bytes,
                                 dev_status, stream);
}
