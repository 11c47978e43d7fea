// Adaptive Region Partition: one-step estimate, per-token score, threshold and
// ordered stream compaction in ONE launch (Sec. 4 "Adaptive Region Partition";
// Algorithm 1: X_hat_0 and E_index / U_index).
//
// Mapping.  A request's N tokens are split over a thread-block cluster of up to
// 8 CTAs (one cluster per request, gridDim = {cluster, B}).  Inside a CTA a
// warp owns 32 consecutive tokens at a time.  C/8 lanes (rounded up to a power
// of two, L) share a token: each lane reads one 16-byte chunk of x_t, v and ref
// (fully coalesced 128-bit loads), the partial sums are folded with xor
// shuffles, and a ballot turns the 32 decisions into one mask word kept in
// shared memory.  The ordered compaction is a popcount prefix sum over those
// words: warp scan -> CTA scan -> cluster scan through distributed shared
// memory, so no global scratch, no atomics and no spinning are needed and the
// index lists come out ascending and deterministic.
//
// A few very long requests (at least 32768 tokens each, fewer cluster blocks than SMs) would leave
// most of the GPU idle in that mapping.  For them the decisions are taken by a launch of their own
// (partition_score_kernel, grid over the tokens, writes the mask bytes) and the same compaction
// kernel follows in a form that reads the mask bytes back instead of scoring (FROM_MASK).
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace regione {

constexpr int kPartMaxThreads = 512;         // block size grows with the tokens per CTA
constexpr int kPartMaxWords = 4096;          // 131072 tokens per CTA
constexpr int kPartMaxCluster = 8;
constexpr int kPartTwoLaunchTokens = 32768;  // requests at least this long may take the two-launch form
constexpr int kPartBlocksPerGpu = 148;       // ... when their clusters are fewer blocks than a B200 has SMs

// Exclusive prefix sum of popcounts of `bits[0..nwords)` into `prefix`; returns the total.
// Every thread of the CTA must call it.  `warp_tot` is shared scratch of 33 ints.
__device__ int block_popc_scan(const uint32_t* bits, int* prefix, int nwords, int* warp_tot) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = blockDim.x >> 5;
    int carry = 0;
    for (int base = 0; base < nwords; base += blockDim.x) {
        const int w = base + tid;
        const int c = (w < nwords) ? __popc(bits[w]) : 0;
        int incl = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int tv = (lane < nwarps) ? warp_tot[lane] : 0;
            int ti = tv;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int y = __shfl_up_sync(0xffffffffu, ti, d);
                if (lane >= d) ti += y;
            }
            if (lane < nwarps) warp_tot[lane] = ti - tv;      // exclusive warp offsets
            if (lane == 31) warp_tot[32] = ti;                // chunk total
        }
        __syncthreads();
        if (w < nwords) prefix[w] = carry + warp_tot[warp] + (incl - c);
        carry += warp_tot[32];
        __syncthreads();
    }
    return carry;
}

// Optional second output of the partition: the joint-sequence row lists of one region-attention
// layer (what regione_region_rows composes from the index lists), written in the same launch.
struct RowLists {
    int32_t* query_rows;     // nullptr: not requested
    int32_t* n_query;
    int32_t* cache_rows;
    int32_t* n_cache;
    int n_text, n_ref, membership, q_cap, c_cap;
};

// Writes mask / slot / edit_idx / keep_idx for tokens [start, start+ntok) of one request from
// the mask words in shared memory.  edit_base / keep_base: entries preceding this CTA's share.
// With row lists requested, an edited token n also becomes query row n_text + n and a kept token
// cache row n_text + n, at the positions `q_off` / `c_off` further into this request's lists.
__device__ void emit_indices(const uint32_t* bits, const int* prefix, int start, int ntok, int N,
                             int edit_base, int keep_base, uint8_t* mask, int32_t* edit_idx,
                             int32_t* keep_idx, int32_t* slot, const RowLists& rl,
                             int32_t* query_rows, int32_t* cache_rows, int q_off, int c_off) {
    for (int tl = threadIdx.x; tl < ntok; tl += blockDim.x) {
        const int n = start + tl;
        if (n >= N) break;
        const uint32_t word = bits[tl >> 5];
        const int i = tl & 31;
        const int er = prefix[tl >> 5] + __popc(word & ((1u << i) - 1u));
        const bool edited = (word >> i) & 1u;
        if (mask != nullptr) mask[n] = edited ? 1 : 0;
        if (edited) {
            slot[n] = edit_base + er;
            edit_idx[edit_base + er] = n;
            if (query_rows != nullptr && q_off + edit_base + er < rl.q_cap)
                query_rows[q_off + edit_base + er] = rl.n_text + n;
        } else {
            slot[n] = -1;
            keep_idx[keep_base + (tl - er)] = n;
            if (cache_rows != nullptr && c_off + keep_base + (tl - er) < rl.c_cap)
                cache_rows[c_off + keep_base + (tl - er)] = rl.n_text + n;
        }
    }
}

// Adds one 16-byte chunk (8 channels) of a token to its partial sums: x0_hat = x_t - t v, then
// cosine terms (dot, |x0_hat|^2, |ref|^2) or the squared distance.
__device__ __forceinline__ void accumulate_chunk(uint4 xv, uint4 vv, uint4 rv, float t, int metric,
                                                 float& a0, float& a1, float& a2) {
    const uint32_t xs[4] = {xv.x, xv.y, xv.z, xv.w};
    const uint32_t vs[4] = {vv.x, vv.y, vv.z, vv.w};
    const uint32_t rs[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float h0 = fmaf(-t, bf16_lo(vs[k]), bf16_lo(xs[k]));
        const float h1 = fmaf(-t, bf16_hi(vs[k]), bf16_hi(xs[k]));
        const float r0 = bf16_lo(rs[k]), r1 = bf16_hi(rs[k]);
        if (metric == REGIONE_METRIC_COSINE) {
            a0 = fmaf(h0, r0, a0); a0 = fmaf(h1, r1, a0);
            a1 = fmaf(h0, h0, a1); a1 = fmaf(h1, h1, a1);
            a2 = fmaf(r0, r0, a2); a2 = fmaf(r1, r1, a2);
        } else {
            const float d0 = h0 - r0, d1 = h1 - r1;
            a0 = fmaf(d0, d0, a0); a0 = fmaf(d1, d1, a0);
        }
    }
}

// Decisions of the 32 tokens n0 .. n0+31 of one request as a mask word (bit i = token n0 + i is
// edited).  Called by whole warps.  L lanes share a token.
template <int L>
__device__ __forceinline__ uint32_t score_word(const uint16_t* __restrict__ x_t, const uint16_t* __restrict__ v,
                                               const uint16_t* __restrict__ ref, size_t req, int n0, int N, int C,
                                               float t, int metric, float threshold, float* __restrict__ score) {
    const int lane = threadIdx.x & 31;
    constexpr int TPI = 32 / L;                 // tokens per sub-iteration
    const int sub = lane % L;                   // chunk lane inside the token group
    const int chunks = C >> 3;                  // 16-byte chunks per token row
    uint32_t mybit = 0;
    // The loads of up to 4 groups of tokens are issued before any of them is reduced, so a
    // warp keeps several kilobytes in flight (one 16-byte chunk per lane and tensor and group).
    constexpr int G = L < 4 ? L : 4;
#pragma unroll
    for (int s0 = 0; s0 < L; s0 += G) {
        uint4 xv[G], vv[G], rv[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int tok = n0 + (s0 + g) * TPI + lane / L;
            xv[g] = vv[g] = rv[g] = make_uint4(0, 0, 0, 0);
            if (tok < N && sub < chunks) {
                const size_t at = (req + tok) * (size_t)C + (sub << 3);
                xv[g] = ld_stream128(x_t + at);
                vv[g] = ld_stream128(v + at);
                rv[g] = ld_stream128(ref + at);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int s = s0 + g;
            const int tok = n0 + s * TPI + lane / L;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f;  // cosine: dot, |x0|^2, |ref|^2 ; l2: a0 only
            accumulate_chunk(xv[g], vv[g], rv[g], t, metric, a0, a1, a2);
            if (L == 32 && tok < N) {            // rows wider than 256 channels: further chunks
                const size_t row = (req + tok) * (size_t)C;
                for (int ch = sub + 32; ch < chunks; ch += 32)
                    accumulate_chunk(ld_stream128(x_t + row + (ch << 3)),
                                     ld_stream128(v + row + (ch << 3)),
                                     ld_stream128(ref + row + (ch << 3)), t, metric, a0, a1, a2);
            }
#pragma unroll
            for (int d = 1; d < L; d <<= 1) {
                a0 += __shfl_xor_sync(0xffffffffu, a0, d);
                a1 += __shfl_xor_sync(0xffffffffu, a1, d);
                a2 += __shfl_xor_sync(0xffffffffu, a2, d);
            }
            float sc;
            bool edited;
            if (metric == REGIONE_METRIC_COSINE) {
                sc = a0 / fmaxf(sqrtf(a1) * sqrtf(a2), 1e-12f);
                edited = sc <= threshold;
            } else {
                sc = sqrtf(a0);
                edited = sc > threshold;
            }
            const bool leader = (sub == 0) && (tok < N);
            if (leader && score != nullptr) score[req + tok] = sc;
            const uint32_t ballot = __ballot_sync(0xffffffffu, leader && edited);
            if (lane / TPI == s) mybit = (ballot >> ((lane % TPI) * L)) & 1u;
        }
    }
    return __ballot_sync(0xffffffffu, mybit != 0);
}

// Large requests, first of two launches: the decisions alone, over a grid that does not depend on the
// request boundaries (blockIdx.y = request, the blocks of a request stride over its mask words).  The
// mask bytes it writes are what the compaction launch behind it reads.
template <int L>
__global__ void __launch_bounds__(256)
partition_score_kernel(const uint16_t* __restrict__ x_t, const uint16_t* __restrict__ v,
                       const uint16_t* __restrict__ ref, int N, int C, const PerRequestF tv, int b0, int metric,
                       float threshold, uint8_t* __restrict__ mask, float* __restrict__ score) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int b = b0 + blockIdx.y;
    const float t = tv.v[blockIdx.y];
    if (t != t) return;                          // NaN: this request sits the call out
    const size_t req = (size_t)b * N;
    const int lane = threadIdx.x & 31;
    const int nwords = (N + 31) >> 5;
    const int warps = (blockDim.x >> 5) * gridDim.x;
    for (int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); w < nwords; w += warps) {
        const uint32_t word = score_word<L>(x_t, v, ref, req, w << 5, N, C, t, metric, threshold, score);
        const int tok = (w << 5) + lane;
        if (tok < N) mask[req + tok] = (word >> lane) & 1u;
    }
}

// FROM_MASK: the decisions were taken by partition_score_kernel; this launch reads the mask bytes back
// (x_t, v, ref are not touched) and does the ordered compaction only.
template <int L, bool FROM_MASK>
__global__ void __launch_bounds__(kPartMaxThreads)
partition_kernel(const uint16_t* __restrict__ x_t, const uint16_t* __restrict__ v,
                 const uint16_t* __restrict__ ref, int N, int C, int share, const PerRequestF tv,
                 int b0, int metric, float threshold, uint8_t* __restrict__ mask, int32_t* __restrict__ edit_idx,
                 int32_t* __restrict__ keep_idx, int32_t* __restrict__ slot,
                 int32_t* __restrict__ n_edit, float* __restrict__ score, const RowLists rl,
                 int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    extern __shared__ uint32_t smem_u32[];
    const int nwords = share >> 5;
    uint32_t* bits = smem_u32;
    int* prefix = reinterpret_cast<int*>(smem_u32 + nwords);
    __shared__ int warp_tot[33];
    __shared__ int cta_count;

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = cluster.block_rank();
    const int csize = cluster.num_blocks();
    const int b = b0 + blockIdx.y;               // this launch covers requests b0 .. b0 + gridDim.y
    const float t = tv.v[blockIdx.y];            // the request's own sampler time
    if (t != t) return;                          // NaN: this request sits the call out (whole cluster)
    const int start = rank * share;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t req = (size_t)b * N;

    // ---- phase 1: score + decision, one mask word per 32 tokens -------------------------
    if constexpr (FROM_MASK) {
        // a thread packs the 32 mask bytes of one word: two 16-byte loads where the word is whole and
        // aligned, byte loads at a ragged end or an odd request offset
        for (int w = threadIdx.x; w < nwords; w += blockDim.x) {
            const int n0 = start + (w << 5);
            const uint8_t* src = mask + req + n0;
            uint32_t word = 0;
            if (n0 + 32 <= N && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
                const uint4 lo = *reinterpret_cast<const uint4*>(src), hi = *reinterpret_cast<const uint4*>(src + 16);
                const uint32_t x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)      // bytes of 0 / 1 -> 4 bits: each byte's bit lands on 21 .. 24
                    word |= (((x[i] & 0x01010101u) * 0x00204081u >> 21) & 0xFu) << (4 * i);
            } else {
                for (int i = 0; i < 32 && n0 + i < N; ++i) word |= (src[i] != 0 ? 1u : 0u) << i;
            }
            bits[w] = word;
        }
    } else {
        const int nwarps = blockDim.x >> 5;
        for (int w = warp; w < nwords; w += nwarps) {
            const uint32_t word = score_word<L>(x_t, v, ref, req, start + (w << 5), N, C, t, metric, threshold, score);
            if (lane == 0) bits[w] = word;
        }
    }
    __syncthreads();

    // ---- phase 2: CTA scan, then cluster scan through distributed shared memory ---------
    const int total = block_popc_scan(bits, prefix, nwords, warp_tot);
    if (threadIdx.x == 0) cta_count = total;
    cluster.sync();
    int edit_base = 0;
    for (int r = 0; r < rank; ++r) edit_base += *cluster.map_shared_rank(&cta_count, r);
    const int keep_base = start - edit_base;     // every token before `start` exists (start <= N)

    // ---- phase 3: coalesced per-token writes --------------------------------------------
    const bool lists = rl.query_rows != nullptr;
    const int q_text = (rl.membership == REGIONE_ROWS_PAPER) ? rl.n_text : 0;     // text rows are queries
    const int c_text = (rl.membership == REGIONE_ROWS_PAPER) ? 0 : rl.n_text;     // ... or cached
    int32_t* const q_rows = lists ? rl.query_rows + (size_t)b * rl.q_cap : nullptr;
    int32_t* const c_rows = lists ? rl.cache_rows + (size_t)b * rl.c_cap : nullptr;
    if (start < N) {
        emit_indices(bits, prefix, start, share, N, edit_base, keep_base, FROM_MASK ? nullptr : mask + req,
                     edit_idx + req, keep_idx + req, slot + req, rl, q_rows, c_rows, q_text, c_text);
    }
    if (rank == csize - 1 && threadIdx.x == 0) n_edit[b] = edit_base + total;
    if (lists) {
        // rows that do not depend on the mask: the text rows and the reference rows, spread over
        // the cluster's threads; the request's totals come from every rank's count
        int ne_all = 0;
        for (int r = 0; r < csize; ++r) ne_all += *cluster.map_shared_rank(&cta_count, r);
        const int nu_all = N - ne_all;
        const int stride = csize * blockDim.x;
        for (int i = rank * blockDim.x + threadIdx.x; i < rl.n_text; i += stride) {
            if (q_text > 0) { if (i < rl.q_cap) q_rows[i] = i; }
            else if (i < rl.c_cap) c_rows[i] = i;
        }
        for (int i = rank * blockDim.x + threadIdx.x; i < rl.n_ref; i += stride) {
            const int at = c_text + nu_all + i;
            if (at < rl.c_cap) c_rows[at] = rl.n_text + N + i;
        }
        if (rank == csize - 1 && threadIdx.x == 0) {
            const int nq = q_text + ne_all, nc = c_text + nu_all + rl.n_ref;
            if (nq > rl.q_cap || nc > rl.c_cap) record_status(dev_status, REGIONE_DEV_BOUNDS);
            rl.n_query[b] = min(nq, rl.q_cap);
            rl.n_cache[b] = min(nc, rl.c_cap);
        }
    }
    cluster.sync();                              // peers may still be reading cta_count
}

// ---- morphological opening + closing, then compaction (one CTA per request) -------------
constexpr int kMorphThreads = 1024;
constexpr int kMorphMaxTokens = 16384;

template <bool ERODE>
__device__ void morph3x3(const uint8_t* in, uint8_t* out, int rows, int cols) {
    for (int p = threadIdx.x; p < rows * cols; p += blockDim.x) {
        const int r = p / cols, c = p - r * cols;
        int acc = ERODE ? 1 : 0;
#pragma unroll
        for (int dr = -1; dr <= 1; ++dr)
#pragma unroll
            for (int dc = -1; dc <= 1; ++dc) {
                const int rr = r + dr, cc = c + dc;
                if (rr >= 0 && rr < rows && cc >= 0 && cc < cols) {
                    const int m = in[rr * cols + cc];
                    acc = ERODE ? (acc & m) : (acc | m);
                }
            }
        out[p] = (uint8_t)acc;
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kMorphThreads)
mask_open_close_kernel(const uint8_t* __restrict__ mask_in, int rows, int cols,
                       uint8_t* __restrict__ mask_out, int32_t* __restrict__ edit_idx,
                       int32_t* __restrict__ keep_idx, int32_t* __restrict__ slot,
                       int32_t* __restrict__ n_edit) {
    grid_dependency_wait();
    grid_launch_dependents();
    __shared__ uint8_t bufA[kMorphMaxTokens];
    __shared__ uint8_t bufB[kMorphMaxTokens];
    __shared__ uint32_t bits[kMorphMaxTokens / 32];
    __shared__ int prefix[kMorphMaxTokens / 32];
    __shared__ int warp_tot[33];
    const int N = rows * cols;
    const int b = blockIdx.x;
    const size_t req = (size_t)b * N;
    for (int p = threadIdx.x; p < N; p += blockDim.x) bufA[p] = mask_in[req + p] ? 1 : 0;
    __syncthreads();
    morph3x3<true>(bufA, bufB, rows, cols);      // opening = erode, dilate
    morph3x3<false>(bufB, bufA, rows, cols);
    morph3x3<false>(bufA, bufB, rows, cols);     // closing = dilate, erode
    morph3x3<true>(bufB, bufA, rows, cols);
    const int nwords = (N + 31) >> 5;
    const int lane = threadIdx.x & 31;
    for (int base = 0; base < nwords * 32; base += blockDim.x) {
        const int p = base + threadIdx.x;
        const uint32_t word = __ballot_sync(0xffffffffu, p < N && bufA[p] != 0);
        if (lane == 0 && (p >> 5) < nwords) bits[p >> 5] = word;
    }
    __syncthreads();
    const int total = block_popc_scan(bits, prefix, nwords, warp_tot);
    const RowLists none = {};
    emit_indices(bits, prefix, 0, nwords * 32, N, 0, 0, mask_out + req, edit_idx + req,
                 keep_idx + req, slot + req, none, nullptr, nullptr, 0, 0);
    if (threadIdx.x == 0) n_edit[b] = total;
}

// ---- joint-sequence row lists ---------------------------------------------------------------
__global__ void region_rows_kernel(const int32_t* __restrict__ edit_idx,
                                   const int32_t* __restrict__ keep_idx,
                                   const int32_t* __restrict__ n_edit, int N, int n_text, int n_ref,
                                   int membership, int32_t* __restrict__ query_rows,
                                   int32_t* __restrict__ n_query, int q_cap,
                                   int32_t* __restrict__ cache_rows, int32_t* __restrict__ n_cache,
                                   int c_cap, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int b = blockIdx.y;
    int ne = n_edit[b];
    if (ne < 0 || ne > N) {
        record_status(dev_status, REGIONE_DEV_BOUNDS);
        ne = max(0, min(ne, N));
    }
    const int nu = N - ne;
    const int q_text = (membership == REGIONE_ROWS_PAPER) ? n_text : 0;
    const int c_text = (membership == REGIONE_ROWS_PAPER) ? 0 : n_text;
    const int nq = q_text + ne;
    const int nc = c_text + nu + n_ref;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        if (nq > q_cap || nc > c_cap) record_status(dev_status, REGIONE_DEV_BOUNDS);
        n_query[b] = min(nq, q_cap);
        n_cache[b] = min(nc, c_cap);
    }
    if (i < nq && i < q_cap) {
        query_rows[(size_t)b * q_cap + i] =
            (i < q_text) ? i : n_text + edit_idx[(size_t)b * N + (i - q_text)];
    }
    if (i < nc && i < c_cap) {
        int r;
        if (i < c_text) r = i;
        else if (i < c_text + nu) r = n_text + keep_idx[(size_t)b * N + (i - c_text)];
        else r = n_text + N + (i - c_text - nu);
        cache_rows[(size_t)b * c_cap + i] = r;
    }
}

}  // namespace regione

using namespace regione;

template <int L, bool FROM_MASK = false>
static cudaError_t launch_partition(int csize, int B, int share, cudaStream_t st,
                                    const uint16_t* x_t, const uint16_t* v, const uint16_t* ref,
                                    int N, int C, const PerRequestF& tv, int b0, int metric,
                                    float thr, uint8_t* mask,
                                    int32_t* edit_idx, int32_t* keep_idx, int32_t* slot,
                                    int32_t* n_edit, float* score, const RowLists& rl,
                                    int32_t* dev_status) {
    cudaLaunchConfig_t cfg = {};
    // enough warps per CTA to keep the loads of a large share in flight (a cluster is at most 8
    // CTAs, so a long request cannot get its memory parallelism from the grid); 512 threads let
    // two CTAs share an SM, which measured faster than one CTA of 1024
    const int threads = share >= 2048 ? 512 : 256;
    cfg.gridDim = dim3(csize, B, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)(share >> 5) * 8;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see grid_dependency_wait
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, partition_kernel<L, FROM_MASK>, x_t, v, ref, N, C, share, tv, b0, metric,
                              thr, mask, edit_idx, keep_idx, slot, n_edit, score, rl, dev_status);
}

static int partition_impl(const regione_bf16* x_t, const regione_bf16* v, const regione_bf16* ref,
                          int B, int N, int C, const float* t, int metric, float threshold, uint8_t* mask,
                          int32_t* edit_idx, int32_t* keep_idx, int32_t* slot, int32_t* n_edit,
                          float* score, const RowLists& rl, int32_t* dev_status, void* stream) {
    if (!x_t || !v || !ref || !mask || !edit_idx || !keep_idx || !slot || !n_edit)
        return REGIONE_INVALID_ARG;
    if (B < 0 || N < 1 || C < 1 || (B > 0 && !t)) return REGIONE_INVALID_ARG;
    if (!aligned16(x_t) || !aligned16(v) || !aligned16(ref)) return REGIONE_INVALID_ARG;
    if (metric != REGIONE_METRIC_COSINE && metric != REGIONE_METRIC_L2) return REGIONE_INVALID_ARG;
    if ((C & 7) != 0 || C > 4096 || B > 65535) return REGIONE_UNSUPPORTED;
    if (N > kPartMaxCluster * kPartMaxWords * 32) return REGIONE_UNSUPPORTED;
    if (B == 0) return REGIONE_OK;
    int csize = (N + 511) / 512;
    if (csize > kPartMaxCluster) csize = kPartMaxCluster;
    int share = (N + csize - 1) / csize;
    share = (share + 31) & ~31;
    int L = 1;
    while (L < 32 && L * 8 < C) L <<= 1;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaSuccess;
    // the per-request times travel by value, kReqChunk requests per launch
    for (int b0 = 0; b0 < B && e == cudaSuccess; b0 += kReqChunk) {
        const int nb = B - b0 < kReqChunk ? B - b0 : kReqChunk;
        PerRequestF tv;
        for (int i = 0; i < nb; ++i) tv.v[i] = t[b0 + i];
        // Few long requests: a cluster is at most 8 blocks per request, so fewer than one block per SM
        // would read the latents (measured, 220 MB of latents: 16 requests of 131072 tokens 73 us, 2 of
        // 1048576 369 us, against 48 us for 32 of 65536).  Then the decisions go to a launch of their own
        // whose grid follows the tokens, and the compaction launch behind it reads the mask bytes back
        // (56 us and 122 us on the same instances; with a block per SM or more the single launch is as
        // fast or faster and stays).
        const bool two_launches = N >= kPartTwoLaunchTokens && (long long)nb * csize <= kPartBlocksPerGpu;
#define REGIONE_PART_CASE(LL)                                                                   \
    case LL:                                                                                    \
        if (two_launches) {                                                                     \
            const int warps_per_block = 8, words_per_warp = 4;                                  \
            const int nwords = (N + 31) / 32;                                                   \
            const dim3 sgrid((nwords + warps_per_block * words_per_warp - 1) /                  \
                             (warps_per_block * words_per_warp), nb);                           \
            e = launch_overlapped(partition_score_kernel<LL>, sgrid, dim3(256), 0, st, x_t, v,  \
                                  ref, N, C, tv, b0, metric, threshold, mask, score);           \
            if (e == cudaSuccess)                                                               \
                e = launch_partition<1, true>(csize, nb, share, st, x_t, v, ref, N, C, tv, b0,  \
                                              metric, threshold, mask, edit_idx, keep_idx,      \
                                              slot, n_edit, nullptr, rl, dev_status);           \
        } else {                                                                                \
            e = launch_partition<LL>(csize, nb, share, st, x_t, v, ref, N, C, tv, b0, metric,   \
                                     threshold, mask, edit_idx, keep_idx, slot, n_edit, score,  \
                                     rl, dev_status);                                           \
        }                                                                                       \
        break;
        switch (L) {
            REGIONE_PART_CASE(1)
            REGIONE_PART_CASE(2)
            REGIONE_PART_CASE(4)
            REGIONE_PART_CASE(8)
            REGIONE_PART_CASE(16)
            default:
            REGIONE_PART_CASE(32)
        }
    }
#undef REGIONE_PART_CASE
    return launch_status(e);
}

extern "C" int regione_partition(const regione_bf16* x_t, const regione_bf16* v,
                                 const regione_bf16* ref, int B, int N, int C, const float* t,
                                 int metric, float threshold, uint8_t* mask, int32_t* edit_idx,
                                 int32_t* keep_idx, int32_t* slot, int32_t* n_edit, float* score,
                                 int32_t* dev_status, void* stream) {
    RowLists none = {};
    return partition_impl(x_t, v, ref, B, N, C, t, metric, threshold, mask, edit_idx, keep_idx, slot,
                          n_edit, score, none, dev_status, stream);
}

extern "C" int regione_partition_rows(const regione_bf16* x_t, const regione_bf16* v,
                                      const regione_bf16* ref, int B, int N, int C, const float* t,
                                      int metric, float threshold, uint8_t* mask, int32_t* edit_idx,
                                      int32_t* keep_idx, int32_t* slot, int32_t* n_edit, float* score,
                                      int n_text, int n_ref, int membership, int32_t* query_rows,
                                      int32_t* n_query, int q_cap, int32_t* cache_rows,
                                      int32_t* n_cache, int c_cap, int32_t* dev_status, void* stream) {
    if (!query_rows || !n_query || !cache_rows || !n_cache) return REGIONE_INVALID_ARG;
    if (n_text < 0 || n_ref < 0 || q_cap < 0 || c_cap < 0) return REGIONE_INVALID_ARG;
    if (membership != REGIONE_ROWS_EDITED_QUERIES && membership != REGIONE_ROWS_PAPER)
        return REGIONE_INVALID_ARG;
    RowLists rl;
    rl.query_rows = query_rows; rl.n_query = n_query; rl.cache_rows = cache_rows; rl.n_cache = n_cache;
    rl.n_text = n_text; rl.n_ref = n_ref; rl.membership = membership; rl.q_cap = q_cap; rl.c_cap = c_cap;
    return partition_impl(x_t, v, ref, B, N, C, t, metric, threshold, mask, edit_idx, keep_idx, slot,
                          n_edit, score, rl, dev_status, stream);
}

extern "C" int regione_mask_open_close(const uint8_t* mask_in, int B, int rows, int cols,
                                       uint8_t* mask_out, int32_t* edit_idx, int32_t* keep_idx,
                                       int32_t* slot, int32_t* n_edit, int32_t* dev_status,
                                       void* stream) {
    (void)dev_status;      // no count or index input exists that could be out of range on the device
    if (!mask_in || !mask_out || !edit_idx || !keep_idx || !slot || !n_edit)
        return REGIONE_INVALID_ARG;
    if (B < 0 || rows < 1 || cols < 1 || mask_in == mask_out) return REGIONE_INVALID_ARG;
    if ((int64_t)rows * cols > kMorphMaxTokens) return REGIONE_UNSUPPORTED;
    if (B == 0) return REGIONE_OK;
    return launch_status(launch_overlapped(mask_open_close_kernel, dim3(B), dim3(kMorphThreads), 0,
                                           (cudaStream_t)stream, mask_in, rows, cols, mask_out,
                                           edit_idx, keep_idx, slot, n_edit));
}

extern "C" int regione_region_rows(const int32_t* edit_idx, const int32_t* keep_idx,
                                   const int32_t* n_edit, int B, int N, int n_text, int n_ref,
                                   int membership, int32_t* query_rows, int32_t* n_query, int q_cap,
                                   int32_t* cache_rows, int32_t* n_cache, int c_cap,
                                   int32_t* dev_status, void* stream) {
    if (!edit_idx || !keep_idx || !n_edit || !query_rows || !n_query || !cache_rows || !n_cache)
        return REGIONE_INVALID_ARG;
    if (B < 0 || N < 1 || n_text < 0 || n_ref < 0 || q_cap < 1 || c_cap < 1)
        return REGIONE_INVALID_ARG;
    if (membership != REGIONE_ROWS_EDITED_QUERIES && membership != REGIONE_ROWS_PAPER)
        return REGIONE_INVALID_ARG;
    if (B > 65535) return REGIONE_UNSUPPORTED;
    if (B == 0) return REGIONE_OK;
    const int span = (q_cap > c_cap ? q_cap : c_cap);
    dim3 grid((span + 255) / 256, B);
    return launch_status(launch_overlapped(region_rows_kernel, grid, dim3(256), 0,
                                           (cudaStream_t)stream, edit_idx, keep_idx, n_edit, N,
                                           n_text, n_ref, membership, query_rows, n_query, q_cap,
                                           cache_rows, n_cache, c_cap, dev_status));
}
