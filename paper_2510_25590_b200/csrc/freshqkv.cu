// Producer of the fresh Q / K / V rows of a region step: gather of the recomputed tokens' rows, per-head
// RMS normalisation of Q and K, rotary position embedding, in one pass over the rows.
//
// The paper takes the attention layer of the editors it accelerates as given and does not state these
// two operations; the editors apply them to Q and K of every attention layer.  What the method fixes
// is where a recomputed token sits: it keeps its position in the joint sequence (Sec. 4 "Region-Aware
// Generation": the region's tokens are gathered and later put back by spatial position), so the row
// index of the gather, idx[b, j], is also the position whose angles rotate the row -- the cached keys
// it meets in the attention were rotated at their own positions in the last full step.
//
//   y = x / sqrt(mean(x^2) + eps) * w           over the D elements of one row and head
//   (a, b) -> (a cos t - b sin t, a sin t + b cos t)   for the D/2 pairs of y; pair i = elements
//   (2i, 2i+1) (interleaved) or (i, i + D/2) (half), t = angle i of the row's position; the caller
//   passes cos and sin of the angles, [N_src, D/2] fp32, so any frequency scheme (several axes
//   included) fits.
//
// HBM-bound row pass: one block per gathered row, a lane owns 8 consecutive elements (16 bytes) of one
// head, the D/8 lanes of a head sit side by side in a warp (sum of squares and, in the half layout,
// the pair partner by shuffles).  Three Q / K loads per lane are in flight before the first is used,
// the V row (a plain copy) is loaded before them and stored after them, four blocks share an SM.  All
// arithmetic in fp32 (reciprocal square root by the hardware approximation, relative error 2^-22),
// one rounding to bf16 at the end.
#include "common.cuh"

namespace regione {

constexpr int kFreshThreads = 256;
constexpr int kFreshUnroll = 3;

__device__ __forceinline__ void unpack8(const uint4& w, float (&x)[8]) {
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}

template <int D, bool HALF>
__global__ void __launch_bounds__(kFreshThreads, 4)
fresh_qkv_kernel(const uint16_t* __restrict__ q_src, const uint16_t* __restrict__ k_src,
                 const uint16_t* __restrict__ v_src, const int32_t* __restrict__ idx,
                 const int32_t* __restrict__ n, int N_src, int cap, int H, int src_compact,
                 const uint16_t* __restrict__ q_weight, const uint16_t* __restrict__ k_weight, float eps,
                 const float* __restrict__ cos_t, const float* __restrict__ sin_t,
                 uint16_t* __restrict__ q_dst, uint16_t* __restrict__ k_dst, uint16_t* __restrict__ v_dst,
                 int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    constexpr int kLanesPerHead = D / 8;                // 16 or 8: divides the warp
    const int b = blockIdx.y, j = blockIdx.x;
    int live = n[b];
    if (live < 0 || live > cap) {
        if (threadIdx.x == 0 && j == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        live = live < 0 ? 0 : cap;
    }
    if (j >= live) return;
    const int row = idx[(size_t)b * cap + j];
    if (row < 0 || row >= N_src) {
        if (threadIdx.x == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        return;
    }
    const int lane = threadIdx.x & 31;
    const int g = lane & (kLanesPerHead - 1);           // this lane's place among the lanes of a head
    constexpr bool half = HALF;                        // pairs (i, i + D/2) instead of (2i, 2i+1)
    const bool upper = g >= kLanesPerHead / 2;          // half layout: this lane holds second elements of pairs

    // What does not depend on the head: the angles of this row's position that this lane's elements
    // use, and the lane's 8 weights of Q and of K.  Interleaved: elements 8g .. 8g+7 are pairs
    // 4g .. 4g+3; half: element e pairs with e +- D/2 under angle e mod D/2.
    constexpr int kAngles = HALF ? 8 : 4;               // angles this lane's 8 elements use
    float cs[kAngles], sn[kAngles];
    {
        const size_t at = (size_t)row * (D / 2) + (half ? (8 * g) % (D / 2) : 4 * g);
        const float4 c0 = *reinterpret_cast<const float4*>(cos_t + at);
        const float4 s0 = *reinterpret_cast<const float4*>(sin_t + at);
        cs[0] = c0.x; cs[1] = c0.y; cs[2] = c0.z; cs[3] = c0.w;
        sn[0] = s0.x; sn[1] = s0.y; sn[2] = s0.z; sn[3] = s0.w;
        if constexpr (HALF) {
            const float4 c1 = *reinterpret_cast<const float4*>(cos_t + at + 4);
            const float4 s1 = *reinterpret_cast<const float4*>(sin_t + at + 4);
            cs[4] = c1.x; cs[5] = c1.y; cs[6] = c1.z; cs[7] = c1.w;
            sn[4] = s1.x; sn[5] = s1.y; sn[6] = s1.z; sn[7] = s1.w;
            // a lane of first elements computes a cos - b sin, a lane of second elements b cos + a sin:
            // the sign goes into the sine once
            if (!upper) {
#pragma unroll
                for (int e = 0; e < 8; ++e) sn[e] = -sn[e];
            }
        }
    }
    // (weights stay packed, 4 registers per tensor, and are widened where they are used)
    uint4 wq = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u), wk = wq;      // bf16 ones
    if (q_weight != nullptr) wq = *reinterpret_cast<const uint4*>(q_weight + 8 * g);
    if (k_weight != nullptr) wk = *reinterpret_cast<const uint4*>(k_weight + 8 * g);

    // source rows: taken at the index (a gather from the whole sequence), or already gathered (row j)
    const size_t dst_off = ((size_t)b * cap + j) * H * D;
    const size_t src_off = src_compact ? dst_off : ((size_t)b * N_src + row) * H * D;
    const int per_tensor = H * kLanesPerHead, total = 2 * per_tensor;   // 16-byte pieces of Q, then of K
    // V is a plain copy; its loads are issued first and stored last, so that they are in flight while
    // the pieces of Q and K are worked on
    constexpr int kVDepth = 2;
    uint4 vv[kVDepth];
#pragma unroll
    for (int u = 0; u < kVDepth; ++u) {
        const int c = threadIdx.x + u * kFreshThreads;
        if (c < per_tensor) vv[u] = ld_stream128(v_src + src_off + (size_t)c * 8);
    }
    // whole warps walk the pieces so that every shuffle below has its 32 lanes
    for (int c0 = (threadIdx.x & ~31); c0 < total; c0 += kFreshUnroll * kFreshThreads) {
        uint4 w[kFreshUnroll];
#pragma unroll
        for (int u = 0; u < kFreshUnroll; ++u) {
            const int c = c0 + u * kFreshThreads + lane;
            w[u] = make_uint4(0u, 0u, 0u, 0u);
            if (c < total)
                w[u] = ld_stream128((c < per_tensor ? q_src : k_src) + src_off +
                                    (size_t)(c < per_tensor ? c : c - per_tensor) * 8);
        }
#pragma unroll
        for (int u = 0; u < kFreshUnroll; ++u) {
            const int c = c0 + u * kFreshThreads + lane;
            if (c0 + u * kFreshThreads >= total) break;                  // (uniform for the warp)
            const bool is_k = c >= per_tensor;
            float x[8];
            unpack8(w[u], x);
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(x[e], x[e], ss);
#pragma unroll
            for (int d = kLanesPerHead / 2; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
            const float r = rsqrtf(ss * (1.0f / D) + eps);
            float y[8], o[8];
            unpack8(is_k ? wk : wq, y);
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] *= x[e] * r;
            if constexpr (HALF) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float partner = __shfl_xor_sync(0xffffffffu, y[e], kLanesPerHead / 2);
                    o[e] = fmaf(partner, sn[e], y[e] * cs[e]);
                }
            } else {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    o[2 * t] = fmaf(-y[2 * t + 1], sn[t], y[2 * t] * cs[t]);
                    o[2 * t + 1] = fmaf(y[2 * t], sn[t], y[2 * t + 1] * cs[t]);
                }
            }
            if (c >= total) continue;
            uint4 out;
            out.x = pack_bf16x2(o[0], o[1]); out.y = pack_bf16x2(o[2], o[3]);
            out.z = pack_bf16x2(o[4], o[5]); out.w = pack_bf16x2(o[6], o[7]);
            *reinterpret_cast<uint4*>((is_k ? k_dst : q_dst) + dst_off + (size_t)(is_k ? c - per_tensor : c) * 8) = out;
        }
    }
#pragma unroll
    for (int u = 0; u < kVDepth; ++u) {
        const int c = threadIdx.x + u * kFreshThreads;
        if (c < per_tensor) *reinterpret_cast<uint4*>(v_dst + dst_off + (size_t)c * 8) = vv[u];
    }
    for (int c = threadIdx.x + kVDepth * kFreshThreads; c < per_tensor; c += kFreshThreads)   // more than 32 heads of 128
        *reinterpret_cast<uint4*>(v_dst + dst_off + (size_t)c * 8) = ld_stream128(v_src + src_off + (size_t)c * 8);
}

}  // namespace regione

using namespace regione;

extern "C" int regione_fresh_qkv(const regione_bf16* q_src, const regione_bf16* k_src,
                                 const regione_bf16* v_src, const int32_t* idx, const int32_t* n, int B,
                                 int N_src, int cap, int H, int D, int src_compact,
                                 const regione_bf16* q_weight, const regione_bf16* k_weight, float eps,
                                 const float* cos_table,
                                 const float* sin_table, int rope_layout, regione_bf16* q_dst,
                                 regione_bf16* k_dst, regione_bf16* v_dst, int32_t* dev_status,
                                 void* stream) {
    if (!q_src || !k_src || !v_src || !idx || !n || !cos_table || !sin_table || !q_dst || !k_dst || !v_dst)
        return REGIONE_INVALID_ARG;
    if (B < 0 || N_src < 1 || cap < 0 || H < 1 || !(eps >= 0.f)) return REGIONE_INVALID_ARG;
    if (rope_layout != REGIONE_ROPE_INTERLEAVED && rope_layout != REGIONE_ROPE_HALF) return REGIONE_INVALID_ARG;
    if (D != 64 && D != 128) return REGIONE_UNSUPPORTED;
    if (B > 65535) return REGIONE_UNSUPPORTED;
    if (!aligned16(q_src) || !aligned16(k_src) || !aligned16(v_src) || !aligned16(q_dst) || !aligned16(k_dst) ||
        !aligned16(v_dst) || !aligned16(cos_table) || !aligned16(sin_table) ||
        (q_weight && !aligned16(q_weight)) || (k_weight && !aligned16(k_weight)))
        return REGIONE_INVALID_ARG;
    if (B == 0 || cap == 0) return REGIONE_OK;
    const dim3 grid(cap, B), block(kFreshThreads);
    cudaStream_t st = (cudaStream_t)stream;
    const bool half = rope_layout == REGIONE_ROPE_HALF;
#define REGIONE_FRESH_LAUNCH(DD, HH)                                                                       \
    launch_overlapped(fresh_qkv_kernel<DD, HH>, grid, block, 0, st, q_src, k_src, v_src, idx, n, N_src, cap, H, \
                      src_compact, q_weight, k_weight, eps, cos_table, sin_table, q_dst, k_dst, v_dst, dev_status)
    const cudaError_t e = D == 128 ? (half ? REGIONE_FRESH_LAUNCH(128, true) : REGIONE_FRESH_LAUNCH(128, false))
                                   : (half ? REGIONE_FRESH_LAUNCH(64, true) : REGIONE_FRESH_LAUNCH(64, false));
#undef REGIONE_FRESH_LAUNCH
    return launch_status(e);
}
