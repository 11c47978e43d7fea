// 8-bit variant of the Region-Instruction KV cache (Sec. 4 "Stabilization Stage": K and V of every
// attention layer are kept from the last full step until the next forced one, i.e. the cache is
// resident for many steps and layers).  The paper keeps the cache in the model's own precision;
// this variant stores it as 8-bit floating point E4M3 (1 sign, 4 exponent, 3 mantissa bits, bias 7,
// largest finite value 448, no infinities) with one power-of-two scale per (row, head), which halves
// the bytes a cached layer occupies.  Before a region step's attention the cache is widened back to
// bf16 by a second kernel; because the scale is a power of two and E4M3 has 3 mantissa bits, the
// widened values are exactly the quantised ones (no second rounding), so the attention sees a cache
// whose every element is  round_to_E4M3(x / s) * s.
//
//   s = 2^k, k the smallest integer with amax / 2^k <= 448 (amax = largest magnitude of the D
//   elements of that row and head); written with frexp(amax) = m * 2^e, m in [0.5, 1):
//   k = e - 9 + (m > 0.875); k = 0 for amax = 0; k is kept >= -100.
//
// Both kernels are HBM-bound row passes: one block per kept row covers K and V of that row, a lane
// owns 8 consecutive elements (16 bytes of bf16, 8 bytes of codes), the D / 8 lanes of one head sit
// side by side in a warp and find the head's maximum by shuffles.
#include "common.cuh"

namespace regione {

constexpr int kQuantThreads = 256;
constexpr int kQuantUnroll = 3;

// Two fp32 -> two E4M3 codes (round to nearest even, saturating); `lo` lands in bits [7:0].
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Two E4M3 codes -> their two values (exact: every E4M3 value is a half-precision value); the code
// in bits [7:0] comes back in `.x`.  (0x7f / 0xff, the NaN codes, are never produced by the
// saturating conversion above.)
__device__ __forceinline__ float2 unpack_e4m3x2(uint32_t codes) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)codes));
    float2 r;
    asm("{.reg .b16 l, h; mov.b32 {l, h}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, h;}"
        : "=f"(r.x), "=f"(r.y) : "r"(h2));
    return r;
}

// k of the scale 2^k for a row-and-head maximum `amax` (>= 0, finite).
__device__ __forceinline__ int scale_exponent(float amax) {
    if (!(amax > 0.f)) return 0;
    int e;
    const float m = frexpf(amax, &e);
    return max(e - 9 + (m > 0.875f ? 1 : 0), -100);
}

// n_keep[b] clamped to the capacity; an out-of-range count is recorded once per request.
__device__ __forceinline__ int live_rows(const int32_t* n_keep, int b, int Nc_cap, int j, int32_t* dev_status) {
    const int live = n_keep[b];
    if (live >= 0 && live <= Nc_cap) return live;
    if (threadIdx.x == 0 && j == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
    return live < 0 ? 0 : Nc_cap;
}

template <int D>
__global__ void __launch_bounds__(kQuantThreads)
rikv_store_e4m3_kernel(const uint16_t* __restrict__ k_full, const uint16_t* __restrict__ v_full,
                       const int32_t* __restrict__ keep_rows, const int32_t* __restrict__ n_keep,
                       int N_full, int Nc_cap, int H, uint8_t* __restrict__ k_q, uint8_t* __restrict__ v_q,
                       float* __restrict__ k_scale, float* __restrict__ v_scale, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    constexpr int kLanesPerHead = D / 8;                // 16 or 8: divides the warp
    const int b = blockIdx.y, j = blockIdx.x;
    if (j >= live_rows(n_keep, b, Nc_cap, j, dev_status)) return;
    const int row = keep_rows[(size_t)b * Nc_cap + j];
    if (row < 0 || row >= N_full) {
        if (threadIdx.x == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        return;
    }
    const size_t src_off = ((size_t)b * N_full + row) * H * D, dst_row = (size_t)b * Nc_cap + j;
    const int per_tensor = H * kLanesPerHead, total = 2 * per_tensor;     // 16-byte pieces of K, then of V
    // whole warps walk the pieces so that every shuffle below has its 32 lanes; kQuantUnroll loads are
    // issued before the first is used (24 heads of 128 are one pass)
    for (int c0 = (threadIdx.x & ~31); c0 < total; c0 += kQuantUnroll * kQuantThreads) {
        uint4 w[kQuantUnroll];
#pragma unroll
        for (int u = 0; u < kQuantUnroll; ++u) {
            const int c = c0 + u * kQuantThreads + (threadIdx.x & 31);
            w[u] = make_uint4(0u, 0u, 0u, 0u);
            if (c < total)
                w[u] = *reinterpret_cast<const uint4*>((c >= per_tensor ? v_full : k_full) + src_off +
                                                       (size_t)(c >= per_tensor ? c - per_tensor : c) * 8);
        }
#pragma unroll
        for (int u = 0; u < kQuantUnroll; ++u) {
            const int c = c0 + u * kQuantThreads + (threadIdx.x & 31);
            const bool live = c < total;
            const int is_v = live && c >= per_tensor, piece = c - (is_v ? per_tensor : 0);
            const float x[8] = {bf16_lo(w[u].x), bf16_hi(w[u].x), bf16_lo(w[u].y), bf16_hi(w[u].y),
                                bf16_lo(w[u].z), bf16_hi(w[u].z), bf16_lo(w[u].w), bf16_hi(w[u].w)};
            float amax = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(x[e]));   // (a NaN element is ignored here)
#pragma unroll
            for (int d = kLanesPerHead / 2; d > 0; d >>= 1)
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
            amax = fminf(amax, 3.0e38f);                // an infinite element saturates at the largest code
            const int k = scale_exponent(amax);
            const float inv = __uint_as_float((uint32_t)(127 - k) << 23);  // 2^-k, exact
            if (!live) continue;
            uint2 q;
            q.x = pack_e4m3x2(x[0] * inv, x[1] * inv) | (pack_e4m3x2(x[2] * inv, x[3] * inv) << 16);
            q.y = pack_e4m3x2(x[4] * inv, x[5] * inv) | (pack_e4m3x2(x[6] * inv, x[7] * inv) << 16);
            *reinterpret_cast<uint2*>((is_v ? v_q : k_q) + dst_row * H * D + (size_t)piece * 8) = q;
            if (piece % kLanesPerHead == 0)
                (is_v ? v_scale : k_scale)[dst_row * H + piece / kLanesPerHead] =
                    __uint_as_float((uint32_t)(127 + k) << 23);
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kQuantThreads)
rikv_load_e4m3_kernel(const uint8_t* __restrict__ k_q, const uint8_t* __restrict__ v_q,
                      const float* __restrict__ k_scale, const float* __restrict__ v_scale,
                      const int32_t* __restrict__ n_keep, int Nc_cap, int H, uint16_t* __restrict__ k_cache,
                      uint16_t* __restrict__ v_cache, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    constexpr int kLanesPerHead = D / 8;
    const int b = blockIdx.y, j = blockIdx.x;
    if (j >= live_rows(n_keep, b, Nc_cap, j, dev_status)) return;
    const size_t dst_row = (size_t)b * Nc_cap + j;
    const int per_tensor = H * kLanesPerHead, total = 2 * per_tensor;
    for (int c = threadIdx.x; c < total; c += kQuantThreads) {
        const int is_v = c >= per_tensor, piece = c - (is_v ? per_tensor : 0);
        const uint2 q = *reinterpret_cast<const uint2*>((is_v ? v_q : k_q) + dst_row * H * D + (size_t)piece * 8);
        const float s = (is_v ? v_scale : k_scale)[dst_row * H + piece / kLanesPerHead];
        // (code value) * 2^k is exact in bf16: 4 significant bits, exponent well inside the range
        const float2 a = unpack_e4m3x2(q.x), c2 = unpack_e4m3x2(q.x >> 16);
        const float2 e = unpack_e4m3x2(q.y), g = unpack_e4m3x2(q.y >> 16);
        uint4 w;
        w.x = pack_bf16x2(a.x * s, a.y * s); w.y = pack_bf16x2(c2.x * s, c2.y * s);
        w.z = pack_bf16x2(e.x * s, e.y * s); w.w = pack_bf16x2(g.x * s, g.y * s);
        *reinterpret_cast<uint4*>((is_v ? v_cache : k_cache) + dst_row * H * D + (size_t)piece * 8) = w;
    }
}

}  // namespace regione

using namespace regione;

static int check_quant_args(const void* a, const void* b, const void* c, const void* d, const void* e,
                            const void* f, int B, int Nc_cap, int H, int D) {
    if (!a || !b || !c || !d || !e || !f) return REGIONE_INVALID_ARG;
    if (B < 0 || Nc_cap < 0 || H < 1) return REGIONE_INVALID_ARG;
    if (D != 64 && D != 128) return REGIONE_UNSUPPORTED;
    if (B > 65535 || Nc_cap > 0x7fffffff / 2) return REGIONE_UNSUPPORTED;
    return REGIONE_OK;
}

extern "C" int regione_rikv_store_e4m3(const regione_bf16* k_full, const regione_bf16* v_full,
                                       const int32_t* keep_rows, const int32_t* n_keep, int B, int N_full,
                                       int Nc_cap, int H, int D, uint8_t* k_q, uint8_t* v_q, float* k_scale,
                                       float* v_scale, int32_t* dev_status, void* stream) {
    int rc = check_quant_args(k_full, v_full, k_q, v_q, k_scale, v_scale, B, Nc_cap, H, D);
    if (rc != REGIONE_OK) return rc;
    if (!keep_rows || !n_keep || N_full < 0) return REGIONE_INVALID_ARG;
    if (!aligned16(k_full) || !aligned16(v_full) || !aligned16(k_q) || !aligned16(v_q)) return REGIONE_INVALID_ARG;
    if (B == 0 || Nc_cap == 0) return REGIONE_OK;
    const dim3 grid(Nc_cap, B);
    cudaError_t e = D == 128
        ? launch_overlapped(rikv_store_e4m3_kernel<128>, grid, dim3(kQuantThreads), 0, (cudaStream_t)stream,
                            k_full, v_full, keep_rows, n_keep, N_full, Nc_cap, H, k_q, v_q, k_scale, v_scale, dev_status)
        : launch_overlapped(rikv_store_e4m3_kernel<64>, grid, dim3(kQuantThreads), 0, (cudaStream_t)stream,
                            k_full, v_full, keep_rows, n_keep, N_full, Nc_cap, H, k_q, v_q, k_scale, v_scale, dev_status);
    return launch_status(e);
}

extern "C" int regione_rikv_load_e4m3(const uint8_t* k_q, const uint8_t* v_q, const float* k_scale,
                                      const float* v_scale, const int32_t* n_keep, int B, int Nc_cap, int H,
                                      int D, regione_bf16* k_cache, regione_bf16* v_cache,
                                      int32_t* dev_status, void* stream) {
    int rc = check_quant_args(k_q, v_q, k_scale, v_scale, k_cache, v_cache, B, Nc_cap, H, D);
    if (rc != REGIONE_OK) return rc;
    if (!n_keep) return REGIONE_INVALID_ARG;
    if (!aligned16(k_q) || !aligned16(v_q) || !aligned16(k_cache) || !aligned16(v_cache)) return REGIONE_INVALID_ARG;
    if (B == 0 || Nc_cap == 0) return REGIONE_OK;
    const dim3 grid(Nc_cap, B);
    cudaError_t e = D == 128
        ? launch_overlapped(rikv_load_e4m3_kernel<128>, grid, dim3(kQuantThreads), 0, (cudaStream_t)stream,
                            k_q, v_q, k_scale, v_scale, n_keep, Nc_cap, H, k_cache, v_cache, dev_status)
        : launch_overlapped(rikv_load_e4m3_kernel<64>, grid, dim3(kQuantThreads), 0, (cudaStream_t)stream,
                            k_q, v_q, k_scale, v_scale, n_keep, Nc_cap, H, k_cache, v_cache, dev_status);
    return launch_status(e);
}
