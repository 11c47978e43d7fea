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
// Both kernels are HBM-bound row passes: one warp per (kept row, head), a lane owns D / 32
// consecutive elements.
#include "common.cuh"

namespace regione {

constexpr int kQuantWarps = 8;

// Two fp32 -> two E4M3 codes (round to nearest even, saturating); `lo` lands in bits [7:0].
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// The value of an E4M3 code, written out from the format: sign, 4-bit exponent (bias 7), 3-bit
// mantissa; exponent 0 is subnormal (m / 8 * 2^-6).  (0x7f / 0xff, the NaN codes, are never produced
// by the saturating conversion above.)
__device__ __forceinline__ float e4m3_value(uint32_t code) {
    const uint32_t e = (code >> 3) & 15u, m = code & 7u;
    const float mag = e == 0 ? (float)m * 0.001953125f                          // m * 2^-9
                             : __uint_as_float(((e + 120u) << 23) | (m << 20)); // (1 + m/8) * 2^(e-7)
    return (code & 0x80u) ? -mag : mag;
}

// k of the scale 2^k for a row-and-head maximum `amax` (>= 0, finite).
__device__ __forceinline__ int scale_exponent(float amax) {
    if (!(amax > 0.f)) return 0;
    int e;
    const float m = frexpf(amax, &e);
    return max(e - 9 + (m > 0.875f ? 1 : 0), -100);
}

template <int D>
__global__ void __launch_bounds__(kQuantWarps * 32)
rikv_store_e4m3_kernel(const uint16_t* __restrict__ k_full, const uint16_t* __restrict__ v_full,
                       const int32_t* __restrict__ keep_rows, const int32_t* __restrict__ n_keep,
                       int N_full, int Nc_cap, int H, uint8_t* __restrict__ k_q, uint8_t* __restrict__ v_q,
                       float* __restrict__ k_scale, float* __restrict__ v_scale, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    constexpr int E = D / 32;                           // elements per lane: 4 or 2
    const int b = blockIdx.y, j = blockIdx.x, is_v = blockIdx.z;
    int live = n_keep[b];
    if (live < 0 || live > Nc_cap) {
        if (threadIdx.x == 0 && j == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        live = live < 0 ? 0 : Nc_cap;
    }
    if (j >= live) return;
    const int row = keep_rows[(size_t)b * Nc_cap + j];
    if (row < 0 || row >= N_full) {
        if (threadIdx.x == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        return;
    }
    const uint16_t* src = (is_v ? v_full : k_full) + ((size_t)b * N_full + row) * H * D;
    uint8_t* dst = (is_v ? v_q : k_q) + ((size_t)b * Nc_cap + j) * H * D;
    float* sc = (is_v ? v_scale : k_scale) + ((size_t)b * Nc_cap + j) * H;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int h = warp; h < H; h += kQuantWarps) {
        float x[E];
        if constexpr (E == 4) {
            const uint2 w = *reinterpret_cast<const uint2*>(src + (size_t)h * D + lane * 4);
            x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
        } else {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(src + (size_t)h * D + lane * 2);
            x[0] = bf16_lo(w); x[1] = bf16_hi(w);
        }
        float amax = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) amax = fmaxf(amax, fabsf(x[e]));     // (a NaN element is ignored here)
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
        amax = fminf(amax, 3.0e38f);                    // an infinite element saturates at the largest code
        const int k = scale_exponent(amax);
        const float inv = __uint_as_float((uint32_t)(127 - k) << 23);   // 2^-k, exact
        if constexpr (E == 4) {
            const uint32_t q = pack_e4m3x2(x[0] * inv, x[1] * inv) | (pack_e4m3x2(x[2] * inv, x[3] * inv) << 16);
            *reinterpret_cast<uint32_t*>(dst + (size_t)h * D + lane * 4) = q;
        } else {
            *reinterpret_cast<uint16_t*>(dst + (size_t)h * D + lane * 2) = (uint16_t)pack_e4m3x2(x[0] * inv, x[1] * inv);
        }
        if (lane == 0) sc[h] = __uint_as_float((uint32_t)(127 + k) << 23);   // 2^k
    }
}

template <int D>
__global__ void __launch_bounds__(kQuantWarps * 32)
rikv_load_e4m3_kernel(const uint8_t* __restrict__ k_q, const uint8_t* __restrict__ v_q,
                      const float* __restrict__ k_scale, const float* __restrict__ v_scale,
                      const int32_t* __restrict__ n_keep, int Nc_cap, int H, uint16_t* __restrict__ k_cache,
                      uint16_t* __restrict__ v_cache, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    constexpr int E = D / 32;
    const int b = blockIdx.y, j = blockIdx.x, is_v = blockIdx.z;
    int live = n_keep[b];
    if (live < 0 || live > Nc_cap) {
        if (threadIdx.x == 0 && j == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        live = live < 0 ? 0 : Nc_cap;
    }
    if (j >= live) return;
    const size_t rowoff = ((size_t)b * Nc_cap + j) * H;
    const uint8_t* src = (is_v ? v_q : k_q) + rowoff * D;
    const float* sc = (is_v ? v_scale : k_scale) + rowoff;
    uint16_t* dst = (is_v ? v_cache : k_cache) + rowoff * D;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int h = warp; h < H; h += kQuantWarps) {
        const float s = sc[h];
        // (code value) * 2^k is exact in bf16: 4 significant bits, exponent well inside the range
        if constexpr (E == 4) {
            const uint32_t q = *reinterpret_cast<const uint32_t*>(src + (size_t)h * D + lane * 4);
            uint2 w;
            w.x = pack_bf16x2(e4m3_value(q & 255u) * s, e4m3_value((q >> 8) & 255u) * s);
            w.y = pack_bf16x2(e4m3_value((q >> 16) & 255u) * s, e4m3_value(q >> 24) * s);
            *reinterpret_cast<uint2*>(dst + (size_t)h * D + lane * 4) = w;
        } else {
            const uint32_t q = *reinterpret_cast<const uint16_t*>(src + (size_t)h * D + lane * 2);
            *reinterpret_cast<uint32_t*>(dst + (size_t)h * D + lane * 2) =
                pack_bf16x2(e4m3_value(q & 255u) * s, e4m3_value(q >> 8) * s);
        }
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
    const dim3 grid(Nc_cap, B, 2);
    cudaError_t e = D == 128
        ? launch_overlapped(rikv_store_e4m3_kernel<128>, grid, dim3(kQuantWarps * 32), 0, (cudaStream_t)stream,
                            k_full, v_full, keep_rows, n_keep, N_full, Nc_cap, H, k_q, v_q, k_scale, v_scale, dev_status)
        : launch_overlapped(rikv_store_e4m3_kernel<64>, grid, dim3(kQuantWarps * 32), 0, (cudaStream_t)stream,
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
    const dim3 grid(Nc_cap, B, 2);
    cudaError_t e = D == 128
        ? launch_overlapped(rikv_load_e4m3_kernel<128>, grid, dim3(kQuantWarps * 32), 0, (cudaStream_t)stream,
                            k_q, v_q, k_scale, v_scale, n_keep, Nc_cap, H, k_cache, v_cache, dev_status)
        : launch_overlapped(rikv_load_e4m3_kernel<64>, grid, dim3(kQuantWarps * 32), 0, (cudaStream_t)stream,
                            k_q, v_q, k_scale, v_scale, n_keep, Nc_cap, H, k_cache, v_cache, dev_status);
    return launch_status(e);
}
