// Plain CUDA-core region attention: one warp per (request, head, query row),
// online softmax over the fresh rows and then the cached rows.  It exists to
// cross-check the tensor-core kernel on the device (same inputs, independent
// arithmetic path) and is reachable only through regione_crosscheck_region_attention; it is
// far from the tensor-core roofline and no product entry point calls it.
// (Sec. 4 "Region-Aware Generation", the attention equation.)
#include "common.cuh"

namespace regione {

constexpr int kSimtWarps = 8;

template <int D>
__global__ void __launch_bounds__(kSimtWarps * 32)
region_attention_simt_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_fresh,
                             const uint16_t* __restrict__ v_fresh,
                             const uint16_t* __restrict__ k_cache,
                             const uint16_t* __restrict__ v_cache, const int32_t* __restrict__ n_q,
                             const int32_t* __restrict__ n_fresh,
                             const int32_t* __restrict__ n_cache, int Nq_cap, int Nf_cap,
                             int Nc_cap, int H, float scale_log2e, uint16_t* __restrict__ out,
                             int32_t* dev_status) {
    __shared__ float qs[kSimtWarps][D];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.z, h = blockIdx.y;
    const int i = blockIdx.x * kSimtWarps + warp;
    int nq = n_q[b], nf = n_fresh[b], nc = n_cache[b];
    if (nq > Nq_cap || nf > Nf_cap || nc > Nc_cap || nq < 0 || nf < 0 || nc < 0) {
        record_status(dev_status, REGIONE_DEV_BOUNDS);
        nq = max(0, min(nq, Nq_cap)); nf = max(0, min(nf, Nf_cap)); nc = max(0, min(nc, Nc_cap));
    }
    if (i >= nq) return;
    const size_t rs = (size_t)H * D;                      // row stride in elements
    const uint16_t* qrow = q + ((size_t)b * Nq_cap + i) * rs + (size_t)h * D;
    for (int d = lane; d < D; d += 32) qs[warp][d] = __uint_as_float((uint32_t)qrow[d] << 16);
    __syncwarp();

    constexpr int DPL = D / 32;
    float acc[DPL];
#pragma unroll
    for (int x = 0; x < DPL; ++x) acc[x] = 0.f;
    float m = -INFINITY, l = 0.f;

    for (int seg = 0; seg < 2; ++seg) {
        const int n = seg == 0 ? nf : nc;
        const int cap = seg == 0 ? Nf_cap : Nc_cap;
        const uint16_t* kb = (seg == 0 ? k_fresh : k_cache);
        const uint16_t* vb = (seg == 0 ? v_fresh : v_cache);
        for (int j0 = 0; j0 < n; j0 += 32) {
            const int j = j0 + lane;
            float s = -INFINITY;
            if (j < n) {
                const uint4* kr = reinterpret_cast<const uint4*>(
                    kb + ((size_t)b * cap + j) * rs + (size_t)h * D);
                float dot = 0.f;
#pragma unroll
                for (int c = 0; c < D / 8; ++c) {
                    const uint4 kv = __ldg(kr + c);
                    const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        dot = fmaf(qs[warp][c * 8 + 2 * x], bf16_lo(w[x]), dot);
                        dot = fmaf(qs[warp][c * 8 + 2 * x + 1], bf16_hi(w[x]), dot);
                    }
                }
                s = dot * scale_log2e;
            }
            float cm = s;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, d));
            const float m_new = fmaxf(m, cm);
            const float corr = exp2f(m - m_new);
            const float p = (j < n) ? exp2f(s - m_new) : 0.f;
            float ps = p;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, d);
            l = l * corr + ps;
            m = m_new;
#pragma unroll
            for (int x = 0; x < DPL; ++x) acc[x] *= corr;
            const int cnt = min(32, n - j0);
            for (int jj = 0; jj < cnt; ++jj) {
                const float pj = __shfl_sync(0xffffffffu, p, jj);
                const uint16_t* vr = vb + ((size_t)b * cap + j0 + jj) * rs + (size_t)h * D;
#pragma unroll
                for (int x = 0; x < DPL; ++x)
                    acc[x] = fmaf(pj, __uint_as_float((uint32_t)__ldg(vr + lane + 32 * x) << 16),
                                  acc[x]);
            }
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    uint16_t* orow = out + ((size_t)b * Nq_cap + i) * rs + (size_t)h * D;
#pragma unroll
    for (int x = 0; x < DPL; ++x) {
        __nv_bfloat16 o = __float2bfloat16_rn(acc[x] * inv);
        orow[lane + 32 * x] = *reinterpret_cast<uint16_t*>(&o);
    }
}

int launch_region_attention_simt(const uint16_t* q, const uint16_t* k_fresh,
                                 const uint16_t* v_fresh, const uint16_t* k_cache,
                                 const uint16_t* v_cache, const int32_t* n_q,
                                 const int32_t* n_fresh, const int32_t* n_cache, int B, int Nq_cap,
                                 int Nf_cap, int Nc_cap, int H, int D, float scale, uint16_t* out,
                                 int32_t* dev_status, cudaStream_t st) {
    dim3 grid((Nq_cap + kSimtWarps - 1) / kSimtWarps, H, B);
    const float sl2 = scale * 1.4426950408889634f;
    if (D == 64)
        region_attention_simt_kernel<64><<<grid, kSimtWarps * 32, 0, st>>>(
            q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, Nq_cap, Nf_cap, Nc_cap, H,
            sl2, out, dev_status);
    else
        region_attention_simt_kernel<128><<<grid, kSimtWarps * 32, 0, st>>>(
            q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, Nq_cap, Nf_cap, Nc_cap, H,
            sl2, out, dev_status);
    return launch_status(cudaGetLastError());
}

}  // namespace regione
