// Elementwise latent updates of the region steps: decayed cached velocity with
// the Euler update of the edited tokens (Sec. 4, case equation of the AVDCache;
// Sec. 3, Euler sampler equation) and the merge with one-step-predicted
// unedited tokens (one-step estimation equation; Algorithm 1).
//
// Both are HBM-bound: one thread owns 8 channels (one 128-bit access per
// tensor), fp32 math, bf16 round-to-nearest-even on the way out.
#include "common.cuh"

namespace regione {

constexpr int kLatThreads = 256;

__device__ __forceinline__ uint4 axpy8(uint4 x, uint4 v, float a) {   // x + a * v, per bf16 lane
    uint4 o;
    o.x = pack_bf16x2(fmaf(a, bf16_lo(v.x), bf16_lo(x.x)), fmaf(a, bf16_hi(v.x), bf16_hi(x.x)));
    o.y = pack_bf16x2(fmaf(a, bf16_lo(v.y), bf16_lo(x.y)), fmaf(a, bf16_hi(v.y), bf16_hi(x.y)));
    o.z = pack_bf16x2(fmaf(a, bf16_lo(v.z), bf16_lo(x.z)), fmaf(a, bf16_hi(v.z), bf16_hi(x.z)));
    o.w = pack_bf16x2(fmaf(a, bf16_lo(v.w), bf16_lo(x.w)), fmaf(a, bf16_hi(v.w), bf16_hi(x.w)));
    return o;
}

// x_e <- x_e - dt * (scale * v_in); optionally v_cache_out <- v_in.  One thread = 8 channels.
__global__ void __launch_bounds__(kLatThreads)
velocity_decay_kernel(const uint4* __restrict__ v_in, const PerRequestF neg_dt_scale_v, int b0,
                      uint4* __restrict__ x_e, uint4* __restrict__ v_cache_out,
                      const int32_t* __restrict__ n_edit, int Ne_cap, int cpr, int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int b = b0 + blockIdx.y;                       // requests b0 .. b0 + gridDim.y of the batch
    const float neg_dt_scale = neg_dt_scale_v.v[blockIdx.y];
    if (neg_dt_scale != neg_dt_scale) return;            // NaN: this request sits the call out
    int ne = n_edit[b];
    if (ne < 0 || ne > Ne_cap) {
        if (threadIdx.x == 0 && blockIdx.x == 0) record_status(dev_status, REGIONE_DEV_BOUNDS);
        ne = max(0, min(ne, Ne_cap));
    }
    const unsigned live = (unsigned)ne * (unsigned)cpr;
    const unsigned e = blockIdx.x * (unsigned)kLatThreads + threadIdx.x;
    if (e >= live) return;
    const size_t off = (size_t)b * Ne_cap * cpr + e;
    const uint4 v = ld_stream128(v_in + off);
    const uint4 x = x_e[off];
    x_e[off] = axpy8(x, v, neg_dt_scale);
    if (v_cache_out != nullptr) v_cache_out[off] = v;
}

// x_out[n] = slot[n] >= 0 ? x_e[slot[n]] : x_full[n] - dt * v_last[n].  One thread = kMergeUnroll
// chunks of 8 channels, blockDim apart; all slots are read first, then every data load is issued
// before the first store, so several independent loads per thread are in flight.
constexpr int kMergeUnroll = 4;

__global__ void __launch_bounds__(kLatThreads)
merge_kernel(const uint4* x_full, const uint4* __restrict__ v_last,
             const uint4* __restrict__ x_e, const int32_t* __restrict__ slot,
             const PerRequestF neg_dt_v, int b0, int N, int Ne_cap, int cpr, uint4* x_out,
             int32_t* dev_status) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int b = b0 + blockIdx.y;
    const float neg_dt = neg_dt_v.v[blockIdx.y];
    if (neg_dt != neg_dt) return;                        // NaN: this request sits the call out
    const unsigned total = (unsigned)N * (unsigned)cpr;
    const unsigned base = blockIdx.x * (unsigned)(kLatThreads * kMergeUnroll) + threadIdx.x;
    const size_t req = (size_t)b * N * cpr;
    int s[kMergeUnroll];
    unsigned c[kMergeUnroll];
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u) {
        const unsigned e = base + (unsigned)u * kLatThreads;
        s[u] = -2;                                   // -2: past the end, nothing to do
        if (e < total) {
            const unsigned n = e / (unsigned)cpr;
            c[u] = e - n * (unsigned)cpr;
            const int sv = slot[(size_t)b * N + n];
            s[u] = sv < 0 ? -1 : sv;                 // any negative slot means "unedited"
            if (s[u] >= Ne_cap) {
                record_status(dev_status, REGIONE_DEV_BOUNDS);
                s[u] = -2;
            }
        }
    }
    uint4 x[kMergeUnroll], v[kMergeUnroll];
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u) {
        const size_t off = req + base + (size_t)u * kLatThreads;
        if (s[u] >= 0) {
            x[u] = ldg128(x_e + ((size_t)b * Ne_cap + s[u]) * cpr + c[u]);
        } else if (s[u] == -1) {
            x[u] = x_full[off];
            v[u] = ld_stream128(v_last + off);
        }
    }
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u) {
        const size_t off = req + base + (size_t)u * kLatThreads;
        if (s[u] >= 0) x_out[off] = x[u];
        else if (s[u] == -1) x_out[off] = axpy8(x[u], v[u], neg_dt);
    }
}

}  // namespace regione

using namespace regione;

extern "C" int regione_velocity_decay(const regione_bf16* v_in, const float* scale, const float* dt,
                                      regione_bf16* x_e, regione_bf16* v_cache_out,
                                      const int32_t* n_edit, int B, int Ne_cap, int C,
                                      int32_t* dev_status, void* stream) {
    if (!v_in || !x_e || !n_edit || !scale || !dt) return REGIONE_INVALID_ARG;
    if (B < 0 || Ne_cap < 0 || C < 1) return REGIONE_INVALID_ARG;
    if (!aligned16(v_in) || !aligned16(x_e) || !aligned16(v_cache_out)) return REGIONE_INVALID_ARG;
    if ((C & 7) != 0 || B > 65535) return REGIONE_UNSUPPORTED;
    const long long cpr = C / 8, total = (long long)Ne_cap * cpr;
    if (total + kLatThreads >= 0x7fffffffLL) return REGIONE_UNSUPPORTED;
    if (B == 0 || Ne_cap == 0) return REGIONE_OK;
    cudaError_t e = cudaSuccess;
    for (int b0 = 0; b0 < B && e == cudaSuccess; b0 += kReqChunk) {
        const int nb = B - b0 < kReqChunk ? B - b0 : kReqChunk;
        PerRequestF a;                       // x - (dt * scale) * v, the product formed in fp32 first
        for (int i = 0; i < nb; ++i) a.v[i] = -(dt[b0 + i] * scale[b0 + i]);
        dim3 grid((unsigned)((total + kLatThreads - 1) / kLatThreads), nb);
        e = launch_overlapped(velocity_decay_kernel, grid, dim3(kLatThreads), 0, (cudaStream_t)stream,
                              (const uint4*)v_in, a, b0, (uint4*)x_e, (uint4*)v_cache_out, n_edit,
                              Ne_cap, (int)cpr, dev_status);
    }
    return launch_status(e);
}

extern "C" int regione_merge(const regione_bf16* x_full, const regione_bf16* v_last_full,
                             const regione_bf16* x_e, const int32_t* slot, const float* dt_unedited, int B,
                             int N, int Ne_cap, int C, regione_bf16* x_out, int32_t* dev_status,
                             void* stream) {
    if (!x_full || !v_last_full || !slot || !x_out || !dt_unedited) return REGIONE_INVALID_ARG;
    if (B < 0 || N < 1 || Ne_cap < 0 || C < 1) return REGIONE_INVALID_ARG;
    if (Ne_cap > 0 && !x_e) return REGIONE_INVALID_ARG;
    if (!aligned16(x_full) || !aligned16(v_last_full) || !aligned16(x_e) || !aligned16(x_out))
        return REGIONE_INVALID_ARG;
    if ((C & 7) != 0 || B > 65535) return REGIONE_UNSUPPORTED;
    const long long cpr = C / 8, total = (long long)N * cpr;
    if (total + kLatThreads >= 0x7fffffffLL) return REGIONE_UNSUPPORTED;
    if (B == 0) return REGIONE_OK;
    const long long per_block = (long long)kLatThreads * kMergeUnroll;
    cudaError_t e = cudaSuccess;
    for (int b0 = 0; b0 < B && e == cudaSuccess; b0 += kReqChunk) {
        const int nb = B - b0 < kReqChunk ? B - b0 : kReqChunk;
        PerRequestF a;
        for (int i = 0; i < nb; ++i) a.v[i] = -dt_unedited[b0 + i];
        dim3 grid((unsigned)((total + per_block - 1) / per_block), nb);
        e = launch_overlapped(merge_kernel, grid, dim3(kLatThreads), 0, (cudaStream_t)stream,
                              (const uint4*)x_full, (const uint4*)v_last_full, (const uint4*)x_e, slot, a,
                              b0, N, Ne_cap, (int)cpr, (uint4*)x_out, dev_status);
    }
    return launch_status(e);
}
