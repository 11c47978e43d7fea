// Fitting the timestep-aware decay correction gamma_t of the Adaptive Velocity Decay Cache
// (Sec. 4 "Adaptive Velocity Decay Cache", decay-factor equation:
// ||v_{t_i}|| / ||v_{t_{i+1}}|| = (1 - dt_i) * gamma_{t_i}; the paper fits gamma on sampled data and
// does not say how).  Given the velocities of S
// sampled trajectories at T+1 consecutive steps, gamma_i is the mean over the samples of the norm
// ratio divided by the solver factor (1 - dt_i).
//
// Two kernels: an HBM-bound sum of squares (one CTA per (sample, step) row, 128-bit streaming
// loads, deterministic block reduction), then one thread per step averaging the S ratios.
#include "common.cuh"

namespace regione {

constexpr int kNormThreads = 256;

// norms[s, i] = || v[s, i, :] ||_2
__global__ void __launch_bounds__(kNormThreads)
velocity_norm_kernel(const uint4* __restrict__ v, long long chunks, float* __restrict__ norms) {
    grid_dependency_wait();
    grid_launch_dependents();
    const long long row = blockIdx.x;
    const uint4* p = v + row * chunks;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    constexpr int U = 8;                     // independent 16-byte loads in flight per thread
    for (long long c = threadIdx.x; c < chunks; c += U * kNormThreads) {
        uint4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long cc = c + (long long)u * kNormThreads;
            x[u] = cc < chunks ? ld_stream128(p + cc) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float a = bf16_lo(w[k]), b = bf16_hi(w[k]);
                acc[k] = fmaf(a, a, acc[k]);
                acc[k] = fmaf(b, b, acc[k]);
            }
        }
    }
    float s = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
    __shared__ float part[kNormThreads / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int w = 0; w < kNormThreads / 32; ++w) tot += part[w];       // fixed order
        norms[row] = sqrtf(tot);
    }
}

// gamma[i] = mean_s( norms[s, i] / norms[s, i+1] ) / (1 - dt[i]),  i < T.  Steps are stored in the
// order the sampler takes them reversed: index i+1 is the earlier (noisier) step, as in the paper.
__global__ void gamma_kernel(const float* __restrict__ norms, const float* __restrict__ dt, int S,
                             int T1, float* __restrict__ gamma) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T1 - 1) return;
    float sum = 0.f;
    for (int s = 0; s < S; ++s) {
        const float den = norms[(size_t)s * T1 + i + 1];
        sum += den > 0.f ? norms[(size_t)s * T1 + i] / den : 0.f;
    }
    gamma[i] = sum / (float)S / (1.f - dt[i]);
}

}  // namespace regione

using namespace regione;

extern "C" int regione_gamma_fit(const regione_bf16* v, int S, int T1, int64_t n, const float* dt,
                                 float* norms, float* gamma, void* stream) {
    if (!v || !dt || !norms || !gamma) return REGIONE_INVALID_ARG;
    if (S < 1 || T1 < 2 || n < 1) return REGIONE_INVALID_ARG;
    if (!aligned16(v)) return REGIONE_INVALID_ARG;
    if ((n & 7) != 0 || (int64_t)S * T1 > 0x7fffffffLL) return REGIONE_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_overlapped(velocity_norm_kernel, dim3((unsigned)(S * T1)), dim3(kNormThreads), 0, st,
                          (const uint4*)v, (long long)(n / 8), norms) != cudaSuccess)
        return REGIONE_CUDA_ERROR;
    return launch_status(launch_overlapped(gamma_kernel, dim3((T1 - 1 + 127) / 128), dim3(128), 0, st,
                                           (const float*)norms, dt, S, T1, gamma));
}
