// Host-only entry points of libregione: version, status names, the AVDCache
// criterion (a scalar recurrence evaluated on the host), and the argument checks
// and entry points of the region attention.

#include "common.cuh"

namespace regione {
int launch_region_attention_simt(const uint16_t*, const uint16_t*, const uint16_t*, const uint16_t*,
                                 const uint16_t*, const int32_t*, const int32_t*, const int32_t*,
                                 int, int, int, int, int, int, float, uint16_t*, int32_t*,
                                 cudaStream_t);
size_t region_attention_tc_workspace(int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D);
int launch_region_attention_tc(const uint16_t*, const uint16_t*, const uint16_t*, const uint16_t*,
                               const uint16_t*, const int32_t*, const int32_t*, const int32_t*, int,
                               int, int, int, int, int, float, uint16_t*, const int32_t*, int, void*,
                               size_t, int32_t*, cudaStream_t, const CacheStore*);
}  // namespace regione

using namespace regione;

extern "C" int regione_version(void) { return 200; }

extern "C" const char* regione_status_string(int status) {
    switch (status) {
        case REGIONE_OK: return "REGIONE_OK";
        case REGIONE_INVALID_ARG: return "REGIONE_INVALID_ARG";
        case REGIONE_UNSUPPORTED: return "REGIONE_UNSUPPORTED";
        case REGIONE_CUDA_ERROR: return "REGIONE_CUDA_ERROR";
        case REGIONE_WORKSPACE_TOO_SMALL: return "REGIONE_WORKSPACE_TOO_SMALL";
        case REGIONE_DEV_TIMEOUT: return "REGIONE_DEV_TIMEOUT";
        case REGIONE_DEV_BOUNDS: return "REGIONE_DEV_BOUNDS";
        default: return "REGIONE_UNKNOWN";
    }
}

extern "C" int regione_avd_step(double* running_product, double dt, double gamma, double delta,
                                int* reuse) {
    if (!running_product || !reuse) return REGIONE_INVALID_ARG;
    const double p = *running_product * (1.0 - dt) * gamma;
    if (1.0 - p > delta) {
        *reuse = 0;
        *running_product = 1.0;
    } else {
        *reuse = 1;
        *running_product = p;
    }
    return REGIONE_OK;
}

// Argument checks shared by every region-attention entry point.
int regione::check_attention_args(const void* q, const void* k_fresh, const void* v_fresh,
                                  const void* k_cache, const void* v_cache, const void* n_q,
                                  const void* n_fresh, const void* n_cache, int B, int Nq_cap,
                                  int Nf_cap, int Nc_cap, int H, int D, const void* out,
                                  bool* nothing_to_do) {
    *nothing_to_do = false;
    if (!q || !out || !n_q || !n_fresh || !n_cache) return REGIONE_INVALID_ARG;
    if (B < 0 || Nq_cap < 0 || Nf_cap < 0 || Nc_cap < 0 || H < 1) return REGIONE_INVALID_ARG;
    if (Nf_cap > 0 && (!k_fresh || !v_fresh)) return REGIONE_INVALID_ARG;
    if (Nc_cap > 0 && (!k_cache || !v_cache)) return REGIONE_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_fresh) || !aligned16(v_fresh) ||
        !aligned16(k_cache) || !aligned16(v_cache))
        return REGIONE_INVALID_ARG;
    if (D != 64 && D != 128) return REGIONE_UNSUPPORTED;
    if (B > 65535 || H > 65535) return REGIONE_UNSUPPORTED;
    *nothing_to_do = (B == 0 || Nq_cap == 0);
    return REGIONE_OK;
}

extern "C" size_t regione_region_attention_workspace(int B, int Nq_cap, int Nf_cap, int Nc_cap,
                                                     int H, int D) {
    if (B <= 0 || Nq_cap <= 0 || H <= 0 || (D != 64 && D != 128)) return 0;
    return region_attention_tc_workspace(B, Nq_cap, Nf_cap, Nc_cap, H, D);
}

// Shared body of regione_region_attention (out_rows == nullptr) and regione_region_attention_scatter.
static int region_attention_impl(const regione_bf16* q, const regione_bf16* k_fresh,
                                 const regione_bf16* v_fresh, const regione_bf16* k_cache,
                                 const regione_bf16* v_cache, const int32_t* n_q,
                                 const int32_t* n_fresh, const int32_t* n_cache, int B, int Nq_cap,
                                 int Nf_cap, int Nc_cap, int H, int D, float softmax_scale,
                                 regione_bf16* out, const int32_t* out_rows, int out_cap,
                                 void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                 void* stream) {
    bool nothing = false;
    const int rc = check_attention_args(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache,
                                        B, Nq_cap, Nf_cap, Nc_cap, H, D, out, &nothing);
    if (rc != REGIONE_OK || nothing) return rc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    const size_t need = region_attention_tc_workspace(B, Nq_cap, Nf_cap, Nc_cap, H, D);
    if (need > 0) {
        if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return REGIONE_INVALID_ARG;
        if (workspace_bytes < need) return REGIONE_WORKSPACE_TOO_SMALL;
    }
    return launch_region_attention_tc(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache,
                                      B, Nq_cap, Nf_cap, Nc_cap, H, D, scale, out, out_rows, out_cap,
                                      workspace, workspace_bytes, dev_status, (cudaStream_t)stream, nullptr);
}

extern "C" int regione_region_attention(const regione_bf16* q, const regione_bf16* k_fresh,
                                        const regione_bf16* v_fresh, const regione_bf16* k_cache,
                                        const regione_bf16* v_cache, const int32_t* n_q,
                                        const int32_t* n_fresh, const int32_t* n_cache, int B,
                                        int Nq_cap, int Nf_cap, int Nc_cap, int H, int D,
                                        float softmax_scale, regione_bf16* out, void* workspace,
                                        size_t workspace_bytes, int32_t* dev_status, void* stream) {
    return region_attention_impl(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, B,
                                 Nq_cap, Nf_cap, Nc_cap, H, D, softmax_scale, out, nullptr, 0,
                                 workspace, workspace_bytes, dev_status, stream);
}

extern "C" int regione_region_attention_scatter(
    const regione_bf16* q, const regione_bf16* k_fresh, const regione_bf16* v_fresh,
    const regione_bf16* k_cache, const regione_bf16* v_cache, const int32_t* n_q,
    const int32_t* n_fresh, const int32_t* n_cache, int B, int Nq_cap, int Nf_cap, int Nc_cap, int H,
    int D, float softmax_scale, regione_bf16* out_full, int out_rows_cap, const int32_t* out_rows,
    void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    if (!out_rows || out_rows_cap < 1) return REGIONE_INVALID_ARG;
    return region_attention_impl(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache, B,
                                 Nq_cap, Nf_cap, Nc_cap, H, D, softmax_scale, out_full, out_rows,
                                 out_rows_cap, workspace, workspace_bytes, dev_status, stream);
}

extern "C" size_t regione_full_attention_store_workspace(int B, int N_cap, int H, int D) {
    return regione_region_attention_workspace(B, N_cap, N_cap, 0, H, D);
}

extern "C" int regione_full_attention_store(
    const regione_bf16* q, const regione_bf16* k, const regione_bf16* v, const int32_t* n_rows, int B,
    int N_cap, int H, int D, float softmax_scale, const int32_t* keep_rows, const int32_t* n_keep,
    int Nc_cap, regione_bf16* k_cache, regione_bf16* v_cache, regione_bf16* out, void* workspace,
    size_t workspace_bytes, int32_t* dev_status, void* stream) {
    bool nothing = false;
    const int rc = check_attention_args(q, k, v, nullptr, nullptr, n_rows, n_rows, n_rows, B, N_cap, N_cap,
                                        0, H, D, out, &nothing);
    if (rc != REGIONE_OK) return rc;
    if (!keep_rows || !n_keep || Nc_cap < 0) return REGIONE_INVALID_ARG;
    if (Nc_cap > 0 && (!k_cache || !v_cache)) return REGIONE_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache)) return REGIONE_INVALID_ARG;
    if (nothing || N_cap == 0) return REGIONE_OK;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    const size_t need = region_attention_tc_workspace(B, N_cap, N_cap, 0, H, D);
    if (need > 0) {
        if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return REGIONE_INVALID_ARG;
        if (workspace_bytes < need) return REGIONE_WORKSPACE_TOO_SMALL;
    }
    CacheStore store;
    store.keep_rows = keep_rows; store.n_keep = n_keep; store.cap = Nc_cap;
    store.k_cache = k_cache; store.v_cache = v_cache;
    // no cached segment: n_cache = nullptr stands for "zero rows" in every request
    return launch_region_attention_tc(q, k, v, nullptr, nullptr, n_rows, n_rows, nullptr, B, N_cap, N_cap, 0,
                                      H, D, scale, out, nullptr, 0, workspace, workspace_bytes, dev_status,
                                      (cudaStream_t)stream, Nc_cap > 0 ? &store : nullptr);
}

// The CUDA-core kernel, reachable only through this symbol: an independent arithmetic path on the
// device that the tests compare the tensor-core kernel with.  Never called by the library itself.
extern "C" int regione_crosscheck_region_attention(
    const regione_bf16* q, const regione_bf16* k_fresh, const regione_bf16* v_fresh,
    const regione_bf16* k_cache, const regione_bf16* v_cache, const int32_t* n_q,
    const int32_t* n_fresh, const int32_t* n_cache, int B, int Nq_cap, int Nf_cap, int Nc_cap, int H,
    int D, float softmax_scale, regione_bf16* out, int32_t* dev_status, void* stream) {
    bool nothing = false;
    const int rc = check_attention_args(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache,
                                        B, Nq_cap, Nf_cap, Nc_cap, H, D, out, &nothing);
    if (rc != REGIONE_OK || nothing) return rc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    return launch_region_attention_simt(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache,
                                        B, Nq_cap, Nf_cap, Nc_cap, H, D, scale, out, dev_status,
                                        (cudaStream_t)stream);
}
