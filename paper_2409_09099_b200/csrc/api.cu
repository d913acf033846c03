// Context management, size queries and status handling of libsste (host only).
#include <new>

#include "common.cuh"

#include <atomic>

static std::atomic<unsigned long long> g_launch_count{0};
void sste_count_launches(int n) { g_launch_count.fetch_add(static_cast<unsigned long long>(n), std::memory_order_relaxed); }
extern "C" unsigned long long sste_debug_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

extern "C" size_t sste_workspace_bytes(void) { return SSTE_WS_BYTES; }
extern "C" size_t sste_workspace_bytes_recommended(void) { return SSTE_WS_RECOMMENDED_BYTES; }

extern "C" const char *sste_status_string(sste_status s)
{
    switch (s) {
    case SSTE_OK: return "ok";
    case SSTE_ERR_INVALID_ARG: return "invalid argument";
    case SSTE_ERR_SHAPE: return "dimension is not a positive multiple of 128";
    case SSTE_ERR_DTYPE: return "unsupported dtype combination";
    case SSTE_ERR_ALIGN: return "pointer is not 128-byte aligned";
    case SSTE_ERR_WORKSPACE: return "workspace missing or too small";
    case SSTE_ERR_ARCH: return "device is not sm_100";
    case SSTE_ERR_CUDA: return "CUDA call failed";
    case SSTE_ERR_DEGENERATE: return "S_soft(W) is identically zero; beta set to 1";
    case SSTE_ERR_TIMEOUT: return "bounded device-side wait expired";
    }
    return "unknown status";
}

extern "C" sste_status sste_create(sste_ctx **out, int device, void *workspace, size_t workspace_bytes)
{
    if (!out) return SSTE_ERR_INVALID_ARG;
    *out = nullptr;
    if (!workspace || workspace_bytes < SSTE_WS_BYTES) return SSTE_ERR_WORKSPACE;
    if (!sste_aligned(workspace, 256)) return SSTE_ERR_ALIGN;
    int count = 0;
    SSTE_CUDA_TRY(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) return SSTE_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    SSTE_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return SSTE_ERR_ARCH;
    sste_device_guard guard(device);
    if (!guard.ok) return SSTE_ERR_CUDA;

    void *encode = nullptr;
    cudaDriverEntryPointQueryResult qres;
    SSTE_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &encode, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !encode) return SSTE_ERR_CUDA;

    sste_ctx *ctx = new (std::nothrow) sste_ctx;
    if (!ctx) return SSTE_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->status_dev = reinterpret_cast<unsigned int *>(ws + SSTE_WS_STATUS_OFF);
    ctx->counter_dev = reinterpret_cast<unsigned int *>(ws + SSTE_WS_COUNTER_OFF);
    ctx->partials_dev = reinterpret_cast<double *>(ws + SSTE_WS_PARTIALS_OFF);
    ctx->cu_tensor_map_encode = encode;
    ctx->splitk_partials = nullptr;
    ctx->splitk_partial_bytes = 0;
    if (workspace_bytes > SSTE_WS_SPLITK_PARTIALS_OFF + (size_t(1) << 20)) {
        ctx->splitk_partials = reinterpret_cast<float *>(ws + SSTE_WS_SPLITK_PARTIALS_OFF);
        ctx->splitk_partial_bytes = workspace_bytes - SSTE_WS_SPLITK_PARTIALS_OFF;
    }
    if (cudaMemset(ws, 0, SSTE_WS_PARTIALS_OFF) != cudaSuccess) {
        delete ctx;
        return SSTE_ERR_CUDA;
    }
    *out = ctx;
    return SSTE_OK;
}

extern "C" sste_status sste_destroy(sste_ctx *ctx)
{
    if (!ctx) return SSTE_ERR_INVALID_ARG;
    delete ctx;
    return SSTE_OK;
}

extern "C" sste_status sste_poll_device_status(sste_ctx *ctx, void *stream)
{
    if (!ctx) return SSTE_ERR_INVALID_ARG;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned int word = 0;
    SSTE_CUDA_TRY(cudaMemcpyAsync(&word, ctx->status_dev, sizeof word, cudaMemcpyDeviceToHost, s));
    SSTE_CUDA_TRY(cudaMemsetAsync(ctx->status_dev, 0, sizeof word, s));
    SSTE_CUDA_TRY(cudaStreamSynchronize(s));
    if (word > SSTE_ERR_TIMEOUT) return SSTE_ERR_CUDA;
    return static_cast<sste_status>(word);
}

extern "C" size_t sste_vals_bytes(int rows, int k, sste_dtype dt)
{
    if (rows <= 0 || k <= 0) return 0;
    size_t elt = (dt == SSTE_BF16) ? 2 : (dt == SSTE_E4M3 || dt == SSTE_E5M2) ? 1 : 0;
    return static_cast<size_t>(rows) * static_cast<size_t>(k / 2) * elt;
}

extern "C" size_t sste_meta_bytes(int rows, int k)
{
    if (rows <= 0 || k <= 0) return 0;
    return static_cast<size_t>(rows) * static_cast<size_t>(k) / 8;
}
