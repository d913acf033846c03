// Shared declarations of libsste's translation units: the context, argument
// checks and the small device helpers every kernel uses.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sste.h"

// The context owns nothing but views into the caller's workspace.
struct sste_ctx {
    int device;
    int sm_count;
    unsigned int *status_dev;   // device status word (first word of the workspace)
    unsigned int *counter_dev;  // ticket counter of the beta reduction
    double *partials_dev;       // 2 doubles per reduction block
    void *cu_tensor_map_encode; // cuTensorMapEncodeTiled, resolved through the runtime
    float *splitk_partials;         // fp32 partial tiles of split-K products; null if the workspace is minimal
    size_t splitk_partial_bytes;
};

constexpr int SSTE_MAX_REDUCE_BLOCKS = 1024;
constexpr size_t SSTE_WS_STATUS_OFF = 0;
constexpr size_t SSTE_WS_COUNTER_OFF = 64;
constexpr size_t SSTE_WS_PARTIALS_OFF = 256;
constexpr size_t SSTE_WS_BYTES = SSTE_WS_PARTIALS_OFF + 2 * sizeof(double) * SSTE_MAX_REDUCE_BLOCKS;
// optional tail of the workspace, used by split-K products
constexpr size_t SSTE_WS_SPLITK_PARTIALS_OFF = (SSTE_WS_BYTES + 1023) / 1024 * 1024;
constexpr size_t SSTE_WS_RECOMMENDED_BYTES = SSTE_WS_SPLITK_PARTIALS_OFF + (size_t(192) << 20);

static inline bool sste_mult128(int v) { return v > 0 && (v % 128) == 0; }
static inline bool sste_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

#define SSTE_CUDA_TRY(expr)                         \
    do {                                            \
        cudaError_t e__ = (expr);                   \
        if (e__ != cudaSuccess) return SSTE_ERR_CUDA; \
    } while (0)

// Make `ctx->device` current for the duration of a call.
struct sste_device_guard {
    int prev = -1;
    bool ok = true;
    explicit sste_device_guard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~sste_device_guard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// ---------------------------------------------------------------- device helpers

__device__ __forceinline__ float sste_bf16_bits_to_f32(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

// fp32 -> bf16 bits, round to nearest even (finite inputs)
__device__ __forceinline__ uint32_t sste_f32_to_bf16_bits(float f)
{
    return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(f)));
}

__device__ __forceinline__ uint32_t sste_f32_to_e4m3(float f)
{
    return static_cast<uint32_t>(__nv_cvt_float_to_fp8(f, __NV_SATFINITE, __NV_E4M3));
}

__device__ __forceinline__ uint32_t sste_f32_to_e5m2(float f)
{
    return static_cast<uint32_t>(__nv_cvt_float_to_fp8(f, __NV_SATFINITE, __NV_E5M2));
}

// FP8 per-tensor scaling (Sec. 5.2): scale = fp8_max / amax, 1 for an all-zero tensor.  Every kernel that
// quantises or rescales forms the scale from the tensor's amax with exactly these single-rounded operations.
__device__ __forceinline__ float sste_scale_from_amax(float amax, float fp8_max)
{
    return (amax == 0.0f) ? 1.0f : __fdiv_rn(fp8_max, amax);
}
// factor that undoes the scales of two quantised operands in a product's epilogue: fl(fl(1/sa) * fl(1/sb))
__device__ __forceinline__ float sste_out_scale(const float *a_amax, float a_fp8_max, const float *b_amax, float b_fp8_max)
{
    if (!a_amax || !b_amax) return 1.0f;
    const float ia = __fdiv_rn(1.0f, sste_scale_from_amax(*a_amax, a_fp8_max));
    const float ib = __fdiv_rn(1.0f, sste_scale_from_amax(*b_amax, b_fp8_max));
    return __fmul_rn(ia, ib);
}
static inline float sste_fp8_max(sste_dtype dt) { return dt == SSTE_E4M3 ? 448.0f : dt == SSTE_E5M2 ? 57344.0f : 0.0f; }

// Byte offset of (row m, K-offset k) inside a 2 KB metadata atom of 128 rows x 128 logical K.
__device__ __host__ __forceinline__ uint32_t sste_meta_atom_byte16(uint32_t m, uint32_t k)
{
    return 16u * (m & 7u) + 2u * ((m >> 3) & 1u) + 256u * (m >> 4) + 128u * ((k >> 4) & 1u) + 4u * (k >> 5) +
           ((k >> 3) & 1u);
}
__device__ __host__ __forceinline__ uint32_t sste_meta_atom_byte8(uint32_t m, uint32_t k) { return 16u * m + (k >> 3); }

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of the path is launched with programmatic stream serialisation: its CTAs may be scheduled,
// and run their prologue (barrier and tensor-memory set-up, descriptor prefetch, index arithmetic), while the
// previous kernel of the stream is still draining.  sste_pdl_wait() returns once that previous kernel has
// finished and its writes are visible; no kernel touches global memory before it.  sste_pdl_trigger(), issued
// first thing, is what lets the NEXT kernel of the stream be scheduled early (it takes effect when every CTA
// of this grid has issued it or exited, so the successor never competes with CTAs not yet started).
__device__ __forceinline__ void sste_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void sste_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t sste_launch(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                               Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Process-wide count of kernels this library has launched (read by sste_debug_launch_count).
void sste_count_launches(int n);
