// sste_beta_init_static: the beta reduction (Eq. 5) for callers that have no device memory to lend.
//
// Some users of this library run where nothing may be allocated on the device: inside a serving or
// training runtime that owns the whole memory pool and hands out no scratch, in a plug-in that is only
// ever given its input and output buffers, or late in a job when the device is full.  They cannot build
// an sste_ctx either, because a context lives in a caller-provided device workspace.  For them the block
// partials and the ticket counter of the reduction live in a fixed array that is part of the library
// image: every GPU that loads libsste holds these STATIC_SCRATCH_BYTES (about 129 KB) until the process
// exits, and in exchange the call needs no cudaMalloc, no workspace and no context.
//
// One block reduces one 128 x 128 tile of W and writes one (numerator, denominator) pair, so the array
// bounds the tensor size: at most SSTE_STATIC_MAX_TILES tiles (O/128 * I/128 <= 8192, i.e. 134 M
// weights); larger tensors are refused with SSTE_ERR_WORKSPACE before anything is launched.
//
// All calls on a device share the one array.  The previous call's partials are still in it (they are
// overwritten, never accumulated), the ticket counter is cleared on the stream at the start of every
// call, and two calls whose kernels overlap on the GPU (different streams, no ordering) corrupt each
// other: keep calls on one device stream-ordered.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int SSTE_STATIC_MAX_TILES = 8192;
constexpr size_t STATIC_PARTIALS_OFF = 256;   // [0, 256): ticket counter; then two doubles per tile
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_PARTIALS_OFF + 2 * sizeof(double) * SSTE_STATIC_MAX_TILES;

// Device scratch.  In host code this name is only a handle for cudaGetSymbolAddress, not an address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
void *g_scratch_addr[MAX_DEVICES] = {};   // device address of g_static_scratch, per device
int g_device_major[MAX_DEVICES] = {};     // compute-capability major of the device, looked up with the address
std::mutex g_setup_mutex;

__device__ __forceinline__ double warp_sum_f64(double v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// One block = one 128 x 128 tile (2048 chunks of 8 bf16, 8 per thread).  s = S_soft(w) in exact
// arithmetic (fp64), products and sums in fp64; the last block to finish adds the tile partials in
// tile order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256)
beta_static_kernel(const uint4 *__restrict__ W, int I, unsigned char *__restrict__ scratch, float *__restrict__ beta_dev)
{
    __shared__ double red[2][8];
    __shared__ bool is_last;
    unsigned int *counter = reinterpret_cast<unsigned int *>(scratch);
    double *partials = reinterpret_cast<double *>(scratch + STATIC_PARTIALS_OFF);
    const int tiles_k = I / 128;
    const int tile = blockIdx.x, rb = tile / tiles_k, kb = tile % tiles_k;
    const size_t row_chunks = static_cast<size_t>(I) / 8;
    double num = 0.0, den = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int c = i * 256 + threadIdx.x;
        const int row = c >> 4, kc = c & 15;
        const uint4 v = __ldg(W + (static_cast<size_t>(rb) * 128 + row) * row_chunks + kb * 16 + kc);
        const uint32_t raw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const uint32_t bits[4] = {raw[2 * g] & 0xffffu, raw[2 * g] >> 16, raw[2 * g + 1] & 0xffffu, raw[2 * g + 1] >> 16};
            double a[4], m[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a[e] = static_cast<double>(sste_bf16_bits_to_f32(bits[e]));
                m[e] = fabs(a[e]);
            }
            // t = second-smallest magnitude of the group (Eq. 4)
            const double t = fmin(fmax(fmin(m[0], m[1]), fmin(m[2], m[3])), fmin(fmax(m[0], m[1]), fmax(m[2], m[3])));
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const double d = m[e] - t;
                if (d > 0.0) {
                    const double s = copysign(d, a[e]);
                    num += a[e] * s;
                    den += s * s;
                }
            }
        }
    }
    num = warp_sum_f64(num);
    den = warp_sum_f64(den);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red[0][warp] = num; red[1][warp] = den; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double bn = 0.0, bd = 0.0;
        for (int w = 0; w < 8; ++w) { bn += red[0][w]; bd += red[1][w]; }
        partials[2 * tile] = bn;
        partials[2 * tile + 1] = bd;
        __threadfence();
        is_last = (atomicAdd(counter, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (is_last && threadIdx.x < 32) {
        __threadfence();
        double tn = 0.0, td = 0.0;
        for (unsigned int b = threadIdx.x; b < gridDim.x; b += 32) {
            tn += __ldcg(partials + 2 * b);
            td += __ldcg(partials + 2 * b + 1);
        }
        tn = warp_sum_f64(tn);
        td = warp_sum_f64(td);
        if (threadIdx.x == 0) *beta_dev = (td == 0.0) ? 1.0f : static_cast<float>(tn / td);
    }
}

// Device address of the scratch array on the current device.  Looked up once per device, together with
// the device's architecture (the kernel image exists for compute capability 10.x only).
sste_status scratch_address(int device, unsigned char **out)
{
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_device_major[device]) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return SSTE_ERR_CUDA;
        g_device_major[device] = major;
    }
    if (g_device_major[device] != 10) return SSTE_ERR_ARCH;
    if (!g_scratch_addr[device]) {
        void *addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return SSTE_ERR_CUDA;
        g_scratch_addr[device] = addr;
    }
    *out = static_cast<unsigned char *>(g_scratch_addr[device]);
    return SSTE_OK;
}

}  // namespace

extern "C" sste_status sste_beta_init_static(int device, const void *W, int O, int I, sste_dtype wdt, float *beta_dev,
                                             void *stream)
{
    if (!W || !beta_dev || device < 0 || device >= MAX_DEVICES) return SSTE_ERR_INVALID_ARG;
    if (wdt != SSTE_BF16) return SSTE_ERR_DTYPE;
    if (!sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    const long long tiles = static_cast<long long>(O / 128) * (I / 128);
    if (tiles > SSTE_STATIC_MAX_TILES) return SSTE_ERR_WORKSPACE;   // the built-in scratch holds 8192 tile partials
    if (!sste_aligned(W, 128) || !sste_aligned(beta_dev, 4)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    unsigned char *scratch = nullptr;
    const sste_status st = scratch_address(device, &scratch);   // first call on a device: one symbol look-up
    if (st != SSTE_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SSTE_CUDA_TRY(cudaMemsetAsync(scratch, 0, sizeof(unsigned int), s));   // the ticket counter starts at zero
    // the launch's own return code: an earlier, unrelated sticky error is not reported as this call's
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned int>(tiles));
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    SSTE_CUDA_TRY(cudaLaunchKernelEx(&cfg, beta_static_kernel, static_cast<const uint4 *>(W), I, scratch, beta_dev));
    sste_count_launches(1);
    return SSTE_OK;
}
