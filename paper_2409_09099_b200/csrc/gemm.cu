// Tensor-core products of the S-STE linear layer (Sec. 5.1) for sm_100a:
//   forward      Z^T = S(W) X^T              sparse A (values + metadata), K-major B
//   grad weight  grad_W = MVUE(grad_Z^T) X   sparse A, MN-major B
//   grad input   grad_X = grad_Z S(W)        dense A, MN-major B
// One persistent, warp-specialised kernel template: a TMA producer warp fills a
// shared-memory ring, one thread issues tcgen05.mma / tcgen05.mma.sp with fp32
// accumulators in tensor memory, four warps drain the accumulators.  The 2:4
// metadata travels HBM -> shared memory (bulk copy) -> tensor memory (tcgen05.cp).
// Every wait is bounded: on expiry the CTA records SSTE_ERR_TIMEOUT and leaves.
#include <cuda.h>

#include "common.cuh"

namespace {

constexpr int BM = 128;            // rows of A per tile (= UMMA M)
constexpr int GEMM_THREADS = 192;  // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..5: epilogue
constexpr int TMEM_COLS = 512;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about two seconds

enum class BMajor { K, MN };

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (after recording a timeout) instead of spinning forever.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned int *status, volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long start = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - start > WAIT_LIMIT_CYCLES) {
            atomicCAS(status, 0u, static_cast<unsigned int>(SSTE_ERR_TIMEOUT));
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// arrive on an mbarrier once all tcgen05 operations issued so far by this thread have completed
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared memory -> tensor memory, 128 lanes x 16 bytes
__device__ __forceinline__ void tc_cp_128x128b(uint32_t taddr, uint64_t sdesc)
{
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
template <bool F8>
__device__ __forceinline__ void tc_mma_dense(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    if (F8)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
template <bool F8>
__device__ __forceinline__ void tc_mma_sparse(uint32_t d, uint64_t a, uint64_t b, uint32_t e, uint32_t idesc,
                                              uint32_t accumulate)
{
    if (F8)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "tcgen05.mma.sp.cta_group::1.kind::f8f6f4 [%0], %1, %2, [%3], %4, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(e), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(e), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns -> 32 registers per thread
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t r[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------ descriptors

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4),
// descriptor version 1, swizzle mode in the top three bits (0 none, 2 = 128 B, 4 = 64 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle)
{
    return static_cast<uint64_t>((addr & 0x3ffffu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
           (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (1ull << 46) | (static_cast<uint64_t>(swizzle) << 61);
}

// Instruction descriptor: sparse selector [0,2), sparse flag [2], D = fp32 [4,6), A format [7,10),
// B format [10,13), A major [15], B major [16] (1 = MN-major), N>>3 [17,23), M>>4 [24,29).
__host__ __device__ constexpr uint32_t instr_desc(bool sparse, uint32_t afmt, uint32_t bfmt, bool b_mn_major, int n)
{
    return (sparse ? 4u : 0u) | (1u << 4) | (afmt << 7) | (bfmt << 10) | ((b_mn_major ? 1u : 0u) << 16) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);
}

// ------------------------------------------------------------------ kernel

struct GemmParams {
    int M, N, K;            // logical problem: D[M, N] = A[M, K] * B
    const uint8_t *meta;    // metadata image of A (sparse only)
    void *D;                // output
    const float *out_scale; // device scalar or null
    unsigned int *status;
    uint32_t afmt, bfmt;    // operand format codes of the instruction descriptor
};

template <bool SPARSE, int BN>
struct Cfg {
    static constexpr int A_STAGE = SPARSE ? 8192 : 16384;       // 128 rows x (64 | 128) bytes
    static constexpr int B_STAGE = BN * 128;                    // BN rows x 128 bytes (or 128 B x BK rows per chunk)
    static constexpr int META_STAGE = SPARSE ? 2048 : 0;
    static constexpr int STAGE = A_STAGE + B_STAGE + META_STAGE;
    static constexpr int STAGES = (BN == 256) ? (SPARSE ? 5 : 4) : (SPARSE ? 8 : 6);
    static constexpr int ACC_BUFS = (BN == 256) ? 1 : 2;
    static constexpr int META_COL0 = 256;                       // accumulators occupy columns [0, 256)
    static constexpr int SMEM_BYTES = STAGES * STAGE + 1024 /* alignment slack */ + 256 /* barriers */;
};

// ELT: operand element size in bytes (2 = bf16 via kind::f16, 1 = fp8 via kind::f8f6f4).
// OUT_T: store D transposed (out[n, m]); OUT_F32: fp32 output instead of bf16.
template <bool SPARSE, BMajor BMAJ, int ELT, int BN, bool OUT_T, bool OUT_F32>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const GemmParams p)
{
    using C = Cfg<SPARSE, BN>;
    constexpr int NS = C::STAGES;
    constexpr int BK = 128 / ELT;                     // logical K per stage (B rows are 128 bytes of K)
    constexpr int MMA_PER_STAGE = SPARSE ? 2 : 4;     // sparse: 64 B of B's K per instruction, dense: 32 B
    constexpr bool F8 = (ELT == 1);
    constexpr int B_CHUNK_N = 128 / ELT;              // MN-major: N elements per 128-byte row
    constexpr int B_CHUNKS = BN / B_CHUNK_N;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = smem_base + NS * C::STAGE;             // barrier block, 8-byte aligned
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (NS + s); };
    auto acc_full_bar = [&](int b) { return bars + 8u * (2 * NS + b); };
    auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * NS + 2 + b); };
    const uint32_t tmem_slot = bars + 8u * (2 * NS + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + (bars - smem_u32(smem_raw)) + 8u * (2 * NS + 5));
    volatile uint32_t *tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m_tiles = p.M / BM;
    const int n_tiles = (p.N + BN - 1) / BN;
    const int num_tiles = m_tiles * n_tiles;
    const int k_blocks = p.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int mt = tile % m_tiles, nt = tile / m_tiles;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, p.status, abort_flag)) { ok = false; break; }
                    const uint32_t a_dst = smem_base + s * C::STAGE;
                    const uint32_t b_dst = a_dst + C::A_STAGE;
                    const bool load_meta = SPARSE && (F8 || (kb & 1) == 0);
                    mbar_arrive_expect_tx(full_bar(s), C::A_STAGE + C::B_STAGE + (load_meta ? 2048u : 0u));
                    // A: rows mt*128.., 64 bytes (compressed) or 128 bytes of K per row
                    tma_load_2d(a_dst, &map_a, full_bar(s), kb * (SPARSE ? BK / 2 : BK), mt * BM);
                    if (BMAJ == BMajor::K) {
                        tma_load_2d(b_dst, &map_b, full_bar(s), kb * BK, nt * BN);
                    } else {
#pragma unroll
                        for (int c = 0; c < B_CHUNKS; ++c)
                            tma_load_2d(b_dst + c * (BK * 128), &map_b, full_bar(s), nt * BN + c * B_CHUNK_N, kb * BK);
                    }
                    if (load_meta) {
                        const int atom_k = F8 ? kb : (kb >> 1);
                        const size_t atom = static_cast<size_t>(mt) * (p.K / 128) + atom_k;
                        bulk_load(b_dst + C::B_STAGE, p.meta + atom * 2048, 2048, full_bar(s));
                    }
                }
            }
            if (!ok) {
                // give copies already in flight time to land before the CTA leaves (bounded)
                const long long start = clock64();
                while (clock64() - start < 4000000ll) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc(SPARSE, p.afmt, p.bfmt, BMAJ == BMajor::MN, BN);
            uint32_t it = 0, local_tile = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local_tile) {
                const int buf = (C::ACC_BUFS == 2) ? (local_tile & 1) : 0;
                const uint32_t use = (C::ACC_BUFS == 2) ? (local_tile >> 1) : local_tile;
                if (!mbar_wait(acc_empty_bar(buf), (use & 1u) ^ 1u, p.status, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1u;
                    if (!mbar_wait(full_bar(s), ph, p.status, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = smem_base + s * C::STAGE;
                    const uint32_t b_src = a_src + C::A_STAGE;
                    uint32_t e_tmem = 0;
                    if (SPARSE) {
                        // One metadata atom (128 logical K, four 32-bit columns) per stage for fp8 and per two
                        // stages for bf16 (it arrives with the even k-block).  Tensor-memory regions rotate
                        // over NS atoms, so a region is rewritten only after the stages that read it retired.
                        const uint32_t atom_it = F8 ? it : (it >> 1);
                        const uint32_t region = tmem_base + C::META_COL0 + 4 * (atom_it % NS);
                        if (F8 || (kb & 1) == 0) {
                            const uint64_t mdesc = smem_desc(b_src + C::B_STAGE, 16, 128, 0);
                            tc_cp_128x128b(region, mdesc);
                        }
                        e_tmem = region + ((!F8 && (kb & 1)) ? 2u : 0u);
                    }
#pragma unroll
                    for (int j = 0; j < MMA_PER_STAGE; ++j) {
                        const uint64_t adesc = SPARSE ? smem_desc(a_src + 32 * j, 16, 512, 4)
                                                      : smem_desc(a_src + 32 * j, 16, 1024, 2);
                        uint64_t bdesc;
                        if (BMAJ == BMajor::K) {
                            bdesc = smem_desc(b_src + (SPARSE ? 64 : 32) * j, 16, 1024, 2);
                        } else {
                            constexpr int ROWS_PER_MMA = BK / MMA_PER_STAGE;     // K rows of 128 bytes per instruction
                            bdesc = smem_desc(b_src + ROWS_PER_MMA * 128 * j, BK * 128, 1024, 2);
                        }
                        const uint32_t acc = (kb > 0 || j > 0) ? 1u : 0u;
                        if (SPARSE) {
                            // bf16: one 32-bit metadata column per instruction, pairs selected by the descriptor's
                            // sparse selector; fp8: two columns per instruction
                            const uint32_t e = F8 ? (e_tmem + 2 * j) : e_tmem;
                            const uint32_t id2 = F8 ? 0u : static_cast<uint32_t>(j);
                            tc_mma_sparse<F8>(d_tmem, adesc, bdesc, e, idesc | id2, acc);
                        } else {
                            tc_mma_dense<F8>(d_tmem, adesc, bdesc, idesc, acc);
                        }
                    }
                    tc_commit(empty_bar(s));     // frees the stage once these MMAs (and the cp) have read it
                }
                if (ok) tc_commit(acc_full_bar(buf));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                  // tensor-memory lanes [32*quarter, 32*quarter + 32)
        const float scale = p.out_scale ? *p.out_scale : 1.0f;
        uint32_t local_tile = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local_tile) {
            const int mt = tile % m_tiles, nt = tile / m_tiles;
            const int buf = (C::ACC_BUFS == 2) ? (local_tile & 1) : 0;
            const uint32_t use = (C::ACC_BUFS == 2) ? (local_tile >> 1) : local_tile;
            if (!mbar_wait(acc_full_bar(buf), use & 1u, p.status, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int m = mt * BM + quarter * 32 + lane;
            const int n_valid = min(BN, p.N - nt * BN);
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (c0 >= n_valid) break;
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN + c0, r);
                tmem_ld_wait();
                const int n0 = nt * BN + c0;
                if (OUT_T) {
                    // out[n, m]: 32 lanes write 32 consecutive m for each n
                    if (OUT_F32) {
                        float *out = static_cast<float *>(p.D);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            out[static_cast<size_t>(n0 + c) * p.M + m] = __fmul_rn(__uint_as_float(r[c]), scale);
                    } else {
                        __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(p.D);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            out[static_cast<size_t>(n0 + c) * p.M + m] =
                                __float2bfloat16_rn(__fmul_rn(__uint_as_float(r[c]), scale));
                    }
                } else {
                    if (OUT_F32) {
                        float4 *out = reinterpret_cast<float4 *>(static_cast<float *>(p.D) + static_cast<size_t>(m) * p.N + n0);
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            out[c] = make_float4(__fmul_rn(__uint_as_float(r[4 * c]), scale),
                                                 __fmul_rn(__uint_as_float(r[4 * c + 1]), scale),
                                                 __fmul_rn(__uint_as_float(r[4 * c + 2]), scale),
                                                 __fmul_rn(__uint_as_float(r[4 * c + 3]), scale));
                    } else {
                        uint4 *out = reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(p.D) + static_cast<size_t>(m) * p.N + n0);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float lo = __fmul_rn(__uint_as_float(r[8 * c + 2 * e]), scale);
                                const float hi = __fmul_rn(__uint_as_float(r[8 * c + 2 * e + 1]), scale);
                                w[e] = sste_f32_to_bf16_bits(lo) | (sste_f32_to_bf16_bits(hi) << 16);
                            }
                            out[c] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(buf));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D row-major tensor [rows, cols] of `elt`-byte elements; box = box_cols x box_rows.
bool make_map(const sste_ctx *ctx, CUtensorMap *map, const void *base, int elt, uint64_t rows, uint64_t cols,
              uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle swz)
{
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * static_cast<uint64_t>(elt)};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = (elt == 2) ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->cu_tensor_map_encode);
    return fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool SPARSE, BMajor BMAJ, int ELT, int BN, bool OUT_T, bool OUT_F32>
sste_status launch(const sste_ctx *ctx, const void *A, const void *B, const GemmParams &p, cudaStream_t stream)
{
    using C = Cfg<SPARSE, BN>;
    constexpr int BK = 128 / ELT;
    CUtensorMap map_a, map_b;
    bool ok;
    if (SPARSE)   // compressed values [M, K/2], 64 bytes of K per row per stage
        ok = make_map(ctx, &map_a, A, ELT, p.M, p.K / 2, BK / 2, BM, CU_TENSOR_MAP_SWIZZLE_64B);
    else
        ok = make_map(ctx, &map_a, A, ELT, p.M, p.K, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (BMAJ == BMajor::K)   // B stored [N, K]
        ok = ok && make_map(ctx, &map_b, B, ELT, p.N, p.K, BK, BN, CU_TENSOR_MAP_SWIZZLE_128B);
    else                     // B stored [K, N]
        ok = ok && make_map(ctx, &map_b, B, ELT, p.K, p.N, 128 / ELT, BK, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return SSTE_ERR_CUDA;
    auto kern = gemm_kernel<SPARSE, BMAJ, ELT, BN, OUT_T, OUT_F32>;
    static bool attr_set = false;   // per instantiation
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
            return SSTE_ERR_CUDA;
        attr_set = true;
    }
    const int m_tiles = p.M / BM, n_tiles = (p.N + BN - 1) / BN;
    int grid = m_tiles * n_tiles;
    if (grid > ctx->sm_count) grid = ctx->sm_count;
    kern<<<grid, GEMM_THREADS, C::SMEM_BYTES, stream>>>(map_a, map_b, p);
    return cudaGetLastError() == cudaSuccess ? SSTE_OK : SSTE_ERR_CUDA;
}

bool fmt_code(sste_dtype dt, int *elt, uint32_t *code)
{
    switch (dt) {
    case SSTE_BF16: *elt = 2; *code = 1; return true;   // kind::f16: 1 = bf16
    case SSTE_E4M3: *elt = 1; *code = 0; return true;   // kind::f8f6f4: 0 = e4m3
    case SSTE_E5M2: *elt = 1; *code = 1; return true;   //               1 = e5m2
    default: return false;
    }
}

// dispatch on output dtype
template <bool SPARSE, BMajor BMAJ, int ELT, int BN, bool OUT_T>
sste_status launch_out(const sste_ctx *ctx, const void *A, const void *B, const GemmParams &p, sste_dtype odt,
                       cudaStream_t s)
{
    if (odt == SSTE_F32) return launch<SPARSE, BMAJ, ELT, BN, OUT_T, true>(ctx, A, B, p, s);
    if (odt == SSTE_BF16) return launch<SPARSE, BMAJ, ELT, BN, OUT_T, false>(ctx, A, B, p, s);
    return SSTE_ERR_DTYPE;
}

}  // namespace

sste_status sste_gemm_launch_check(const sste_ctx *) { return SSTE_OK; }

extern "C" sste_status sste_linear_fwd(sste_ctx *ctx, const void *X, int T, const void *vals, const void *meta, int O,
                                       int I, sste_dtype opdt, const float *out_scale_dev, void *Y, sste_dtype ydt,
                                       void *stream)
{
    if (!ctx || !X || !vals || !meta || !Y) return SSTE_ERR_INVALID_ARG;
    int elt;
    uint32_t code;
    if (!fmt_code(opdt, &elt, &code) || opdt == SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (ydt != SSTE_BF16 && ydt != SSTE_F32) return SSTE_ERR_DTYPE;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(X, 128) || !sste_aligned(vals, 128) || !sste_aligned(meta, 128) || !sste_aligned(Y, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    // Z^T[O, T] = S(W)[O, I] X^T: M = O, N = T, K = I; the output is stored transposed as Y[T, O]
    GemmParams p{O, T, I, static_cast<const uint8_t *>(meta), Y, out_scale_dev, ctx->status_dev, code, code};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (elt == 2) return launch_out<true, BMajor::K, 2, 256, true>(ctx, vals, X, p, ydt, s);
    return launch_out<true, BMajor::K, 1, 256, true>(ctx, vals, X, p, ydt, s);
}

extern "C" sste_status sste_linear_bwd_weight(sste_ctx *ctx, const void *gvals, const void *gmeta, int O, int T,
                                              sste_dtype gdt, const void *X, int I, sste_dtype xdt,
                                              const float *out_scale_dev, void *dW, sste_dtype dwdt, void *stream)
{
    if (!ctx || !gvals || !gmeta || !X || !dW) return SSTE_ERR_INVALID_ARG;
    int ea, eb;
    uint32_t ca, cb;
    if (!fmt_code(gdt, &ea, &ca) || !fmt_code(xdt, &eb, &cb) || ea != eb) return SSTE_ERR_DTYPE;
    if (gdt == SSTE_E4M3 || xdt == SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (dwdt != SSTE_BF16 && dwdt != SSTE_F32) return SSTE_ERR_DTYPE;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(X, 128) || !sste_aligned(gvals, 128) || !sste_aligned(gmeta, 128) || !sste_aligned(dW, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    // grad_W[O, I] = G[O, T] X[T, I]: M = O, N = I, K = T; X is [K, N] row-major = MN-major B
    GemmParams p{O, I, T, static_cast<const uint8_t *>(gmeta), dW, out_scale_dev, ctx->status_dev, ca, cb};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (ea == 2) return launch_out<true, BMajor::MN, 2, 256, false>(ctx, gvals, X, p, dwdt, s);
    return launch_out<true, BMajor::MN, 1, 256, false>(ctx, gvals, X, p, dwdt, s);
}

extern "C" sste_status sste_linear_bwd_input(sste_ctx *ctx, const void *dY, int T, int O, sste_dtype gdt,
                                             const void *Wt_dense, int I, sste_dtype wdt,
                                             const float *out_scale_dev, void *dX, sste_dtype xdt, void *stream)
{
    if (!ctx || !dY || !Wt_dense || !dX) return SSTE_ERR_INVALID_ARG;
    int ea, eb;
    uint32_t ca, cb;
    if (!fmt_code(gdt, &ea, &ca) || !fmt_code(wdt, &eb, &cb) || ea != eb) return SSTE_ERR_DTYPE;
    if (gdt == SSTE_E4M3 || wdt == SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (xdt != SSTE_BF16 && xdt != SSTE_F32) return SSTE_ERR_DTYPE;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(dY, 128) || !sste_aligned(Wt_dense, 128) || !sste_aligned(dX, 128)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    // grad_X[T, I] = grad_Z[T, O] S(W)[O, I]: M = T, N = I, K = O; S(W) is [K, N] row-major = MN-major B
    GemmParams p{T, I, O, nullptr, dX, out_scale_dev, ctx->status_dev, ca, cb};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (ea == 2) return launch_out<false, BMajor::MN, 2, 256, false>(ctx, dY, Wt_dense, p, xdt, s);
    return launch_out<false, BMajor::MN, 1, 256, false>(ctx, dY, Wt_dense, p, xdt, s);
}
