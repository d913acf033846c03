// Tensor-core products of the S-STE linear layer (Sec. 5.1) for sm_100a:
//   forward      Z^T = S(W) X^T              sparse A (values + metadata), K-major B
//   grad weight  grad_W = MVUE(grad_Z^T) X   sparse A, MN-major B
//   grad input   grad_X = grad_Z S(W)        dense A, MN-major B
//
// One persistent, warp-specialised kernel template run by CTA PAIRS (cluster of two,
// tcgen05 cta_group::2).  A pair owns a 256 x 256 output tile: each CTA holds its own
// 128 rows of A and HALF of the B tile, so the B operand is streamed from shared memory
// at half the rate per SM -- with one CTA per tile the sparse instruction is bound by that
// stream and runs no faster than the dense one -- and L2 -> SM traffic per flop drops.
//   warp 0    TMA producer (both CTAs; all transaction bytes land on the leader's barrier)
//   warp 1    leader CTA: tcgen05.mma[.sp] issue; both CTAs: tensor-memory allocation
//   warps 2-5 epilogue: TMEM -> registers -> bf16 -> shared memory -> TMA store
//   warps 6-9 sparse A: metadata HBM -> registers -> tensor memory (tcgen05.st), so that no
//             metadata copy sits between two MMAs in the tensor pipe (a tcgen05.cp there drains it);
//             compressed B (grad_X from the forward's operand): expansion of values + metadata
//             into the dense shared-memory stage
// Output tiles are handed out band by band (tile_coords) so that operands are read from HBM about
// once; tile width, split-K plan and band height come from cost models on the host (make_plan).
// Every wait is bounded: on expiry the CTA records SSTE_ERR_TIMEOUT and leaves.
#include <cuda.h>

#include <mutex>
#include <type_traits>

#include "common.cuh"

namespace {

constexpr int BM = 128;            // rows of A per CTA (a pair covers 256)
constexpr int TMEM_COLS = 512;
constexpr int STAGING_BYTES = 32768;   // two epilogue panels of 128 x 64 bf16
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // two seconds of wall time (%globaltimer)

enum class BMajor { K, MN };

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// arrive on a barrier that may live in the peer CTA (shared::cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// One try: the thread is suspended by the hardware until the phase completes or a time limit of
// about a millisecond passes, so a waiting thread does not poll shared memory (the sparse MMA streams
// its operands at 3/4 of the shared-memory bandwidth and is slowed down by pollers).
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(1000000u)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait of ONE thread.  Returns false (after recording a timeout) instead of spinning forever.
// The limit is wall time (nanoseconds of %globaltimer), so it does not depend on the SM clock.
struct WaitCtx {
    unsigned int *status;              // the context's device status word
    volatile int *abort_flag;          // this CTA's "a wait has expired" flag (shared memory)
    unsigned long long limit_ns;       // WAIT_LIMIT_NS, or the short limit of the stall-injection test hook
};
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx &wc)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long start = global_ns();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*wc.abort_flag) return false;
        if (global_ns() - start > wc.limit_ns) {
            atomicCAS(wc.status, 0u, static_cast<unsigned int>(SSTE_ERR_TIMEOUT));
            *wc.abort_flag = 1;
            return false;
        }
    }
}
// Bounded wait of a whole warp: lane 0 waits, the others park at the warp barrier.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const WaitCtx &wc)
{
    uint32_t ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, wc) ? 1u : 0u;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}

// 2-D tiled TMA load into this CTA's shared memory; the transaction bytes are signalled on
// `bar`, which may be the pair leader's barrier (cta_group::2 form).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// Barrier of the 128 epilogue threads that also combines a flag: true only if every thread passed true.
// The four epilogue warps wait for an accumulator separately; they must leave TOGETHER when one wait
// expired, or the others would park at the next epilogue barrier for good.
__device__ __forceinline__ bool epilogue_all(bool ok)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, 128, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(ok ? 1u : 0u)
        : "memory");
    return r != 0;
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair once every
// tcgen05 operation issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(static_cast<uint16_t>(3))
        : "memory");
}
template <bool F8>
__device__ __forceinline__ void tc_mma_dense(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    if (F8)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
template <bool F8>
__device__ __forceinline__ void tc_mma_sparse(uint32_t d, uint64_t a, uint64_t b, uint32_t e, uint32_t idesc,
                                              uint32_t accumulate)
{
    if (F8)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "tcgen05.mma.sp.cta_group::2.kind::f8f6f4 [%0], %1, %2, [%3], %4, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(e), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
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
// M is 256: the pair's two 128-row halves.
__host__ __device__ constexpr uint32_t instr_desc(bool sparse, uint32_t afmt, uint32_t bfmt, bool b_mn_major, int bn)
{
    return (sparse ? 4u : 0u) | (1u << 4) | (afmt << 7) | (bfmt << 10) | ((b_mn_major ? 1u : 0u) << 16) |
           (static_cast<uint32_t>(bn >> 3) << 17) | (static_cast<uint32_t>((2 * BM) >> 4) << 24);
}

// ------------------------------------------------------------------ kernel

// Order in which output tiles are handed to the CTA pairs (pair p takes tiles p, p + pairs, ...).  Tiles are
// numbered band by band: a band is `group_m` consecutive rows of tiles, and inside a band the row index runs
// fastest.  The 74 tiles in flight at any time therefore cover group_m tile rows x 74 / group_m tile columns,
// and the A rows of a band stay in L2 while the band sweeps over all of B.  group_m = m_tiles is plain
// column-major order (all of A resident, B streamed once).
__host__ __device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, int group_m, int &mt, int &nt)
{
    const int per_band = group_m * n_tiles;
    const int band = tile / per_band;
    const int first = band * group_m;
    const int rows = (m_tiles - first < group_m) ? (m_tiles - first) : group_m;
    const int within = tile - band * per_band;
    mt = first + within % rows;
    nt = within / rows;
}

struct GemmParams {
    int M, N, K;            // logical problem: D[M, N] = A[M, K] * B
    void *D;                // output (used by the direct-store fp32 epilogue)
    // FP8 operands (Sec. 5.2): device scalars max|a|, max|b| of the tensors the operands were quantised from and the
    // largest finite value of each operand's format; the epilogue multiplies by 1/scale_a * 1/scale_b.  Null for bf16.
    const float *a_amax, *b_amax;
    float a_fp8_max, b_fp8_max;
    unsigned int *out_amax; // nullable: receives max|D| (bit pattern of a non-negative fp32) by atomic maximum
    unsigned int *status;
    uint32_t afmt, bfmt;    // operand format codes of the instruction descriptor
    const uint8_t *b_vals;  // compressed-B kernels: the 2:4 values of B [K, N/2]; its metadata image is `meta`
    unsigned long long wait_limit_ns;   // limit of every device-side wait
    int skip_last_stage;    // stall-injection test hook: the producer leaves the last K stage of the launch unloaded
    int group_m;            // tile rows per band of the tile order (see tile_coords)
    int splits;             // split-K factor of the tiles from `split_from` on (1 = none)
    int split_from;         // first split tile: tiles below it are computed whole
    float *partials;        // split-K: fp32 partial tiles [tile][cta][split][128][BN], summed by splitk_reduce_kernel
};

// 32 lanes x 16 consecutive 32-bit columns <- 16 registers per thread (four metadata atoms in one instruction)
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint4 (&v)[4])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0].x), "r"(v[0].y), "r"(v[0].z), "r"(v[0].w), "r"(v[1].x), "r"(v[1].y), "r"(v[1].z),
          "r"(v[1].w), "r"(v[2].x), "r"(v[2].y), "r"(v[2].z), "r"(v[2].w), "r"(v[3].x), "r"(v[3].y), "r"(v[3].z),
          "r"(v[3].w)
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory / tensor-memory plan of one CTA for a tile of 256 x BN.  A stage holds 128 bytes of K per
// A row and, for the sparse kernels, two B sub-tiles of 128 bytes of K each (the compressed A row covers
// twice the K of one B row); the dense kernel pairs it with one B sub-tile.  A sparse tile of BN = 256
// leaves room for one accumulator buffer beside the metadata regions in the 512 tensor-memory columns;
// BN <= 192, and every dense tile, has two, so the epilogue of a tile overlaps the next tile's main loop.
template <bool SPARSE, int BN, bool BCOMP = false>
struct Cfg {
    static constexpr int A_STAGE = 16384;                        // 128 rows x 128 bytes
    static constexpr int B_SUB = (BN / 2) * 128;                 // this CTA's half of one B sub-tile
    static constexpr int B_STAGE = SPARSE ? 2 * B_SUB : B_SUB;
    static constexpr int STAGE = A_STAGE + B_STAGE;
    static constexpr int FIT = (232448 - 1024 - 512 - STAGING_BYTES) / STAGE;   // 227 KB of shared memory per CTA
    static constexpr int STAGES = FIT > 8 ? 8 : FIT;
    static constexpr int ACC_BUFS = (!SPARSE || BN <= 224) ? 2 : 1;   // the dense kernel keeps no metadata in TMEM
    static constexpr int META_COL0 = ACC_BUFS * BN;              // metadata regions follow the accumulators
    static constexpr int META_FIT = (TMEM_COLS - META_COL0) / 16;
    static constexpr int META_REGIONS = !SPARSE ? 1 : (META_FIT > 8 ? 8 : META_FIT);   // regions of 16 columns (four atoms)
    static constexpr int THREADS = (SPARSE || BCOMP) ? 320 : 192;     // + 4 metadata (sparse A) or expander (compressed B) warps
    static constexpr int PANEL = (BN % 64 == 0) ? 64 : 32;       // columns per epilogue panel (one TMA store)
    static constexpr int SMEM_BYTES = STAGES * STAGE + STAGING_BYTES + 1024 /* alignment slack */ + 512 /* barriers */;
    static_assert(META_COL0 + (SPARSE ? META_REGIONS * 16 : 0) <= TMEM_COLS, "tensor memory budget");
    static_assert(!SPARSE || META_REGIONS >= 4, "metadata regions");
    static_assert(STAGES >= 3, "pipeline depth");
};

// ELT: operand element size in bytes (2 = bf16 via kind::f16, 1 = fp8 via kind::f8f6f4).
// OUT_T: store D transposed (out[n, m]); OUT_F32: fp32 output (direct stores) instead of bf16 (TMA stores).
// BCOMP: the (dense-product) B operand is given in compressed 2:4 form and expanded in shared memory.
template <bool SPARSE, BMajor BMAJ, int ELT, int BN, bool OUT_T, bool OUT_F32, bool BCOMP = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Cfg<SPARSE, BN, BCOMP>::THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_p,
            const uint8_t *__restrict__ meta, const GemmParams p)
{
    sste_pdl_trigger();
    using C = Cfg<SPARSE, BN, BCOMP>;
    constexpr int META_REGIONS = C::META_REGIONS;
    constexpr int NS = C::STAGES;
    constexpr int NB = C::ACC_BUFS;
    constexpr bool F8 = (ELT == 1);
    constexpr int BK = (SPARSE ? 256 : 128) / ELT;    // logical K per stage
    constexpr int B_SUBS = SPARSE ? 2 : 1;
    constexpr int SUB_K = 128 / ELT;                  // logical K of one B sub-tile
    constexpr int ATOMS_PER_STAGE = SPARSE ? BK / 128 : 1;   // metadata atoms (128 logical K) per stage
    constexpr int B_CHUNK_N = 128 / ELT;              // MN-major: N elements per 128-byte row
    constexpr int B_CHUNKS_HALF = (BN / 2) / B_CHUNK_N;
    constexpr uint32_t STAGE_TX = 2u * (BCOMP ? C::A_STAGE : C::STAGE);   // both CTAs' bytes that arrive by TMA
    constexpr int PANEL = C::PANEL;                   // the epilogue works in panels of 64 (or 32) columns
    constexpr int DIRECT_PANELS = (BN - 128) / PANEL; // the last 128 columns go through registers (early release)
    static_assert(BMAJ == BMajor::K || (BN / 2) % B_CHUNK_N == 0, "MN-major B needs whole 128-byte chunks per CTA");
    static_assert(PANEL == 64 || (OUT_T && !OUT_F32), "32-column panels exist for the transposed bf16 store only");
    static_assert(!BCOMP || (!SPARSE && BMAJ == BMajor::MN), "compressed B: dense A, MN-major B");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging = smem_base + NS * C::STAGE;
    const uint32_t bars = staging + STAGING_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };              // used in the leader only
    auto empty_bar = [&](int s) { return bars + 8u * (NS + s); };      // one per CTA
    auto acc_full_bar = [&](int b) { return bars + 8u * (2 * NS + b); };           // one per CTA
    auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * NS + 2 + b); };      // leader only, 2 arrivals
    auto meta_full_bar = [&](int r) { return bars + 8u * (2 * NS + 4 + r); };             // leader only, 8 arrivals
    auto meta_empty_bar = [&](int r) { return bars + 8u * (2 * NS + 4 + META_REGIONS + r); };   // one per CTA
    constexpr int MISC = 2 * NS + 4 + 2 * META_REGIONS;
    const uint32_t tmem_slot = bars + 8u * MISC;
    uint8_t *bars_generic = smem_raw + (bars - smem_u32(smem_raw));
    volatile uint32_t *tmem_slot_ptr = reinterpret_cast<volatile uint32_t *>(bars_generic + 8u * MISC);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_generic + 8u * (MISC + 1));
    uint8_t *staging_generic = smem_raw + (staging - smem_u32(smem_raw));
    static_assert(8 * (MISC + 2) + 64 <= 512, "barrier block (+ the expander's 16-entry selector table)");
    const WaitCtx wc{p.status, abort_flag, p.wait_limit_ns};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = (rank == 0);
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int m_tiles = (p.M + 2 * BM - 1) / (2 * BM);
    const int n_tiles = (p.N + BN - 1) / BN;
    const int num_tiles = m_tiles * n_tiles;
    const int k_blocks_total = (p.K + BK - 1) / BK;   // a ragged last stage reads zero-filled K
    // Work units: tiles [0, split_from) are whole; every later tile is cut into `splits` K ranges (the
    // host makes the division exact).  Whole tiles fill complete waves, the split ones spread the
    // last, partial wave over all pairs.
    const int num_units = p.split_from + (num_tiles - p.split_from) * p.splits;
    struct Unit { int tile, split, k_blocks; };
    auto decode = [&](int unit) {
        Unit u;
        if (unit < p.split_from) { u.tile = unit; u.split = 0; u.k_blocks = k_blocks_total; }
        else {
            const int v = unit - p.split_from;
            u.tile = p.split_from + v / p.splits;
            u.split = v % p.splits;
            u.k_blocks = k_blocks_total / p.splits;
        }
        return u;
    };
    const int k_atoms = p.K / 128;

    if (threadIdx.x == 0) {
        // full: the producer's arrival with the TMA byte count (+ the eight expander warps of the pair)
        for (int s = 0; s < NS; ++s) { mbar_init(full_bar(s), BCOMP ? 9 : 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 2); }
        for (int r = 0; r < META_REGIONS; ++r) { mbar_init(meta_full_bar(r), 8); mbar_init(meta_empty_bar(r), 1); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_a);
        if (!BCOMP) prefetch_tensormap(&map_b);
        if (!OUT_F32) prefetch_tensormap(&map_d);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();          // the peer's barriers are initialised before anything signals them
    tc_fence_after();
    sste_pdl_wait();         // everything above overlapped the previous kernel; global memory from here on
    const uint32_t tmem_base = *tmem_slot_ptr;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int unit = pair; unit < num_units && ok; unit += num_pairs) {
                const Unit u = decode(unit);
                const int tile = u.tile, k_blocks = u.k_blocks, kb0 = u.split * u.k_blocks;
                int mt, nt;
                tile_coords(tile, m_tiles, n_tiles, p.group_m, mt, nt);
                const int m0 = mt * 2 * BM + static_cast<int>(rank) * BM;      // this CTA's rows of A
                const int n0 = nt * BN + static_cast<int>(rank) * (BN / 2);    // this CTA's half of B
                for (int kb = kb0; kb < kb0 + k_blocks; ++kb, ++it) {
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1u;
                    // test hook: the stage is never loaded nor announced, so the MMA warp's wait for it runs out
                    if (p.skip_last_stage && unit + num_pairs >= num_units && kb == kb0 + k_blocks - 1) break;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, wc)) { ok = false; break; }
                    const uint32_t lead_full = map_to_cta(full_bar(s), 0);
                    if (leader) mbar_arrive_expect_tx(full_bar(s), STAGE_TX);
                    const uint32_t a_dst = smem_base + s * C::STAGE;
                    const uint32_t b_dst = a_dst + C::A_STAGE;
                    // A: 128 bytes per row = BK/2 compressed (sparse) or BK dense elements
                    tma_load_2d(a_dst, &map_a, lead_full, kb * (SPARSE ? BK / 2 : BK), m0);
                    if (BCOMP) {
                        // B is written into the stage by the expander warps
                    } else if (BMAJ == BMajor::K) {
#pragma unroll
                        for (int u = 0; u < B_SUBS; ++u)
                            tma_load_2d(b_dst + u * C::B_SUB, &map_b, lead_full, kb * BK + u * SUB_K, n0);
                    } else {
                        // MN-major: one box per 128-byte N chunk spans the whole stage's K rows
#pragma unroll
                        for (int c = 0; c < B_CHUNKS_HALF; ++c)
                            tma_load_2d(b_dst + c * (BK * 128), &map_b, lead_full, n0 + c * B_CHUNK_N, kb * BK);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader && lane == 0) {
            const uint32_t idesc = instr_desc(SPARSE, p.afmt, p.bfmt, BMAJ == BMajor::MN, BN);
            uint32_t it = 0, local_tile = 0, group_it = 0;
            bool ok = true;
            for (int unit = pair; unit < num_units && ok; unit += num_pairs, ++local_tile) {
                const int k_blocks = decode(unit).k_blocks;
                const uint32_t buf = local_tile % NB, use = local_tile / NB;
                if (!mbar_wait(acc_empty_bar(buf), (use & 1u) ^ 1u, wc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {     // stage index inside the unit's K range
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1u;
                    uint32_t meta_cols = 0;
                    if (SPARSE) {
                        // metadata groups of four atoms rotate over META_REGIONS tensor-memory regions,
                        // written by the metadata warps of both CTAs
                        const int atom0 = kb * ATOMS_PER_STAGE;
                        const uint32_t region = group_it % META_REGIONS;
                        if ((atom0 & 3) == 0 &&
                            !mbar_wait(meta_full_bar(region), (group_it / META_REGIONS) & 1u, wc)) {
                            ok = false;
                            break;
                        }
                        meta_cols = tmem_base + C::META_COL0 + 16 * region + 4 * (atom0 & 3);
                    }
                    if (!mbar_wait(full_bar(s), ph, wc)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = smem_base + s * C::STAGE;
                    const uint32_t b_src = a_src + C::A_STAGE;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint64_t adesc = smem_desc(a_src + 32 * j, 16, 1024, 2);
                        uint64_t bdesc;
                        if (BMAJ == BMajor::K) {
                            bdesc = SPARSE ? smem_desc(b_src + (j >> 1) * C::B_SUB + 64 * (j & 1), 16, 1024, 2)
                                           : smem_desc(b_src + 32 * j, 16, 1024, 2);
                        } else {
                            constexpr int ROWS_PER_MMA = BK / 4;     // K rows of 128 bytes per instruction
                            bdesc = smem_desc(b_src + ROWS_PER_MMA * 128 * j, BK * 128, 1024, 2);
                        }
                        const uint32_t acc = (kb > 0 || j > 0) ? 1u : 0u;
                        if (SPARSE) {
                            // bf16: one 32-bit metadata column per instruction, the column pair is addressed and
                            // the descriptor's sparse selector picks the column; fp8: two columns per instruction
                            const uint32_t e = meta_cols + (F8 ? 2 * j : (j & 2));
                            const uint32_t id2 = F8 ? 0u : static_cast<uint32_t>(j & 1);
                            tc_mma_sparse<F8>(d_tmem, adesc, bdesc, e, idesc | id2, acc);
                        } else {
                            tc_mma_dense<F8>(d_tmem, adesc, bdesc, idesc, acc);
                        }
                    }
                    tc_commit_pair(empty_bar(s));     // frees the stage in both CTAs once these MMAs have read it
                    if (SPARSE) {
                        const int atom_end = (kb + 1) * ATOMS_PER_STAGE;
                        if ((atom_end & 3) == 0 || kb == k_blocks - 1) {
                            tc_commit_pair(meta_empty_bar(group_it % META_REGIONS));
                            ++group_it;
                        }
                    }
                }
                if (ok) tc_commit_pair(acc_full_bar(buf));
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int quarter = warp & 3;                  // tensor-memory lanes [32*quarter, 32*quarter + 32)
        const int row = quarter * 32 + lane;           // row of this CTA's 128 x BN accumulator
        const float scale = sste_out_scale(p.a_amax, p.a_fp8_max, p.b_amax, p.b_fp8_max);
        const bool want_amax = (p.out_amax != nullptr);
        const bool plain = !want_amax && scale == 1.0f;
        uint32_t amax2 = 0;                            // bf16 output: running max of the magnitude bits, two lanes of 16
        float amaxf = 0.0f;                            // fp32 output
        const bool store_thread = (threadIdx.x == 64);
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        uint32_t local_tile = 0, panel_it = 0;
        bool ok = true;
        for (int unit = pair; unit < num_units && ok; unit += num_pairs, ++local_tile) {
            const Unit u = decode(unit);
            const int tile = u.tile, split = u.split;
            int mt, nt;
            tile_coords(tile, m_tiles, n_tiles, p.group_m, mt, nt);
            const int m0 = mt * 2 * BM + static_cast<int>(rank) * BM;
            const int n0 = nt * BN;
            const uint32_t buf = local_tile % NB, use = local_tile / NB;
            const uint32_t acc_base = lane_base + buf * BN;
            const uint32_t lead_acc_empty = map_to_cta(acc_empty_bar(buf), 0);
            if (!epilogue_all(mbar_wait_warp(acc_full_bar(buf), use & 1u, wc))) { ok = false; break; }
            tc_fence_after();
            if (OUT_F32) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_32x32(acc_base + c0, r);
                    tmem_ld_wait();
                    const int m = m0 + row;
                    if (m < p.M && n0 + c0 < p.N) {
                        float v[32];
#pragma unroll
                        for (int c = 0; c < 32; ++c) v[c] = __fmul_rn(__uint_as_float(r[c]), scale);
                        if (want_amax) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) amaxf = fmaxf(amaxf, fabsf(v[c]));
                        }
                        if (OUT_T) {
                            float *out = static_cast<float *>(p.D);
#pragma unroll
                            for (int c = 0; c < 32; ++c) out[static_cast<size_t>(n0 + c0 + c) * p.M + m] = v[c];
                        } else {
                            float4 *out = reinterpret_cast<float4 *>(static_cast<float *>(p.D) +
                                                                     static_cast<size_t>(m) * p.N + n0 + c0);
#pragma unroll
                            for (int c = 0; c < 8; ++c) out[c] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                        }
                    }
                }
                tc_fence_before();
                epilogue_barrier();
                if (store_thread) mbar_arrive_cluster(lead_acc_empty);
                continue;
            }
            if (unit >= p.split_from && p.splits > 1) {
                // Split-K: the unit stores its fp32 partial tile [128][BN]; a second kernel adds the
                // partials of a tile in split order (bit-reproducible) and writes the bf16 result.
                // Panels of 32 fp32 columns (128-byte rows, swizzled) go out through the staging buffers and
                // TMA stores: whole lines instead of 16-byte pieces of 32 different rows per instruction.
                const int part_row0 =
                    static_cast<int>(((static_cast<size_t>(tile - p.split_from) * 2 + rank) * p.splits + split) * BM);
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    if (store_thread) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    epilogue_barrier();
                    const uint32_t off = (panel_it & 1u) * 16384u;
                    uint32_t r[32];
                    tmem_ld_32x32(acc_base + c0, r);
                    tmem_ld_wait();
                    uint8_t *dst = staging_generic + off + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4 *>(dst + ((c ^ (row & 7)) << 4)) = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
                    fence_proxy_async();
                    epilogue_barrier();
                    if (store_thread) {
                        tma_store_2d(&map_p, staging + off, c0, part_row0);
                        tma_store_commit();
                    }
                    ++panel_it;
                }
                tc_fence_before();
                epilogue_barrier();
                if (store_thread) mbar_arrive_cluster(lead_acc_empty);
                continue;
            }
            // bf16 output in panels of PANEL columns through two 16 KB staging buffers and TMA stores.
            // 32 accumulator columns -> bf16 -> staging buffer `sb`, columns [c0, c0 + 32) of the panel
            // Two accumulator values -> one word of two bf16 (packed conversion).  PLAIN: unit scale and no amax
            // wanted (every bf16 product of the path): no multiply, no maximum.
            auto pack2 = [&](uint32_t a, uint32_t b, auto plain_tag) -> uint32_t {
                float lo = __uint_as_float(a), hi = __uint_as_float(b);
                if (!decltype(plain_tag)::value) {
                    lo = __fmul_rn(lo, scale);
                    hi = __fmul_rn(hi, scale);
                }
                const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
                const uint32_t w = *reinterpret_cast<const uint32_t *>(&v);
                if (!decltype(plain_tag)::value) amax2 = __vmaxu2(amax2, w & 0x7fff7fffu);
                return w;
            };
            auto stage_impl = [&](const uint32_t (&r)[32], uint8_t *sb, int c0, auto plain_tag) {
                if (OUT_T) {
                    // staging[n][m]: PANEL rows of 128 bf16; a warp writes 32 consecutive m per n
                    uint16_t *st = reinterpret_cast<uint16_t *>(sb);
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const uint32_t w = pack2(r[c], r[c + 1], plain_tag);
                        st[(c0 + c) * BM + row] = static_cast<uint16_t>(w);
                        st[(c0 + c + 1) * BM + row] = static_cast<uint16_t>(w >> 16);
                    }
                } else {
                    // [128 rows][64 bf16] with the 128-byte swizzle of the TMA store: 16-byte chunk index ^= row & 7
                    uint8_t *dst = sb + row * 128;
                    const int chunk0 = c0 >> 3;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) w[e] = pack2(r[8 * c + 2 * e], r[8 * c + 2 * e + 1], plain_tag);
                        *reinterpret_cast<uint4 *>(dst + (((chunk0 + c) ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            };
            auto stage_chunk = [&](const uint32_t (&r)[32], uint8_t *sb, int c0) {
                if (plain) stage_impl(r, sb, c0, std::true_type{});
                else stage_impl(r, sb, c0, std::false_type{});
            };
            // staging buffer of the next panel becomes writable once the store issued two panels ago has read it
            auto acquire_staging = [&]() -> uint32_t {
                if (store_thread) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                epilogue_barrier();
                return (panel_it & 1u) * 16384u;
            };
            auto store_panel = [&](uint32_t off, int panel) {
                fence_proxy_async();
                epilogue_barrier();
                if (store_thread) {
                    if (OUT_T) tma_store_2d(&map_d, staging + off, m0, n0 + PANEL * panel);
                    else tma_store_2d(&map_d, staging + off, n0 + PANEL * panel, m0);
                    tma_store_commit();
                }
                ++panel_it;
            };
#pragma unroll 1
            for (int pnl = 0; pnl < DIRECT_PANELS; ++pnl) {
                const uint32_t off = acquire_staging();
                uint32_t ra[32], rb[32];
                tmem_ld_32x32(acc_base + PANEL * pnl, ra);
                if (PANEL == 64) tmem_ld_32x32(acc_base + PANEL * pnl + 32, rb);
                tmem_ld_wait();
                stage_chunk(ra, staging_generic + off, 0);
                if (PANEL == 64) stage_chunk(rb, staging_generic + off, 32);
                store_panel(off, pnl);
            }
            // last 128 columns -> registers, then the accumulator buffer is free for the next tile
            uint32_t r0[32], r1[32], r2[32], r3[32];
            tmem_ld_32x32(acc_base + BN - 128, r0);
            tmem_ld_32x32(acc_base + BN - 96, r1);
            tmem_ld_32x32(acc_base + BN - 64, r2);
            tmem_ld_32x32(acc_base + BN - 32, r3);
            tmem_ld_wait();
            tc_fence_before();
            {
                const uint32_t off = acquire_staging();      // includes the barrier after everyone's loads
                if (store_thread) mbar_arrive_cluster(lead_acc_empty);
                stage_chunk(r0, staging_generic + off, 0);
                if (PANEL == 64) stage_chunk(r1, staging_generic + off, 32);
                store_panel(off, DIRECT_PANELS);
            }
            if (PANEL == 32) {
                const uint32_t off = acquire_staging();
                stage_chunk(r1, staging_generic + off, 0);
                store_panel(off, DIRECT_PANELS + 1);
            }
            {
                const uint32_t off = acquire_staging();
                stage_chunk(r2, staging_generic + off, 0);
                if (PANEL == 64) stage_chunk(r3, staging_generic + off, 32);
                store_panel(off, DIRECT_PANELS + (PANEL == 64 ? 1 : 2));
            }
            if (PANEL == 32) {
                const uint32_t off = acquire_staging();
                stage_chunk(r3, staging_generic + off, 0);
                store_panel(off, DIRECT_PANELS + 3);
            }
        }
        if (want_amax) {
            // max|D| of this warp's share, as the bits of a non-negative fp32 (they order like unsigned integers)
            uint32_t best = OUT_F32 ? __float_as_uint(amaxf) : (max(amax2 & 0xffffu, amax2 >> 16) << 16);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
            if (lane == 0 && best != 0) atomicMax(p.out_amax, best);
        }
        if (store_thread && !OUT_F32) tma_store_wait_all();
    } else if (SPARSE) {
        // ------------------------------------------------------------ metadata warps (6..9, both CTAs)
        // HBM -> registers -> tensor memory: lane L of an atom's image is exactly the 16 bytes the
        // instruction expects in tensor-memory lane L, four 32-bit columns per atom.
        // The loads run six groups (of four atoms) ahead of the stores, in registers: a group's round trip
        // to L2 / HBM is then off the path that feeds the MMA warp (with load -> store -> signal in sequence
        // per group, that latency, not the tensor pipe, set the pace of every sparse product; with three groups
        // in flight the 8-bit kinds, which consume two atoms per stage, were still paced by it).
        const int quarter = warp & 3;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + C::META_COL0;
        // loader cursor: (unit, first atom of the next group)
        int l_unit = pair, l_a0 = 0, l_end = 0;
        const uint4 *l_src = nullptr;
        bool l_rows = false;
        auto l_setup = [&]() {
            if (l_unit >= num_units) return;
            const Unit u = decode(l_unit);
            int mt, nt;
            tile_coords(u.tile, m_tiles, n_tiles, p.group_m, mt, nt);
            const int m0 = mt * 2 * BM + static_cast<int>(rank) * BM;
            l_rows = m0 < p.M;
            l_src = reinterpret_cast<const uint4 *>(meta + static_cast<size_t>(m0 / BM) * k_atoms * 2048) + quarter * 32 + lane;
            l_a0 = u.split * u.k_blocks * ATOMS_PER_STAGE;
            l_end = l_a0 + u.k_blocks * ATOMS_PER_STAGE;
        };
        auto l_issue = [&](uint4 (&v)[4]) -> bool {
            if (l_unit >= num_units) return false;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                v[i] = (l_rows && l_a0 + i < k_atoms) ? __ldg(l_src + static_cast<size_t>(l_a0 + i) * 128)
                                                      : make_uint4(0, 0, 0, 0);
            l_a0 += 4;
            if (l_a0 >= l_end) {
                l_unit += num_pairs;
                l_setup();
            }
            return true;
        };
        l_setup();
        // META_DEPTH groups of loads are in flight per lane (a ring of registers; the loop is unrolled over it):
        // a group must be on its way for several stages before its turn, or the round trip to L2 paces the warp
        constexpr int META_DEPTH = 6;
        uint4 q[META_DEPTH][4];
        bool have[META_DEPTH];
#pragma unroll
        for (int d = 0; d < META_DEPTH; ++d) have[d] = l_issue(q[d]);
        uint32_t group_it = 0;
        bool running = true;
        while (running) {
#pragma unroll
            for (int d = 0; d < META_DEPTH; ++d) {
                if (!running) break;
                if (!have[d]) { running = false; break; }
                const uint32_t region = group_it % META_REGIONS;
                if (!mbar_wait_warp(meta_empty_bar(region), ((group_it / META_REGIONS) & 1u) ^ 1u, wc)) { running = false; break; }
                tc_fence_after();
                tmem_st_32x16(lane_base + 16 * region, q[d]);      // one store for the group's four atoms
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(meta_full_bar(region), 0));
                ++group_it;
                have[d] = l_issue(q[d]);
            }
        }
    } else if (BCOMP) {
        // ------------------------------------------------------------ expander warps (6..9, both CTAs)
        // grad_X = grad_Z S(W) reads S(W) [O, I] as its MN-major B operand.  Here S(W) is given as the forward's
        // compressed operand (2:4 values + metadata image) and every stage's K rows are expanded into the shared-
        // memory image a TMA load of the dense matrix would have left: rows of 128 bytes of N, 16-byte chunks
        // XOR-swizzled with the row, +0 in the pruned positions.  A unit is 16 bytes of values (8 groups of fp8,
        // 4 of bf16) = 32 bytes of the dense row; the loads of the next stage are in flight while this one is
        // expanded.
        constexpr int SEGS = (BN / 2) * ELT / 32;          // units per K row of this CTA's half of the tile
        constexpr int UNITS = BK * SEGS / 128;             // units per thread and stage
        static_assert(!BCOMP || (BK * SEGS) % 128 == 0, "units per stage");
        const int t = static_cast<int>(threadIdx.x) - 192;
        // byte-permute selectors per metadata nibble p0 | p1 << 2: which source byte feeds each output byte
        // (4 = a zero byte).  bf16: low / high 16 bits select the two output words of a group from the pair word;
        // fp8: 16 bits select the output word of a group from its two value bytes (0, 1).
        uint32_t *lut = reinterpret_cast<uint32_t *>(bars_generic + 8u * (MISC + 2));
        if (t < 16) {
            const uint32_t p0 = t & 3, p1 = t >> 2;
            uint32_t sel = 0;
            for (uint32_t h = 0; h < 4; ++h) {
                if (F8) sel |= (h == p0 ? 0u : h == p1 ? 1u : 4u) << (4 * h);
                else sel |= (h == p0 ? 0x10u : h == p1 ? 0x32u : 0x44u) << (8 * h);
            }
            lut[t] = sel;
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        // A thread's units of a stage: the same 32-byte column segment `seg` of rows r0 + j * ROWS_STEP.
        constexpr int ROWS_STEP = 128 / SEGS;
        constexpr int EPU = 32 / ELT;                      // dense elements per unit
        const int seg = t % SEGS, r0 = t / SEGS;
        const size_t row_bytes = static_cast<size_t>(p.N / 2) * ELT;     // one row of compressed values
        const size_t atom_row_bytes = static_cast<size_t>(p.N / 128) * 2048;
        uint32_t moff[UNITS];                              // metadata byte of unit j inside its (half) atom
#pragma unroll
        for (int j = 0; j < UNITS; ++j) {
            const uint32_t m = static_cast<uint32_t>(r0 + j * ROWS_STEP), k = static_cast<uint32_t>(seg * EPU);
            moff[j] = F8 ? sste_meta_atom_byte8(m, k) : sste_meta_atom_byte16(m, k);
        }
        // loader cursor: (unit, stage) of the next loads
        int e_unit = pair, e_kb = 0, e_kend = 0;
        const uint8_t *e_vals = nullptr, *e_meta = nullptr;
        bool e_cols = false;
        auto e_setup = [&]() {
            if (e_unit >= num_units) return;
            const Unit u = decode(e_unit);
            int mt, nt;
            tile_coords(u.tile, m_tiles, n_tiles, p.group_m, mt, nt);
            const int n0 = nt * BN + static_cast<int>(rank) * (BN / 2);
            e_cols = n0 < p.N;
            e_vals = p.b_vals + (static_cast<size_t>(n0 / 2) + seg * (EPU / 2)) * ELT + r0 * row_bytes;
            e_meta = meta + static_cast<size_t>(n0 >> 7) * 2048;
            e_kb = u.split * u.k_blocks;
            e_kend = e_kb + u.k_blocks;
        };
        auto e_issue = [&](uint4 (&v)[UNITS], uint32_t (&m)[UNITS]) -> bool {
            if (e_unit >= num_units) return false;
            const uint32_t krow0 = static_cast<uint32_t>(e_kb) * BK;             // first K row of the stage
            const uint8_t *vp = e_vals + krow0 * row_bytes;
            const uint8_t *mp = e_meta + (krow0 >> 7) * atom_row_bytes + ((BK == 64 && (krow0 & 64u)) ? 1024u : 0u);
#pragma unroll
            for (int j = 0; j < UNITS; ++j) {
                if (e_cols) {
                    v[j] = __ldg(reinterpret_cast<const uint4 *>(vp + static_cast<size_t>(j) * ROWS_STEP * row_bytes));
                    if (F8) m[j] = __ldg(reinterpret_cast<const uint32_t *>(mp + moff[j]));
                    else m[j] = __ldg(reinterpret_cast<const uint16_t *>(mp + moff[j]));
                } else {
                    v[j] = make_uint4(0, 0, 0, 0);         // columns beyond N: zeros (any valid code will do)
                    m[j] = 0x44444444u;
                }
            }
            if (++e_kb >= e_kend) {
                e_unit += num_pairs;
                e_setup();
            }
            return true;
        };
        e_setup();
        // three stages of loads in flight in registers: a round trip to L2 is longer than two stages of MMAs
        uint4 v0[UNITS], v1[UNITS], v2[UNITS];
        uint32_t m0[UNITS], m1[UNITS], m2[UNITS];
        bool h0 = e_issue(v0, m0), h1 = e_issue(v1, m1), h2 = e_issue(v2, m2);
        uint32_t it = 0;
        uint8_t *const ring = smem_raw + (smem_base - smem_u32(smem_raw));
        while (h0) {
            const int s = it % NS;
            const uint32_t ph = (it / NS) & 1u;
            if (!mbar_wait_warp(empty_bar(s), ph ^ 1u, wc)) break;
            uint8_t *b_dst = ring + s * C::STAGE + C::A_STAGE + (seg >> 2) * (BK * 128);
            const int j0 = (seg & 3) * 2;
#pragma unroll
            for (int j = 0; j < UNITS; ++j) {
                const int r = r0 + j * ROWS_STEP;
                const uint32_t w[4] = {v0[j].x, v0[j].y, v0[j].z, v0[j].w};
                uint32_t o[8];
                if (F8) {
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const uint32_t pairw = (g & 1) ? (w[g >> 1] >> 16) : w[g >> 1];    // value bytes 0, 1
                        o[g] = __byte_perm(pairw, 0, lut[(m0[j] >> (4 * g)) & 0xfu]);
                    }
                } else {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const uint32_t sel = lut[(m0[j] >> (4 * g)) & 0xfu];
                        o[2 * g] = __byte_perm(w[g], 0, sel & 0xffffu);
                        o[2 * g + 1] = __byte_perm(w[g], 0, sel >> 16);
                    }
                }
                uint8_t *rowp = b_dst + r * 128;
                *reinterpret_cast<uint4 *>(rowp + ((j0 ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4 *>(rowp + (((j0 + 1) ^ (r & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
            }
            fence_proxy_async();        // the tensor core reads the stage through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(full_bar(s), 0));
#pragma unroll
            for (int j = 0; j < UNITS; ++j) { v0[j] = v1[j]; m0[j] = m1[j]; v1[j] = v2[j]; m1[j] = m2[j]; }
            h0 = h1;
            h1 = h2;
            h2 = e_issue(v2, m2);
            ++it;
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync();          // neither CTA frees tensor memory while the pair still uses it
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
    const CUtensorMapDataType dt = (elt == 4)   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                   : (elt == 2) ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                : CU_TENSOR_MAP_DATA_TYPE_UINT8;
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->cu_tensor_map_encode);
    return fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Split-K second pass over the split tiles: out[m, n] = bf16(scale * sum over splits, in split order, of
// the fp32 partial tiles [split tile][cta][split][128][bn]).  One thread per 8 consecutive n.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partials, int M, int N, int bn, int splits, int m_tiles, int n_tiles,
                     int group_m, int split_from,
                     int n_split_tiles, const float *__restrict__ a_amax, float a_fp8_max,
                     const float *__restrict__ b_amax, float b_fp8_max, unsigned int *__restrict__ out_amax,
                     uint4 *__restrict__ out)
{
    sste_pdl_trigger();
    const int vec_per_row = bn / 8;
    const size_t vecs = static_cast<size_t>(n_split_tiles) * 2 * BM * vec_per_row;
    sste_pdl_wait();
    const float scale = sste_out_scale(a_amax, a_fp8_max, b_amax, b_fp8_max);
    uint32_t amax2 = 0;
    for (size_t v = static_cast<size_t>(blockIdx.x) * 256 + threadIdx.x; v < vecs; v += static_cast<size_t>(gridDim.x) * 256) {
        const int col = static_cast<int>(v % vec_per_row) * 8;
        const int row = static_cast<int>((v / vec_per_row) % BM);
        const size_t slot = v / (static_cast<size_t>(vec_per_row) * BM);        // (split tile, cta)
        const int tile = split_from + static_cast<int>(slot >> 1);
        int mt, nt;
        tile_coords(tile, m_tiles, n_tiles, group_m, mt, nt);
        const int m = mt * 2 * BM + static_cast<int>(slot & 1) * BM + row;
        const int n = nt * bn + col;
        if (m >= M || n >= N) continue;
        const float *src = partials + (slot * splits * BM + row) * bn + col;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int s = 0; s < splits; ++s) {
            const float4 a = __ldcg(reinterpret_cast<const float4 *>(src + static_cast<size_t>(s) * BM * bn));
            const float4 b = __ldcg(reinterpret_cast<const float4 *>(src + static_cast<size_t>(s) * BM * bn) + 1);
            acc[0] = __fadd_rn(acc[0], a.x); acc[1] = __fadd_rn(acc[1], a.y); acc[2] = __fadd_rn(acc[2], a.z); acc[3] = __fadd_rn(acc[3], a.w);
            acc[4] = __fadd_rn(acc[4], b.x); acc[5] = __fadd_rn(acc[5], b.y); acc[6] = __fadd_rn(acc[6], b.z); acc[7] = __fadd_rn(acc[7], b.w);
        }
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            w[e] = sste_f32_to_bf16_bits(__fmul_rn(acc[2 * e], scale)) | (sste_f32_to_bf16_bits(__fmul_rn(acc[2 * e + 1], scale)) << 16);
        if (out_amax) {
#pragma unroll
            for (int e = 0; e < 4; ++e) amax2 = __vmaxu2(amax2, w[e] & 0x7fff7fffu);
        }
        out[(static_cast<size_t>(m) * N + n) / 8] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (out_amax) {
        uint32_t best = max(amax2 & 0xffffu, amax2 >> 16) << 16;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
        if ((threadIdx.x & 31) == 0 && best != 0) atomicMax(out_amax, best);
    }
}

// Runs `fn` once per device ordinal (and again after a failure); thread-safe.
struct DeviceOnce {
    static constexpr int MAX_DEVICES = 64;
    std::mutex mu;
    bool done[MAX_DEVICES] = {};
    template <typename F>
    bool run(int device, F fn)
    {
        if (device < 0 || device >= MAX_DEVICES) return fn();
        std::lock_guard<std::mutex> lock(mu);
        if (!done[device]) done[device] = fn();
        return done[device];
    }
};

int g_inject_stall = 0;   // test hook: see sste_debug_inject_stall
int g_force_group_m = 0;  // test hook: 0 = automatic band height of the tile order

// Band height of the tile order from the operand sizes (a_tile / b_tile: bytes of one tile row of A / one tile
// column of B over the whole reduction).  L2 is 126 MB; an operand that takes less than half of it stays
// resident whatever the order.
//   A small: plain column-major order (every pair of a wave shares a few columns of B, B is read once).
//   else:    bands of about sqrt(pairs * b_tile / a_tile) tile rows: a wave then loads the least bytes, the band's
//            A rows are read once while B, if it fits, stays in L2 across bands.
int pick_group_m(int m_tiles, int n_tiles, int pairs, double a_tile, double b_tile)
{
    if (g_force_group_m > 0) return g_force_group_m < m_tiles ? g_force_group_m : m_tiles;
    const double l2_budget = 56e6;
    if (a_tile * m_tiles <= l2_budget || m_tiles <= 1 || n_tiles <= 1) return m_tiles;
    double g = __builtin_sqrt(static_cast<double>(pairs) * b_tile / a_tile);
    int gm = static_cast<int>(g + 0.5);
    if (gm < 1) gm = 1;
    if (gm > m_tiles) gm = m_tiles;
    return gm;
}

struct SplitPlan { int splits, split_from; };
SplitPlan pick_split_plan(int sm_count, size_t partial_bytes, int tiles, int k_blocks, int align, int bn, double stage_us);

// Everything the host decides about one product launch of a given tile width (the width itself: pick_bn).
struct LaunchPlan { int splits, split_from, group_m; };
LaunchPlan make_plan(bool sparse, int elt, int bn, bool out_t, bool out_f32, bool bcomp, int sm_count,
                     size_t partial_bytes, int M, int N, int K)
{
    const int bk = (sparse ? 256 : 128) / elt;
    const int m_tiles = (M + 2 * BM - 1) / (2 * BM), n_tiles = (N + bn - 1) / bn, tiles = m_tiles * n_tiles;
    LaunchPlan plan{1, tiles, m_tiles};
    plan.group_m = pick_group_m(m_tiles, n_tiles, sm_count / 2,
                                static_cast<double>(K) * (sparse ? 0.5 * elt + 0.125 : 1.0 * elt) * 2 * BM,
                                static_cast<double>(K) * ((bcomp ? 0.5 : 1.0) * elt) * bn);
    if (!out_f32 && !out_t) {   // a stage takes about 790 clk (sparse) / 512 clk (dense) at 1.9 GHz
        const SplitPlan sp = pick_split_plan(sm_count, partial_bytes, tiles, (K + bk - 1) / bk, sparse ? 4 / (bk / 128) : 1,
                                             bn, sparse ? 0.42 : 0.27);
        plan.splits = sp.splits;
        plan.split_from = sp.split_from;
    }
    return plan;
}

template <bool SPARSE, BMajor BMAJ, int ELT, int BN, bool OUT_T, bool OUT_F32, bool BCOMP = false>
sste_status launch(const sste_ctx *ctx, const void *A, const void *B, const void *meta, const GemmParams &p,
                   cudaStream_t stream)
{
    using C = Cfg<SPARSE, BN, BCOMP>;
    constexpr int BK = (SPARSE ? 256 : 128) / ELT;
    CUtensorMap map_a, map_b, map_d, map_p;
    bool ok;
    if (SPARSE)   // compressed values [M, K/2]: 128 bytes per row per stage
        ok = make_map(ctx, &map_a, A, ELT, p.M, p.K / 2, BK / 2, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    else
        ok = make_map(ctx, &map_a, A, ELT, p.M, p.K, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (BCOMP)               // B is expanded from its compressed form by the kernel: no map
        map_b = map_a;
    else if (BMAJ == BMajor::K)   // B stored [N, K]: sub-tiles of BN/2 rows by 128 bytes of K
        ok = ok && make_map(ctx, &map_b, B, ELT, p.N, p.K, 128 / ELT, BN / 2, CU_TENSOR_MAP_SWIZZLE_128B);
    else                     // B stored [K, N]: chunks of 128 bytes of N by BK rows of K
        ok = ok && make_map(ctx, &map_b, B, ELT, p.K, p.N, 128 / ELT, BK, CU_TENSOR_MAP_SWIZZLE_128B);
    if (OUT_F32) {
        map_d = map_a;       // unused: the fp32 epilogue stores directly
    } else if (OUT_T) {      // out[N, M] bf16: panels of 128 m x 64 (or 32) n
        ok = ok && make_map(ctx, &map_d, p.D, 2, p.N, p.M, BM, C::PANEL, CU_TENSOR_MAP_SWIZZLE_NONE);
    } else {                 // out[M, N] bf16: panels of 64 n x 128 m, 128-byte swizzle
        ok = ok && make_map(ctx, &map_d, p.D, 2, p.M, p.N, 64, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    }
    if (!ok) return SSTE_ERR_CUDA;
    auto kern = gemm_kernel<SPARSE, BMAJ, ELT, BN, OUT_T, OUT_F32, BCOMP>;
    // The opt-in to more than 48 KB of dynamic shared memory is a per-DEVICE attribute of the kernel:
    // set once per (instantiation, device), under a lock (contexts may be used from several host threads).
    static DeviceOnce attr_done;
    if (!attr_done.run(ctx->device, [&] {
            return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) == cudaSuccess;
        }))
        return SSTE_ERR_CUDA;
    const int m_tiles = (p.M + 2 * BM - 1) / (2 * BM), n_tiles = (p.N + BN - 1) / BN;
    GemmParams pp = p;
    pp.wait_limit_ns = WAIT_LIMIT_NS;
    pp.skip_last_stage = 0;
    if (g_inject_stall) {
        // Test hook (sste_debug_inject_stall): only a dense product of ONE output tile takes the fault, so that
        // exactly one CTA pair runs into the expired wait; every other launch refuses while the hook is armed.
        if (SPARSE || BCOMP || OUT_F32 || m_tiles * n_tiles != 1) return SSTE_ERR_INVALID_ARG;
        pp.wait_limit_ns = 1000000ull;      // one millisecond
        pp.skip_last_stage = 1;
    }
    if (BCOMP) pp.b_vals = static_cast<const uint8_t *>(B);
    if (pp.out_amax && cudaMemsetAsync(pp.out_amax, 0, sizeof(unsigned int), stream) != cudaSuccess) return SSTE_ERR_CUDA;
    const int tiles = m_tiles * n_tiles;
    const LaunchPlan plan = make_plan(SPARSE, ELT, BN, OUT_T, OUT_F32, BCOMP, ctx->sm_count,
                                      ctx->splitk_partials ? ctx->splitk_partial_bytes : 0, p.M, p.N, p.K);
    pp.group_m = plan.group_m;
    pp.splits = plan.splits;
    pp.split_from = plan.split_from;
    pp.partials = ctx->splitk_partials;
    const int n_split_tiles = tiles - pp.split_from;
    int pairs = pp.split_from + n_split_tiles * pp.splits;
    if (pairs > ctx->sm_count / 2) pairs = ctx->sm_count / 2;
    map_p = map_a;   // unused without split-K
    if (pp.splits > 1 &&
        !make_map(ctx, &map_p, pp.partials, 4, static_cast<uint64_t>(n_split_tiles) * 2 * pp.splits * BM, BN, 32, BM,
                  CU_TENSOR_MAP_SWIZZLE_128B))
        return SSTE_ERR_CUDA;
    if (sste_launch(kern, dim3(2 * pairs), dim3(C::THREADS), C::SMEM_BYTES, stream, map_a, map_b, map_d, map_p,
                    static_cast<const uint8_t *>(meta), pp) != cudaSuccess)
        return SSTE_ERR_CUDA;
    if (pp.splits > 1) {
        const size_t vecs = static_cast<size_t>(n_split_tiles) * 2 * BM * (BN / 8);
        size_t blocks = (vecs + 255) / 256;
        if (blocks > static_cast<size_t>(ctx->sm_count) * 16) blocks = static_cast<size_t>(ctx->sm_count) * 16;
        if (sste_launch(splitk_reduce_kernel, dim3(static_cast<unsigned int>(blocks)), dim3(256), 0, stream,
                        pp.partials, p.M, p.N, BN, pp.splits, m_tiles, n_tiles, pp.group_m, pp.split_from, n_split_tiles, p.a_amax,
                        p.a_fp8_max, p.b_amax, p.b_fp8_max, pp.out_amax, static_cast<uint4 *>(p.D)) != cudaSuccess)
            return SSTE_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return SSTE_ERR_CUDA;
    sste_count_launches(pp.splits > 1 ? 2 : 1);
    return SSTE_OK;
}

int g_force_splits = 0;   // test hook: 0 = automatic split-K factor


// Split-K plan.  Tiles that fill complete waves of CTA pairs are computed whole; the tiles of the last,
// partial wave (all of them when there are fewer tiles than pairs, as for the weight gradient of a
// GPT-2-sized layer: 36 tiles, 74 pairs) are cut into `splits` K ranges so that the wave takes 1/splits
// of a tile time.  `align` = stages per metadata group (K ranges must start on a group boundary).
SplitPlan pick_split_plan(int sm_count, size_t partial_bytes, int tiles, int k_blocks, int align, int bn, double stage_us)
{
    SplitPlan none{1, tiles};
    if (partial_bytes == 0) return none;
    const int pairs = sm_count / 2;
    const int whole = (tiles / pairs) * pairs;
    const int tail = tiles - whole;
    if (tail == 0) return none;
    int best = 1;
    const double tile_us = k_blocks * stage_us;
    double best_cost = tile_us;        // time of the last wave, microseconds
    for (int s = 2; s <= 4; ++s) {
        if (k_blocks % (s * align) != 0 || k_blocks / s < 8) continue;
        if (static_cast<size_t>(tail) * 2 * s * BM * bn * sizeof(float) > partial_bytes) continue;
        if (g_force_splits == s) return SplitPlan{s, whole};
        const int waves = (tail * s + pairs - 1) / pairs;
        // + the second pass (a launch of its own) and the partial tiles' round trip through L2
        const double cost = tile_us * waves / s + 4.0 + 0.3 * s;
        if (cost < best_cost - 1e-9) { best = s; best_cost = cost; }
    }
    if (g_force_splits == 1 || best == 1) return none;
    return SplitPlan{best, whole};
}

// Tile width of the forward (K-major B), from timings on B200 over the GPT-2- and 7B-shaped layers.
// bf16: the time of a tile is close to  K * bn * k(bn) + f(bn)  microseconds with
//   bn = 192: k = 1.93e-5, f = 0.4;   224: k = 1.83e-5, f = 0.5;   256: k = 1.52e-5, f = 1.7
// (wider tiles stream less B per flop; the 256-wide tile has one accumulator, so its epilogue is exposed), and
// the launch takes ceil(tiles / pairs) such tile times: the width with the smallest product wins, which is
// mostly a matter of how the tile count quantises into waves.  FP8: 256 columns unless they quantise badly.
int pick_bn(bool b_k_major, int elt, int M, int N, int K, int pairs)
{
    if (!b_k_major) return 256;
    const long m_tiles = (M + 2 * BM - 1) / (2 * BM);
    auto waves = [&](int bn) { return (m_tiles * ((N + bn - 1) / bn) + pairs - 1) / pairs; };
    if (elt == 2) {
        const int widths[3] = {224, 192, 256};
        const double k[3] = {1.83e-5, 1.93e-5, 1.52e-5}, f[3] = {0.5, 0.4, 1.7};
        int best = 0;
        double best_cost = 0.0;
        for (int i = 0; i < 3; ++i) {
            const double cost = static_cast<double>(waves(widths[i])) * (static_cast<double>(K) * widths[i] * k[i] + f[i]);
            if (i == 0 || cost < best_cost * 0.995) { best = i; best_cost = cost; }
        }
        return widths[best];
    }
    if (K <= 1024) return 192;
    // Longer reductions: 256 columns unless the tile count quantises badly; a 192-wide tile costs about 8 %
    // more per flop (measured at many waves).
    return (waves(192) * 192 * 108 < waves(256) * 256 * 100) ? 192 : 256;
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

int g_force_bn = 0;   // test hook: 0 = automatic tile width

// Dispatch on tile width and output dtype.  fp32 output (a test / debug path) always uses 256-wide tiles.
template <bool SPARSE, BMajor BMAJ, int ELT, bool OUT_T>
sste_status launch_out(const sste_ctx *ctx, const void *A, const void *B, const void *meta, const GemmParams &p,
                       sste_dtype odt, cudaStream_t s)
{
    if (odt == SSTE_F32) return launch<SPARSE, BMAJ, ELT, 256, OUT_T, true>(ctx, A, B, meta, p, s);
    if (odt != SSTE_BF16) return SSTE_ERR_DTYPE;
    constexpr bool MN = (BMAJ == BMajor::MN);
    int cands[4], n = 0;
    cands[n++] = 256;
    if (!(MN && ELT == 1)) cands[n++] = 128;   // MN-major B: each CTA needs whole 128-byte chunks of N
    if (!MN) cands[n++] = 192;
    if (!MN && SPARSE && OUT_T) cands[n++] = 224;
    int bn = pick_bn(!MN, ELT, p.M, p.N, p.K, ctx->sm_count / 2);
    for (int i = 0; i < n; ++i)
        if (cands[i] == g_force_bn) bn = g_force_bn;
    if constexpr (!MN && SPARSE && OUT_T) {
        if (bn == 224) return launch<SPARSE, BMAJ, ELT, 224, OUT_T, false>(ctx, A, B, meta, p, s);
    }
    if constexpr (!MN) {
        if (bn == 192) return launch<SPARSE, BMAJ, ELT, 192, OUT_T, false>(ctx, A, B, meta, p, s);
    }
    if constexpr (!(MN && ELT == 1)) {
        if (bn == 128) return launch<SPARSE, BMAJ, ELT, 128, OUT_T, false>(ctx, A, B, meta, p, s);
    }
    return launch<SPARSE, BMAJ, ELT, 256, OUT_T, false>(ctx, A, B, meta, p, s);
}

// FP8 operands come with the amax of the tensors they were quantised from (both or neither); bf16 with none.
bool amax_args_ok(int elt, const float *a_amax, const float *b_amax)
{
    return elt == 1 ? (a_amax && b_amax) : (!a_amax && !b_amax);
}

}  // namespace

extern "C" sste_status sste_debug_force_splits(int splits)
{
    if (splits < 0 || splits > 4) return SSTE_ERR_INVALID_ARG;
    g_force_splits = splits;
    return SSTE_OK;
}
extern "C" sste_status sste_debug_plan(int product, sste_dtype opdt, int O, int I, int T, int sm_count,
                                       size_t workspace_bytes, int *tile_width, int *splits, int *split_from,
                                       int *group_m)
{
    int elt;
    uint32_t code;
    if (!fmt_code(opdt, &elt, &code) || product < 0 || product > 2 || sm_count < 2) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    // the (M, N, K) of the launch, as in the three entry points below
    const int M = product == 2 ? T : O, N = product == 0 ? T : I, K = product == 0 ? I : product == 1 ? T : O;
    const bool sparse = product != 2, mn = product != 0, out_t = product == 0;
    int bn = pick_bn(!mn, elt, M, N, K, sm_count / 2);
    const int cands[4] = {256, (mn && elt == 1) ? 0 : 128, mn ? 0 : 192, (!mn && sparse) ? 224 : 0};
    for (int c : cands)
        if (c && c == g_force_bn) bn = c;
    const size_t partial_bytes =
        workspace_bytes > SSTE_WS_SPLITK_PARTIALS_OFF + (size_t(1) << 20) ? workspace_bytes - SSTE_WS_SPLITK_PARTIALS_OFF : 0;
    const LaunchPlan plan = make_plan(sparse, elt, bn, out_t, false, false, sm_count, partial_bytes, M, N, K);
    if (tile_width) *tile_width = bn;
    if (splits) *splits = plan.splits;
    if (split_from) *split_from = plan.split_from;
    if (group_m) *group_m = plan.group_m;
    return SSTE_OK;
}
// Host-only self-check of the once-per-device guard the launches use for per-device kernel attributes: `fn` must
// run once per device ordinal, again after a failure, and never for a device that already succeeded.
extern "C" sste_status sste_debug_selftest_device_once(void)
{
    DeviceOnce once;
    int calls[4] = {0, 0, 0, 0};
    bool fail_next = true;
    auto fn = [&](int dev) {
        return once.run(dev, [&] {
            ++calls[dev];
            if (dev == 2 && fail_next) { fail_next = false; return false; }   // first attempt on device 2 fails
            return true;
        });
    };
    const bool r0 = fn(0), r0b = fn(0), r1 = fn(1), r2 = fn(2), r2b = fn(2), r2c = fn(2), r3 = fn(3), r1b = fn(1);
    const bool ok = r0 && r0b && r1 && !r2 && r2b && r2c && r3 && r1b && calls[0] == 1 && calls[1] == 1 &&
                    calls[2] == 2 && calls[3] == 1;
    return ok ? SSTE_OK : SSTE_ERR_INVALID_ARG;
}
extern "C" sste_status sste_debug_tile_coords(int tile, int m_tiles, int n_tiles, int group_m, int *mt, int *nt)
{
    if (tile < 0 || m_tiles <= 0 || n_tiles <= 0 || group_m <= 0 || tile >= m_tiles * n_tiles || !mt || !nt)
        return SSTE_ERR_INVALID_ARG;
    tile_coords(tile, m_tiles, n_tiles, group_m < m_tiles ? group_m : m_tiles, *mt, *nt);
    return SSTE_OK;
}
extern "C" sste_status sste_debug_force_tile_order(int group_m)
{
    if (group_m < 0) return SSTE_ERR_INVALID_ARG;
    g_force_group_m = group_m;
    return SSTE_OK;
}
extern "C" sste_status sste_debug_inject_stall(int on)
{
    g_inject_stall = on ? 1 : 0;
    return SSTE_OK;
}
extern "C" sste_status sste_debug_force_tile_width(int bn)
{
    if (bn != 0 && bn != 128 && bn != 192 && bn != 224 && bn != 256) return SSTE_ERR_INVALID_ARG;
    g_force_bn = bn;
    return SSTE_OK;
}

extern "C" sste_status sste_linear_fwd(sste_ctx *ctx, const void *X, int T, const void *vals, const void *meta, int O,
                                       int I, sste_dtype opdt, const float *x_amax_dev, const float *w_amax_dev,
                                       void *Y, sste_dtype ydt, float *y_amax_out_dev, void *stream)
{
    if (!ctx || !X || !vals || !meta || !Y) return SSTE_ERR_INVALID_ARG;
    int elt;
    uint32_t code;
    if (!fmt_code(opdt, &elt, &code) || opdt == SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (ydt != SSTE_BF16 && ydt != SSTE_F32) return SSTE_ERR_DTYPE;
    if (!amax_args_ok(elt, w_amax_dev, x_amax_dev)) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(X, 128) || !sste_aligned(vals, 128) || !sste_aligned(meta, 128) || !sste_aligned(Y, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    // Z^T[O, T] = S(W)[O, I] X^T: M = O, N = T, K = I; the output is stored transposed as Y[T, O]
    GemmParams p{O, T, I, Y, w_amax_dev, x_amax_dev, sste_fp8_max(opdt), sste_fp8_max(opdt),
                 reinterpret_cast<unsigned int *>(y_amax_out_dev), ctx->status_dev, code, code, nullptr};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (elt == 2) return launch_out<true, BMajor::K, 2, true>(ctx, vals, X, meta, p, ydt, s);
    return launch_out<true, BMajor::K, 1, true>(ctx, vals, X, meta, p, ydt, s);
}

extern "C" sste_status sste_linear_bwd_weight(sste_ctx *ctx, const void *gvals, const void *gmeta, int O, int T,
                                              sste_dtype gdt, const void *X, int I, sste_dtype xdt,
                                              const float *g_amax_dev, const float *x_amax_dev, void *dW,
                                              sste_dtype dwdt, void *stream)
{
    if (!ctx || !gvals || !gmeta || !X || !dW) return SSTE_ERR_INVALID_ARG;
    int ea, eb;
    uint32_t ca, cb;
    if (!fmt_code(gdt, &ea, &ca) || !fmt_code(xdt, &eb, &cb) || ea != eb) return SSTE_ERR_DTYPE;
    if (gdt == SSTE_E4M3 || xdt == SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (dwdt != SSTE_BF16 && dwdt != SSTE_F32) return SSTE_ERR_DTYPE;
    if (!amax_args_ok(ea, g_amax_dev, x_amax_dev)) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(X, 128) || !sste_aligned(gvals, 128) || !sste_aligned(gmeta, 128) || !sste_aligned(dW, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    // grad_W[O, I] = G[O, T] X[T, I]: M = O, N = I, K = T; X is [K, N] row-major = MN-major B
    GemmParams p{O, I, T, dW, g_amax_dev, x_amax_dev, sste_fp8_max(gdt), sste_fp8_max(xdt), nullptr,
                 ctx->status_dev, ca, cb, nullptr};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (ea == 2) return launch_out<true, BMajor::MN, 2, false>(ctx, gvals, X, gmeta, p, dwdt, s);
    return launch_out<true, BMajor::MN, 1, false>(ctx, gvals, X, gmeta, p, dwdt, s);
}

extern "C" sste_status sste_linear_bwd_input(sste_ctx *ctx, const void *dY, int T, int O, sste_dtype gdt,
                                             const void *Wt_dense, const void *vals, const void *meta, int I,
                                             sste_dtype wdt, const float *g_amax_dev, const float *w_amax_dev,
                                             void *dX, sste_dtype xdt, float *dx_amax_out_dev, void *stream)
{
    if (!ctx || !dY || !dX) return SSTE_ERR_INVALID_ARG;
    if (!Wt_dense && !(vals && meta)) return SSTE_ERR_INVALID_ARG;
    int ea, eb;
    uint32_t ca, cb;
    if (!fmt_code(gdt, &ea, &ca) || !fmt_code(wdt, &eb, &cb) || ea != eb) return SSTE_ERR_DTYPE;
    if (gdt == SSTE_E4M3 || wdt == SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (xdt != SSTE_BF16 && xdt != SSTE_F32) return SSTE_ERR_DTYPE;
    if (!amax_args_ok(ea, g_amax_dev, w_amax_dev)) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(T) || !sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(dY, 128) || !sste_aligned(Wt_dense, 128) || !sste_aligned(vals, 128) || !sste_aligned(meta, 128) ||
        !sste_aligned(dX, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    // grad_X[T, I] = grad_Z[T, O] S(W)[O, I]: M = T, N = I, K = O; S(W) is [K, N] row-major = MN-major B
    GemmParams p{T, I, O, dX, g_amax_dev, w_amax_dev, sste_fp8_max(gdt), sste_fp8_max(wdt),
                 reinterpret_cast<unsigned int *>(dx_amax_out_dev), ctx->status_dev, ca, cb, nullptr};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!Wt_dense) {
        // S(W) from the forward's compressed operand, expanded in shared memory (256-wide tiles)
        const bool f32 = (xdt == SSTE_F32);
        if (ea == 2)
            return f32 ? launch<false, BMajor::MN, 2, 256, false, true, true>(ctx, dY, vals, meta, p, s)
                       : launch<false, BMajor::MN, 2, 256, false, false, true>(ctx, dY, vals, meta, p, s);
        return f32 ? launch<false, BMajor::MN, 1, 256, false, true, true>(ctx, dY, vals, meta, p, s)
                   : launch<false, BMajor::MN, 1, 256, false, false, true>(ctx, dY, vals, meta, p, s);
    }
    if (ea == 2) return launch_out<false, BMajor::MN, 2, false>(ctx, dY, Wt_dense, nullptr, p, xdt, s);
    return launch_out<false, BMajor::MN, 1, false>(ctx, dY, Wt_dense, nullptr, p, xdt, s);
}
