// HBM-bound kernels of the S-STE linear layer: beta (Eq. 5), the fused
// projection + scale + 2:4 compression (Eq. 4, Sec. 4.2), the fused MVUE +
// compression of the output gradient (Sec. 5.1) and the FP8 scaling helpers
// (Sec. 5.2).  Every fp32 step is a single rounded operation (no FMA
// contraction) in a fixed order, so results are reproducible bit for bit.
#include "common.cuh"

namespace {

constexpr int EW_THREADS = 256;
constexpr int PC_ROWS = 32;                                  // rows of W per project+compress CTA
constexpr int PC_CHUNKS = PC_ROWS * 16 / EW_THREADS;         // 16-byte chunks per thread

// ---------------------------------------------------------------- group of four: S_soft + kept pair

struct SoftGroup {
    float w[4];       // beta * S_soft (times the FP8 scale), pruned entries +0
    uint32_t p0, p1;  // kept positions, p0 < p1
};

// w01 = a0 | a1 << 16, w23 = a2 | a3 << 16 (bf16 bit patterns).  Written for instruction count (the kernel
// is bound by instruction issue): the threshold t = second-smallest magnitude comes from packed 16-bit
// min/max on the magnitude bits (bf16 magnitudes order like unsigned integers), sign(a)(|a| - t) is the single
// subtraction a - copysign(t, a), and the kept pair is the top two of four integer keys
// (magnitude << 2 | 3 - index: magnitude descending, index ascending; pairwise distinct) found with a
// seven-operation min/max network.
// MODE 0: the method's projection (threshold |t2|); MODE 1: interpolated threshold
// t = (1 - gamma) |t2| + gamma |t3| (Sec. 4.1); MODE 2: hard thresholding (Eq. 2), the kept pair unchanged.
template <bool FP8, int MODE>
__device__ __forceinline__ SoftGroup soft_group(uint32_t w01, uint32_t w23, float beta, float wscale, float gamma)
{
    SoftGroup r;
    const uint32_t m01 = w01 & 0x7fff7fffu, m23 = w23 & 0x7fff7fffu;
    // second-smallest of the four magnitudes, in both halves of t2
    const uint32_t lo = __vminu2(m01, m23), hi = __vmaxu2(m01, m23);
    const uint32_t lmax = __vmaxu2(lo, __byte_perm(lo, 0, 0x1032));
    const uint32_t hmin = __vminu2(hi, __byte_perm(hi, 0, 0x1032));
    const uint32_t t2 = __vminu2(lmax, hmin);
    uint32_t tb = t2 << 16;                             // fp32 bits of t
    if (MODE == 1) {                                    // third-smallest magnitude: the other of (lmax, hmin)
        const float t3 = __uint_as_float(__vmaxu2(lmax, hmin) << 16);
        tb = __float_as_uint(__fadd_rn(__fmul_rn(__fsub_rn(1.0f, gamma), __uint_as_float(tb)), __fmul_rn(gamma, t3)));
    }
    const float t = __uint_as_float(tb);
    const uint32_t ab[4] = {w01 << 16, w01 & 0xffff0000u, w23 << 16, w23 & 0xffff0000u};
    if (MODE != 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float a = __uint_as_float(ab[i]);
            const float st = __uint_as_float(tb | (ab[i] & 0x80000000u));     // copysign(t, a)
            float w = __fmul_rn(__fsub_rn(a, st), beta);                        // sign(a) (|a| - t) beta
            if (FP8) w = __fmul_rn(w, wscale);
            r.w[i] = (fabsf(a) > t) ? w : 0.0f;
        }
    }
    const uint32_t k0 = (m01 & 0xffffu) * 4u + 3u, k1 = (m01 >> 16) * 4u + 2u;
    const uint32_t k2 = (m23 & 0xffffu) * 4u + 1u, k3 = (m23 >> 16) * 4u;
    const uint32_t a = max(k0, k1), b = min(k0, k1), c = max(k2, k3), d = min(k2, k3);
    const uint32_t top1 = max(a, c), top2 = max(min(a, c), max(b, d));
    const uint32_t i1 = (top1 & 3u) ^ 3u, i2 = (top2 & 3u) ^ 3u;
    r.p0 = min(i1, i2);
    r.p1 = max(i1, i2);
    if (MODE == 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float a = __uint_as_float(ab[i]);
            float w = __fmul_rn(a, beta);
            if (FP8) w = __fmul_rn(w, wscale);
            const bool kept = (static_cast<uint32_t>(i) == r.p0) || (static_cast<uint32_t>(i) == r.p1);
            r.w[i] = (kept && fabsf(a) > 0.0f) ? w : 0.0f;      // a kept zero is +0 like every pruned entry
        }
    }
    return r;
}

// ---------------------------------------------------------------- project + compress

// One CTA: 32 rows x 128 input features of W (a quarter of a metadata atom, 512 contiguous bytes of its
// image); a thread handles two chunks of 8 consecutive features.  Small tiles keep even the 2.4 M-element
// GPT-2 weights spread over several CTAs per SM.
template <bool FP8, int MODE>
__global__ void __launch_bounds__(EW_THREADS)
project_compress_kernel(const uint4 *__restrict__ W, int I, const float *__restrict__ beta_dev,
                        const float *__restrict__ w_amax_dev, float gamma, void *__restrict__ vals,
                        uint8_t *__restrict__ meta, void *__restrict__ dense)
{
    __shared__ __align__(16) uint8_t meta_s[512];
    const int tid = threadIdx.x;
    const int kb = blockIdx.x, rb = blockIdx.y;
    sste_pdl_trigger();
    sste_pdl_wait();
    const float beta = *beta_dev;
    const float wscale = FP8 ? sste_scale_from_amax(*w_amax_dev, 448.0f) : 1.0f;
    const size_t row_chunks = static_cast<size_t>(I) / 8;

    uint4 in[PC_CHUNKS];
#pragma unroll
    for (int i = 0; i < PC_CHUNKS; ++i) {
        const int c = i * EW_THREADS + tid;
        const int row = c >> 4, kc = c & 15;
        in[i] = __ldg(W + (static_cast<size_t>(rb) * PC_ROWS + row) * row_chunks + kb * 16 + kc);
    }
#pragma unroll
    for (int i = 0; i < PC_CHUNKS; ++i) {
        const int c = i * EW_THREADS + tid;
        const int row = c >> 4, kc = c & 15;
        const uint32_t raw[4] = {in[i].x, in[i].y, in[i].z, in[i].w};
        uint32_t kept[2];      // per group: the two kept values, packed (bf16: 32 bits, fp8: 16 bits)
        uint32_t dn[2][2];     // per group: the four projected values, packed (bf16: two words, fp8: word 0)
        uint32_t mbyte = 0;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const SoftGroup s = soft_group<FP8, MODE>(raw[2 * g], raw[2 * g + 1], beta, wscale, gamma);
            if (FP8) {
                const uint32_t e01 = __nv_cvt_float2_to_fp8x2(make_float2(s.w[0], s.w[1]), __NV_SATFINITE, __NV_E4M3);
                const uint32_t e23 = __nv_cvt_float2_to_fp8x2(make_float2(s.w[2], s.w[3]), __NV_SATFINITE, __NV_E4M3);
                dn[g][0] = e01 | (e23 << 16);
                kept[g] = __byte_perm(dn[g][0], 0, s.p0 | (s.p1 << 4) | 0x4400u);
            } else {
                const __nv_bfloat162 d01 = __floats2bfloat162_rn(s.w[0], s.w[1]);
                const __nv_bfloat162 d23 = __floats2bfloat162_rn(s.w[2], s.w[3]);
                dn[g][0] = *reinterpret_cast<const uint32_t *>(&d01);
                dn[g][1] = *reinterpret_cast<const uint32_t *>(&d23);
                // halfword p0 -> low half, halfword p1 -> high half
                kept[g] = __byte_perm(dn[g][0], dn[g][1], 0x1010u + 0x22u * s.p0 + 0x2200u * s.p1);
            }
            mbyte |= (s.p0 | (s.p1 << 2)) << (4 * g);
        }
        const uint32_t k = 8u * kc;
        const uint32_t arow = (rb & 3) * PC_ROWS + row;   // row inside the 128-row atom
        meta_s[(FP8 ? sste_meta_atom_byte8(arow, k) : sste_meta_atom_byte16(arow, k)) - 512u * (rb & 3)] =
            static_cast<uint8_t>(mbyte);
        const size_t grow = static_cast<size_t>(rb) * PC_ROWS + row;
        const size_t chunk = grow * row_chunks + kb * 16 + kc;   // index in units of 8 input features
        if (FP8) {
            reinterpret_cast<uint32_t *>(vals)[chunk] = kept[0] | (kept[1] << 16);
            if (dense) reinterpret_cast<uint2 *>(dense)[chunk] = make_uint2(dn[0][0], dn[1][0]);
        } else {
            reinterpret_cast<uint2 *>(vals)[chunk] = make_uint2(kept[0], kept[1]);
            if (dense) reinterpret_cast<uint4 *>(dense)[chunk] = make_uint4(dn[0][0], dn[0][1], dn[1][0], dn[1][1]);
        }
    }
    __syncthreads();
    if (tid < 32) {
        const size_t atom = static_cast<size_t>(rb >> 2) * (I / 128) + kb;
        reinterpret_cast<uint4 *>(meta + atom * 2048 + 512 * (rb & 3))[tid] = reinterpret_cast<const uint4 *>(meta_s)[tid];
    }
}

// ---------------------------------------------------------------- beta

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// fp64 sums of <w, s> and <s, s>, s = S_soft(w) in exact arithmetic; per-block partials are
// combined by the last block in a fixed order.
// L1 = false: beta = <w, S_soft(w)> / ||S_soft(w)||^2 (Eq. 5); L1 = true: ||w||_1 / ||S_soft(w)||_1 (Sec. 4.2,
// the rescaling the method replaces).
template <bool L1>
__global__ void __launch_bounds__(EW_THREADS)
beta_kernel(const uint4 *__restrict__ W, size_t n_chunks, double *__restrict__ partials,
            unsigned int *__restrict__ counter, float *__restrict__ beta_dev, unsigned int *__restrict__ status)
{
    __shared__ double red[2][EW_THREADS / 32];
    __shared__ bool is_last;
    sste_pdl_trigger();
    sste_pdl_wait();
    double num = 0.0, den = 0.0;
    for (size_t c = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; c < n_chunks;
         c += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const uint4 v = __ldg(W + c);
        const uint32_t raw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const uint32_t bits[4] = {raw[2 * g] & 0xffffu, raw[2 * g] >> 16, raw[2 * g + 1] & 0xffffu,
                                      raw[2 * g + 1] >> 16};
            double a[4], m[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[i] = static_cast<double>(sste_bf16_bits_to_f32(bits[i]));
                m[i] = fabs(a[i]);
            }
            const double lo1 = fmin(m[0], m[1]), hi1 = fmax(m[0], m[1]);
            const double lo2 = fmin(m[2], m[3]), hi2 = fmax(m[2], m[3]);
            const double t = fmin(fmax(lo1, lo2), fmin(hi1, hi2));
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const double d = m[i] - t;
                if (L1) {
                    num += m[i];
                    if (d > 0.0) den += d;
                } else if (d > 0.0) {
                    const double s = copysign(d, a[i]);
                    num += a[i] * s;
                    den += s * s;
                }
            }
        }
    }
    num = warp_sum(num);
    den = warp_sum(den);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red[0][warp] = num; red[1][warp] = den; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double bn = 0.0, bd = 0.0;
        for (int w = 0; w < EW_THREADS / 32; ++w) { bn += red[0][w]; bd += red[1][w]; }
        partials[2 * blockIdx.x] = bn;
        partials[2 * blockIdx.x + 1] = bd;
        __threadfence();
        const unsigned int ticket = atomicAdd(counter, 1u);
        is_last = (ticket == gridDim.x - 1);
    }
    __syncthreads();
    if (is_last && threadIdx.x < 32) {
        __threadfence();
        double tn = 0.0, td = 0.0;
        for (unsigned int b = threadIdx.x; b < gridDim.x; b += 32) {
            tn += __ldcg(partials + 2 * b);
            td += __ldcg(partials + 2 * b + 1);
        }
        tn = warp_sum(tn);
        td = warp_sum(td);
        if (threadIdx.x == 0) {
            if (td == 0.0) {
                *beta_dev = 1.0f;
                atomicCAS(status, 0u, static_cast<unsigned int>(SSTE_ERR_DEGENERATE));
            } else {
                *beta_dev = static_cast<float>(tn / td);
            }
            *counter = 0u;
        }
    }
}

// ---------------------------------------------------------------- Philox4x32-10

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4])
{
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;   // one wide multiply gives both halves
        const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
        c0 = n0; c1 = static_cast<uint32_t>(p1); c2 = n2; c3 = static_cast<uint32_t>(p0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ---------------------------------------------------------------- MVUE of one group

// a <= b as an integer mask (all ones / zero) in one instruction
__device__ __forceinline__ int fset_le(float a, float b)
{
    int r;
    asm("set.le.s32.f32 %0, %1, %2;" : "=r"(r) : "f"(a), "f"(b));
    return r;
}

struct MvueGroup {
    uint32_t q0, q1;  // kept positions q0 < q1
    float v0, v1;     // their values before the cast
};

// Inclusion probabilities p_i = min(1, c |a_i|) with sum 2, kept values a_i / p_i, systematic sampling
// with one uniform u.  With x the first largest magnitude and rest the sum of the others:
//   clipped   (m_x >= rest): x is kept as is; one other element j, chosen with probability m_j / rest
//                            by the point u*rest on the others' cumulative sums (kept below rest), carries
//                            sign(a_j)*rest;
//   unclipped (m_x <  rest): the points u*S/2 and u*S/2 + S/2 on the cumulative sums pick two elements,
//                            both carry sign(a_j)*S/2.
// The kernel is bound by instruction issue, not by HBM, so this is written for instruction count: no
// branches, one-hot predicates, compares counted as 0 / -1 masks, and the two kept inputs picked by a byte
// permute of the packed bf16 pairs p01 = a0 | a1 << 16, p23 = a2 | a3 << 16 (only their sign, or for the
// clipped maximum their 16 bits, is needed).  Every fp32 step is a single rounded operation.
__device__ __forceinline__ MvueGroup mvue_group(uint32_t p01, uint32_t p23, float u)
{
    const float a0 = __uint_as_float(p01 << 16), a1 = __uint_as_float(p01 & 0xffff0000u);
    const float a2 = __uint_as_float(p23 << 16), a3 = __uint_as_float(p23 & 0xffff0000u);
    const float m0 = fabsf(a0), m1 = fabsf(a1), m2 = fabsf(a2), m3 = fabsf(a3);
    const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
    const bool e0 = (m0 == mx);
    const bool e1 = !e0 && (m1 == mx);
    const bool e2 = !e0 && !e1 && (m2 == mx);
    const bool e3 = !e0 && !e1 && !e2;
    const uint32_t xi = e0 ? 0u : e1 ? 1u : e2 ? 2u : 3u;
    // cumulative sums without x (adding +0 is exact) and with it
    const float z0 = e0 ? 0.0f : m0;
    const float z1 = __fadd_rn(z0, e1 ? 0.0f : m1);
    const float z2 = __fadd_rn(z1, e2 ? 0.0f : m2);
    const float rest = __fadd_rn(z2, e3 ? 0.0f : m3);
    const float s1 = __fadd_rn(m0, m1);
    const float s2 = __fadd_rn(s1, m2);
    const float s3 = __fadd_rn(s2, m3);
    const bool clipped = (mx >= rest);
    const float h = clipped ? rest : __fmul_rn(0.5f, s3);
    const float c0 = clipped ? z0 : m0, c1 = clipped ? z1 : s1, c2 = clipped ? z2 : s2;
    const float r1 = __fmul_rn(u, h);
    const float r2 = __fadd_rn(r1, h);
    // Clipped: a point that rounding put AT rest (possible only when u * rest is subnormal) counts as just below
    // it, which selects the last other element of nonzero magnitude.  (rest == 0: the second operand is a NaN and
    // fminf returns r1; that case is decided below.)
    const float r1c = clipped ? fminf(r1, __uint_as_float(__float_as_uint(rest) - 1u)) : r1;
    // number of cumulative sums at or below each point: compares as 0 / -1, one three-input add each
    const int j1 = -(fset_le(c0, r1c) + fset_le(c1, r1c) + fset_le(c2, r1c));
    const int n2 = -(fset_le(c0, r2) + fset_le(c1, r2) + fset_le(c2, r2));
    // index pair before ordering: (other, x) when clipped; (j1, j2) otherwise, where a first point in the
    // last element (j1 = 3) gives the pair (2, 3)
    const int ia_c = (rest == 0.0f) ? (e0 ? 1 : 0) : j1;
    const int ia_u = min(j1, 2);
    const int ib_u = min(max(j1 + 1, n2), 3);
    const uint32_t ia = static_cast<uint32_t>(clipped ? ia_c : ia_u);
    const uint32_t ib = clipped ? xi : static_cast<uint32_t>(ib_u);
    // bf16 bits of a_ia and a_ib in the upper half (lower half: don't care)
    const uint32_t sa = __byte_perm(p01, p23, ia * 0x2200u + 0x1000u);
    const uint32_t sb = __byte_perm(p01, p23, ib * 0x2200u + 0x1000u);
    // kept values sign(a_i) * h; a zero h yields +0; the clipped maximum keeps its own value
    const uint32_t hb = __float_as_uint(h);
    const uint32_t sgn = (hb == 0u) ? 0u : 0x80000000u;
    const float va = __uint_as_float((sa & sgn) | hb);
    const float vb = __uint_as_float(clipped ? (sb & 0xffff0000u) : ((sb & sgn) | hb));
    MvueGroup r;
    const bool swap = ia > ib;
    r.q0 = min(ia, ib);
    r.q1 = max(ia, ib);
    r.v0 = swap ? vb : va;
    r.v1 = swap ? va : vb;
    return r;
}

// The group rule on explicit inputs (test / debug): group i = four bf16 values a[4 i .. 4 i + 3] and the uniform
// u[i] = k[i] * 2^-24; out: kept positions (q0 | q1 << 2) and the two fp32 values before the cast.
__global__ void __launch_bounds__(EW_THREADS)
mvue_groups_kernel(const uint2 *__restrict__ a, const uint32_t *__restrict__ k24, size_t n, uint32_t *__restrict__ pos,
                   float2 *__restrict__ val)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    for (size_t i = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; i < n;
         i += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const uint2 g = a[i];
        const float u = __uint2float_rn(k24[i] & 0xffffffu) * 0x1p-24f;
        const MvueGroup r = mvue_group(g.x, g.y, u);
        pos[i] = r.q0 | (r.q1 << 2);
        val[i] = make_float2(r.v0, r.v1);
    }
}

// ---------------------------------------------------------------- MVUE + compress (transposing)

// One CTA: 128 tokens x 128 output columns of dY.  A thread task is 4 tokens x 8 columns
// (8 groups, two Philox calls); results are transposed through shared memory so that every
// output row (= column of dY) receives whole 128-byte lines.
// ANY_COUNTER: counter_cols is not a multiple of 4 (a padded, odd column count), so a thread's eight
// consecutive group indices do not start on a Philox block and span three blocks instead of two.
template <bool FP8, bool ANY_COUNTER>
__global__ void __launch_bounds__(EW_THREADS, 4)
mvue_kernel(const uint4 *__restrict__ dY, int O, int T, uint32_t key0, uint32_t key1, uint32_t tensor_id,
            uint32_t step, uint64_t tg_offset, uint32_t counter_cols, const float *__restrict__ g_amax_dev,
            void *__restrict__ gvals,
            uint8_t *__restrict__ gmeta, void *__restrict__ dense_q)
{
    // bf16: 128 rows x 32 words; fp8: 128 rows x 16 words
    __shared__ __align__(16) uint32_t vals_s[128 * (FP8 ? 16 : 32)];
    __shared__ __align__(16) uint8_t meta_s[2048];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int jb = blockIdx.x, tb = blockIdx.y;   // column block, token block
    sste_pdl_trigger();
    sste_pdl_wait();
    const float gscale = FP8 ? sste_scale_from_amax(*g_amax_dev, 57344.0f) : 1.0f;
    const size_t row_chunks = static_cast<size_t>(O) / 8;

#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int bidx = it * 8 + warp;
        const int jc = (bidx & 1) * 8 + (lane & 7);      // column chunk 0..15
        const int tgl = (bidx >> 1) * 4 + (lane >> 3);   // token group 0..31 inside the tile
        const size_t tok0 = static_cast<size_t>(tb) * 128 + 4 * tgl;
        uint4 in[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) in[i] = __ldg(dY + (tok0 + i) * row_chunks + jb * 16 + jc);

        const uint64_t g0 = (tg_offset + static_cast<uint64_t>(tb) * 32 + tgl) * static_cast<uint64_t>(counter_cols) +
                            static_cast<uint64_t>(jb) * 128 + jc * 8;
        const uint64_t q = g0 >> 2;
        uint32_t rnd[8];
        if (!ANY_COUNTER) {
            philox4x32_10(static_cast<uint32_t>(q), static_cast<uint32_t>(q >> 32), tensor_id, step, key0, key1, rnd);
            philox4x32_10(static_cast<uint32_t>(q + 1), static_cast<uint32_t>((q + 1) >> 32), tensor_id, step, key0,
                          key1, rnd + 4);
        } else {
            uint32_t r12[12];
#pragma unroll
            for (int b = 0; b < 3; ++b)
                philox4x32_10(static_cast<uint32_t>(q + b), static_cast<uint32_t>((q + b) >> 32), tensor_id, step, key0,
                              key1, r12 + 4 * b);
            const uint32_t sh = static_cast<uint32_t>(g0) & 3u;     // group g0 + e uses word (g0 + e) & 3 of block (g0 + e) >> 2
#pragma unroll
            for (int e = 0; e < 8; ++e)
                rnd[e] = sh == 0 ? r12[e] : sh == 1 ? r12[e + 1] : sh == 2 ? r12[e + 2] : r12[e + 3];
        }

        const uint32_t raw[4][4] = {{in[0].x, in[0].y, in[0].z, in[0].w},
                                    {in[1].x, in[1].y, in[1].z, in[1].w},
                                    {in[2].x, in[2].y, in[2].z, in[2].w},
                                    {in[3].x, in[3].y, in[3].z, in[3].w}};
        uint32_t nibs = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            // the group of column e: one bf16 from each of the four token rows, packed in pairs
            const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
            const uint32_t p01 = __byte_perm(raw[0][e >> 1], raw[1][e >> 1], sel);
            const uint32_t p23 = __byte_perm(raw[2][e >> 1], raw[3][e >> 1], sel);
            const float u = __uint2float_rn(rnd[e] >> 8) * 0x1p-24f;
            const MvueGroup r = mvue_group(p01, p23, u);
            nibs |= (r.q0 | (r.q1 << 2)) << (4 * e);
            const int jl = jc * 8 + e;
            if (FP8) {
                const uint32_t pair = static_cast<uint32_t>(__nv_cvt_float2_to_fp8x2(
                    make_float2(__fmul_rn(r.v0, gscale), __fmul_rn(r.v1, gscale)), __NV_SATFINITE, __NV_E5M2));
                reinterpret_cast<uint16_t *>(vals_s)[jl * 32 + (tgl ^ (8 * (jc & 3)))] = static_cast<uint16_t>(pair);
            } else {
                const __nv_bfloat162 pair = __floats2bfloat162_rn(r.v0, r.v1);
                vals_s[jl * 32 + (tgl ^ (4 * (jc & 7)))] = *reinterpret_cast<const uint32_t *>(&pair);
            }
        }
        if (FP8 && dense_q) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t b[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint32_t word = raw[i][e >> 1];
                    const float v = sste_bf16_bits_to_f32((e & 1) ? (word >> 16) : (word & 0xffffu));
                    b[e] = sste_f32_to_e5m2(__fmul_rn(v, gscale));
                }
                uint2 d;
                d.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
                d.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
                reinterpret_cast<uint2 *>(dense_q)[(tok0 + i) * row_chunks + jb * 16 + jc] = d;
            }
        }
        // two token groups share a metadata byte: lane ^ 8 holds the neighbouring token group
        const uint32_t other = __shfl_xor_sync(0xffffffffu, nibs, 8);
        if ((tgl & 1) == 0) {
            const uint32_t k = 4u * tgl;
            // the eight bytes (own nibble | neighbour's nibble << 4) of columns e = 0..7, four at a time:
            // even columns from the low nibbles of each byte of `nibs`, odd columns from the high ones
            const uint32_t even = (nibs & 0x0f0f0f0fu) | ((other << 4) & 0xf0f0f0f0u);
            const uint32_t odd = ((nibs >> 4) & 0x0f0f0f0fu) | (other & 0xf0f0f0f0u);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t jl = jc * 8 + e;
                const uint32_t byte = ((e & 1) ? odd : even) >> (8 * (e >> 1));
                meta_s[FP8 ? sste_meta_atom_byte8(jl, k) : sste_meta_atom_byte16(jl, k)] = static_cast<uint8_t>(byte);
            }
        }
    }
    __syncthreads();
    // rows of the transposed tile: bf16 128 B (8 vectors of 16 B), fp8 64 B (4 vectors)
    constexpr int VECS = FP8 ? 4 : 8;
    const size_t out_row_vecs = static_cast<size_t>(T) / (FP8 ? 32 : 16);   // 16-byte vectors per output row
#pragma unroll
    for (int it = 0; it < (128 * VECS) / EW_THREADS; ++it) {
        const int v = it * EW_THREADS + tid;
        const int row = v / VECS, vec = v % VECS;
        const int pvec = FP8 ? (vec ^ ((row >> 3) & 3)) : (vec ^ ((row >> 3) & 7));
        const uint4 data = reinterpret_cast<const uint4 *>(vals_s)[row * VECS + pvec];
        reinterpret_cast<uint4 *>(gvals)[(static_cast<size_t>(jb) * 128 + row) * out_row_vecs + tb * VECS + vec] = data;
    }
    if (tid < 128) {
        const size_t atom = static_cast<size_t>(jb) * (T / 128) + tb;
        reinterpret_cast<uint4 *>(gmeta + atom * 2048)[tid] = reinterpret_cast<const uint4 *>(meta_s)[tid];
    }
}

// ---------------------------------------------------------------- FP8 helpers

__global__ void __launch_bounds__(EW_THREADS)
amax_kernel(const uint4 *__restrict__ x, size_t n_chunks, float *__restrict__ amax_dev)
{
    uint32_t best2 = 0;   // magnitude bits of bf16 compare like unsigned integers: running maximum in both halves
    sste_pdl_trigger();
    sste_pdl_wait();
    // four independent 16-byte loads per thread and iteration: a pure read needs the bytes in flight
    const size_t stride = static_cast<size_t>(gridDim.x) * EW_THREADS;
    for (size_t c = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; c < n_chunks; c += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (c + j * stride < n_chunks) ? __ldg(x + c + j * stride) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            best2 = __vmaxu2(best2, v[j].x & 0x7fff7fffu);
            best2 = __vmaxu2(best2, v[j].y & 0x7fff7fffu);
            best2 = __vmaxu2(best2, v[j].z & 0x7fff7fffu);
            best2 = __vmaxu2(best2, v[j].w & 0x7fff7fffu);
        }
    }
    uint32_t best = max(best2 & 0xffffu, best2 >> 16);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
    if ((threadIdx.x & 31) == 0 && best != 0)
        atomicMax(reinterpret_cast<unsigned int *>(amax_dev), best << 16);   // non-negative floats order as uints
}

// amax of the bf16 projection w~ = bf16(beta * S_soft(W)) without writing it: rounding to bf16 is monotone,
// so the maximum of the rounded magnitudes is the rounded maximum of the fp32 ones.
__global__ void __launch_bounds__(EW_THREADS)
project_amax_kernel(const uint4 *__restrict__ W, size_t n_chunks, const float *__restrict__ beta_dev,
                    float *__restrict__ amax_dev)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const float beta = *beta_dev;
    float best = 0.0f;
    const size_t stride = static_cast<size_t>(gridDim.x) * EW_THREADS;
    for (size_t c = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; c < n_chunks; c += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (c + j * stride < n_chunks) ? __ldg(W + c + j * stride) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t raw[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                // the largest |w~| of a group belongs to its largest |w|: one product per group suffices
                const uint32_t m01 = raw[2 * g] & 0x7fff7fffu, m23 = raw[2 * g + 1] & 0x7fff7fffu;
                const uint32_t lo = __vminu2(m01, m23), hi = __vmaxu2(m01, m23);
                const uint32_t t2 = __vminu2(__vmaxu2(lo, __byte_perm(lo, 0, 0x1032)), __vminu2(hi, __byte_perm(hi, 0, 0x1032)));
                const uint32_t mx = __vmaxu2(hi, __byte_perm(hi, 0, 0x1032));
                const float d = __fsub_rn(__uint_as_float(mx << 16), __uint_as_float(t2 << 16));
                best = fmaxf(best, fabsf(__fmul_rn(d, beta)));
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, off));
    const uint32_t bits = sste_f32_to_bf16_bits(best);
    if ((threadIdx.x & 31) == 0 && bits != 0)
        atomicMax(reinterpret_cast<unsigned int *>(amax_dev), bits << 16);   // non-negative floats order as uints
}

__global__ void fp8_scale_kernel(const float *amax_dev, float fp8_max, float *scale_dev, float *inv_scale_dev)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const float a = *amax_dev;
    const float s = sste_scale_from_amax(a, fp8_max);
    *scale_dev = s;
    if (inv_scale_dev) *inv_scale_dev = __fdiv_rn(1.0f, s);
}

template <bool E5M2>
__global__ void __launch_bounds__(EW_THREADS)
quantize_kernel(const uint4 *__restrict__ x, size_t n_chunks, const float *__restrict__ amax_dev,
                uint2 *__restrict__ q)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const float scale = sste_scale_from_amax(*amax_dev, E5M2 ? 57344.0f : 448.0f);
    const size_t stride = static_cast<size_t>(gridDim.x) * EW_THREADS;
    for (size_t c = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; c < n_chunks; c += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (c + j * stride < n_chunks) ? __ldg(x + c + j * stride) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (c + j * stride >= n_chunks) break;
            const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
            uint32_t h[4];           // two codes per word: packed conversion of (low half, high half)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = make_float2(__fmul_rn(__uint_as_float(w[i] << 16), scale),
                                             __fmul_rn(__uint_as_float(w[i] & 0xffff0000u), scale));
                h[i] = static_cast<uint32_t>(__nv_cvt_float2_to_fp8x2(f, __NV_SATFINITE, E5M2 ? __NV_E5M2 : __NV_E4M3));
            }
            q[c + j * stride] = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
        }
    }
}

// ---------------------------------------------------------------- metadata image -> canonical

template <bool EIGHT_BIT>
__global__ void __launch_bounds__(EW_THREADS)
meta_to_canonical_kernel(const uint8_t *__restrict__ meta, int rows, int k, uint16_t *__restrict__ out)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const size_t words = static_cast<size_t>(rows) * (k / 16);
    for (size_t w = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; w < words;
         w += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const uint32_t r = static_cast<uint32_t>(w / (k / 16));
        const uint32_t kk = static_cast<uint32_t>(w % (k / 16)) * 16;   // first K index of this word
        const size_t atom = static_cast<size_t>(r >> 7) * (k / 128) + (kk >> 7);
        const uint8_t *base = meta + atom * 2048;
        const uint32_t m = r & 127u, ko = kk & 127u;
        const uint32_t b0 = EIGHT_BIT ? sste_meta_atom_byte8(m, ko) : sste_meta_atom_byte16(m, ko);
        const uint32_t b1 = EIGHT_BIT ? sste_meta_atom_byte8(m, ko + 8) : sste_meta_atom_byte16(m, ko + 8);
        out[w] = static_cast<uint16_t>(base[b0] | (base[b1] << 8));
    }
}

// ---------------------------------------------------------------- compressed operand -> dense (test / debug)

// One thread per 16 bytes of values: bf16 4 groups (16 dense elements), fp8 8 groups (32 dense elements).
template <bool EIGHT_BIT>
__global__ void __launch_bounds__(EW_THREADS)
decompress_kernel(const uint4 *__restrict__ vals, const uint8_t *__restrict__ meta, int k, size_t n_units,
                  uint4 *__restrict__ dense)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const size_t units_per_row = static_cast<size_t>(k) / (EIGHT_BIT ? 32 : 16);
    for (size_t un = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; un < n_units;
         un += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const uint32_t row = static_cast<uint32_t>(un / units_per_row);
        const uint32_t kk = static_cast<uint32_t>(un % units_per_row) * (EIGHT_BIT ? 32u : 16u);
        const uint8_t *atom = meta + (static_cast<size_t>(row >> 7) * (k / 128) + (kk >> 7)) * 2048;
        const uint4 v = __ldg(vals + un);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[8];
        if (EIGHT_BIT) {
            const uint32_t codes = *reinterpret_cast<const uint32_t *>(atom + sste_meta_atom_byte8(row & 127u, kk & 127u));
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const uint32_t nib = (codes >> (4 * g)) & 0xfu, p0 = nib & 3u, p1 = nib >> 2;
                const uint32_t pr = (g & 1) ? (w[g >> 1] >> 16) : (w[g >> 1] & 0xffffu);
                o[g] = ((pr & 0xffu) << (8 * p0)) | ((pr >> 8) << (8 * p1));
            }
        } else {
            const uint32_t codes = *reinterpret_cast<const uint16_t *>(atom + sste_meta_atom_byte16(row & 127u, kk & 127u));
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const uint32_t nib = (codes >> (4 * g)) & 0xfu, p0 = nib & 3u, p1 = nib >> 2;
                const uint64_t d = (static_cast<uint64_t>(w[g] & 0xffffu) << (16 * p0)) |
                                   (static_cast<uint64_t>(w[g] >> 16) << (16 * p1));
                o[2 * g] = static_cast<uint32_t>(d);
                o[2 * g + 1] = static_cast<uint32_t>(d >> 32);
            }
        }
        dense[2 * un] = make_uint4(o[0], o[1], o[2], o[3]);
        dense[2 * un + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// ---------------------------------------------------------------- zero padding to multiples of 128 and back

// dst [rows_p, cols_p] <- src [rows, cols] in the top-left corner, zeros elsewhere; 2-byte elements, one
// thread per 8 destination elements (16-byte stores; element-wise loads, src rows need no alignment).
__global__ void __launch_bounds__(EW_THREADS)
pad_2d_kernel(const uint16_t *__restrict__ src, int rows, int cols, uint4 *__restrict__ dst, int cols_p, size_t n_vec)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const size_t vec_per_row = static_cast<size_t>(cols_p) / 8;
    for (size_t v = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; v < n_vec;
         v += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const size_t r = v / vec_per_row;
        const int c0 = static_cast<int>(v % vec_per_row) * 8;
        uint32_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            e[i] = (r < static_cast<size_t>(rows) && c0 + i < cols) ? __ldg(src + r * cols + c0 + i) : 0u;
        dst[v] = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
    }
}

// dst [rows, cols] <- top-left corner of src [rows_p, cols_p]; one thread per element pair would be wasteful for
// odd cols, so one thread per destination element (coalesced 2-byte accesses).
__global__ void __launch_bounds__(EW_THREADS)
crop_2d_kernel(const uint16_t *__restrict__ src, int cols_p, uint16_t *__restrict__ dst, int cols, size_t n)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    for (size_t i = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; i < n;
         i += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const size_t r = i / cols, c = i % cols;
        dst[i] = __ldg(src + r * cols_p + c);
    }
}

int grid_for(size_t work_items, int sm_count)
{
    size_t blocks = (work_items + EW_THREADS - 1) / EW_THREADS;
    size_t cap = static_cast<size_t>(sm_count) * 8;
    if (cap > SSTE_MAX_REDUCE_BLOCKS) cap = SSTE_MAX_REDUCE_BLOCKS;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return static_cast<int>(blocks);
}

// every entry point of this file launches exactly one kernel
sste_status launch_result()
{
    if (cudaGetLastError() != cudaSuccess) return SSTE_ERR_CUDA;
    sste_count_launches(1);
    return SSTE_OK;
}

// ---------------------------------------------------------------- SR-STE decay term (Sec. 3.2)

// grad_W += lambda * w on the entries the 2:4 mask prunes: the gradient of (lambda / 2) ||w (1 - m_h(w))||^2.
// A thread handles 8 consecutive features of a row (two groups: one metadata byte of the operand image).
template <bool EIGHT_BIT>
__global__ void __launch_bounds__(EW_THREADS)
srste_decay_kernel(const uint4 *__restrict__ W, const uint8_t *__restrict__ meta, int I, size_t n_chunks, float lambda,
                   uint4 *__restrict__ dW)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    const size_t row_chunks = static_cast<size_t>(I) / 8;
    for (size_t c = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; c < n_chunks;
         c += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const uint32_t row = static_cast<uint32_t>(c / row_chunks), k = static_cast<uint32_t>(c % row_chunks) * 8u;
        const size_t atom = static_cast<size_t>(row >> 7) * (I / 128) + (k >> 7);
        const uint32_t byte = __ldg(meta + atom * 2048 + (EIGHT_BIT ? sste_meta_atom_byte8(row & 127u, k & 127u)
                                                                     : sste_meta_atom_byte16(row & 127u, k & 127u)));
        const uint4 w = __ldg(W + c);
        uint4 g = dW[c];
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
        uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
        for (int grp = 0; grp < 2; ++grp) {
            const uint32_t nib = (byte >> (4 * grp)) & 0xfu;
            const uint32_t keep = (1u << (nib & 3u)) | (1u << (nib >> 2));
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (keep & (1u << e)) continue;
                const int word = 2 * grp + (e >> 1), sh = 16 * (e & 1);
                const float wv = sste_bf16_bits_to_f32((ww[word] >> sh) & 0xffffu);
                const float gv = sste_bf16_bits_to_f32((gw[word] >> sh) & 0xffffu);
                const uint32_t out = sste_f32_to_bf16_bits(__fadd_rn(gv, __fmul_rn(lambda, wv)));
                gw[word] = (gw[word] & ~(0xffffu << sh)) | (out << sh);
            }
        }
        dW[c] = make_uint4(gw[0], gw[1], gw[2], gw[3]);
    }
}

// ---------------------------------------------------------------- flip count (Sec. 3.1, "Flip rate")

// Number of entries in which the 2:4 masks of two operand images differ.  Both images have the same layout,
// so nibbles are compared in place: a nibble p0 | p1 << 2 stands for the mask (1 << p0) | (1 << p1).
__global__ void __launch_bounds__(EW_THREADS)
flip_count_kernel(const uint4 *__restrict__ a, const uint4 *__restrict__ b, size_t n_vec,
                  unsigned long long *__restrict__ count)
{
    sste_pdl_trigger();
    sste_pdl_wait();
    unsigned int local = 0;
    for (size_t v = static_cast<size_t>(blockIdx.x) * EW_THREADS + threadIdx.x; v < n_vec;
         v += static_cast<size_t>(gridDim.x) * EW_THREADS) {
        const uint4 x = __ldg(a + v), y = __ldg(b + v);
        const uint32_t wx[4] = {x.x, x.y, x.z, x.w}, wy[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            if (wx[w] == wy[w]) continue;
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                const uint32_t nx = (wx[w] >> (4 * n)) & 0xfu, ny = (wy[w] >> (4 * n)) & 0xfu;
                const uint32_t mx = (1u << (nx & 3u)) | (1u << (nx >> 2)), my = (1u << (ny & 3u)) | (1u << (ny >> 2));
                local += __popc(mx ^ my);
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
    if ((threadIdx.x & 31) == 0 && local) atomicAdd(count, static_cast<unsigned long long>(local));
}

}  // namespace

// ---------------------------------------------------------------- entry points

namespace {

sste_status beta_launch(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt, float *beta_dev, void *stream, bool l1)
{
    if (!ctx || !W || !beta_dev) return SSTE_ERR_INVALID_ARG;
    if (wdt != SSTE_BF16) return SSTE_ERR_DTYPE;
    if (!sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(W, 128) || !sste_aligned(beta_dev, 4)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_chunks = static_cast<size_t>(O) * I / 8;
    const int grid = grid_for(n_chunks, ctx->sm_count);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (l1)
        sste_launch(beta_kernel<true>, dim3(grid), dim3(EW_THREADS), 0, s, static_cast<const uint4 *>(W), n_chunks,
                    ctx->partials_dev, ctx->counter_dev, beta_dev, ctx->status_dev);
    else
        sste_launch(beta_kernel<false>, dim3(grid), dim3(EW_THREADS), 0, s, static_cast<const uint4 *>(W), n_chunks,
                    ctx->partials_dev, ctx->counter_dev, beta_dev, ctx->status_dev);
    return launch_result();
}

// mode: 0 = the method's projection, 1 = interpolated threshold, 2 = hard thresholding
sste_status project_launch(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt, const float *beta_dev,
                           const float *w_amax_dev, sste_dtype odt, int mode, float gamma, void *vals, void *meta,
                           void *dense_out, void *stream)
{
    if (!ctx || !W || !beta_dev || !vals || !meta) return SSTE_ERR_INVALID_ARG;
    if (wdt != SSTE_BF16 || (odt != SSTE_BF16 && odt != SSTE_E4M3)) return SSTE_ERR_DTYPE;
    if (odt == SSTE_E4M3 && !w_amax_dev) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(W, 128) || !sste_aligned(vals, 128) || !sste_aligned(meta, 128) ||
        !sste_aligned(dense_out, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const dim3 grid(I / 128, O / PC_ROWS);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint4 *w = static_cast<const uint4 *>(W);
    uint8_t *m = static_cast<uint8_t *>(meta);
    const bool f8 = (odt == SSTE_E4M3);
#define SSTE_PC_LAUNCH(F8, MODE)                                                                                   \
    sste_launch(project_compress_kernel<F8, MODE>, dim3(grid), dim3(EW_THREADS), 0, s, w, I, beta_dev,           \
                F8 ? w_amax_dev : nullptr, gamma, vals, m, dense_out)
    if (mode == 0) { if (f8) SSTE_PC_LAUNCH(true, 0); else SSTE_PC_LAUNCH(false, 0); }
    else if (mode == 1) { if (f8) SSTE_PC_LAUNCH(true, 1); else SSTE_PC_LAUNCH(false, 1); }
    else { if (f8) SSTE_PC_LAUNCH(true, 2); else SSTE_PC_LAUNCH(false, 2); }
#undef SSTE_PC_LAUNCH
    return launch_result();
}

}  // namespace

extern "C" sste_status sste_beta_init(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt, float *beta_dev,
                                      void *stream)
{
    return beta_launch(ctx, W, O, I, wdt, beta_dev, stream, false);
}

extern "C" sste_status sste_beta_init_l1(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt, float *beta_dev,
                                         void *stream)
{
    return beta_launch(ctx, W, O, I, wdt, beta_dev, stream, true);
}

extern "C" sste_status sste_project_compress(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt,
                                             const float *beta_dev, const float *w_amax_dev, sste_dtype odt,
                                             void *vals, void *meta, void *dense_out, void *stream)
{
    return project_launch(ctx, W, O, I, wdt, beta_dev, w_amax_dev, odt, 0, 0.0f, vals, meta, dense_out, stream);
}

extern "C" sste_status sste_project_compress_variant(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt,
                                                     const float *beta_dev, const float *w_amax_dev, sste_dtype odt,
                                                     sste_pruning pruning, float gamma, void *vals, void *meta,
                                                     void *dense_out, void *stream)
{
    if (pruning != SSTE_PRUNE_SOFT && pruning != SSTE_PRUNE_HARD) return SSTE_ERR_INVALID_ARG;
    if (!(gamma >= 0.0f && gamma <= 1.0f)) return SSTE_ERR_INVALID_ARG;
    const int mode = (pruning == SSTE_PRUNE_HARD) ? 2 : (gamma == 0.0f ? 0 : 1);
    return project_launch(ctx, W, O, I, wdt, beta_dev, w_amax_dev, odt, mode, gamma, vals, meta, dense_out, stream);
}

extern "C" sste_status sste_srste_decay(sste_ctx *ctx, const void *W, const void *meta, int O, int I,
                                        sste_dtype meta_dt, float lambda, void *dW, void *stream)
{
    if (!ctx || !W || !meta || !dW) return SSTE_ERR_INVALID_ARG;
    if (meta_dt != SSTE_BF16 && meta_dt != SSTE_E4M3 && meta_dt != SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (!sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(W, 16) || !sste_aligned(meta, 16) || !sste_aligned(dW, 16)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_chunks = static_cast<size_t>(O) * I / 8;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (meta_dt == SSTE_BF16)
        sste_launch(srste_decay_kernel<false>, dim3(grid_for(n_chunks, ctx->sm_count)), dim3(EW_THREADS), 0, s,
                    static_cast<const uint4 *>(W), static_cast<const uint8_t *>(meta), I, n_chunks, lambda,
                    static_cast<uint4 *>(dW));
    else
        sste_launch(srste_decay_kernel<true>, dim3(grid_for(n_chunks, ctx->sm_count)), dim3(EW_THREADS), 0, s,
                    static_cast<const uint4 *>(W), static_cast<const uint8_t *>(meta), I, n_chunks, lambda,
                    static_cast<uint4 *>(dW));
    return launch_result();
}

extern "C" sste_status sste_mvue_sparsify(sste_ctx *ctx, const void *dY, int T, int O, sste_dtype gdt, uint64_t seed,
                                          uint32_t tensor_id, uint32_t step, uint64_t token_offset, int counter_cols,
                                          const float *g_amax_dev, sste_dtype odt, void *gvals, void *gmeta,
                                          void *dense_q_out, void *stream)
{
    if (!ctx || !dY || !gvals || !gmeta) return SSTE_ERR_INVALID_ARG;
    if (gdt != SSTE_BF16 || (odt != SSTE_BF16 && odt != SSTE_E5M2)) return SSTE_ERR_DTYPE;
    if (odt == SSTE_E5M2 && !g_amax_dev) return SSTE_ERR_INVALID_ARG;
    if (counter_cols < 0 || counter_cols > O) return SSTE_ERR_INVALID_ARG;
    const uint32_t ccols = static_cast<uint32_t>(counter_cols == 0 ? O : counter_cols);
    if (odt == SSTE_BF16 && dense_q_out) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(O) || !sste_mult128(T) || (token_offset % 4) != 0) return SSTE_ERR_SHAPE;
    if (!sste_aligned(dY, 128) || !sste_aligned(gvals, 128) || !sste_aligned(gmeta, 128) ||
        !sste_aligned(dense_q_out, 128))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const dim3 grid(O / 128, T / 128);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t key0 = static_cast<uint32_t>(seed), key1 = static_cast<uint32_t>(seed >> 32);
    const uint4 *g = static_cast<const uint4 *>(dY);
    uint8_t *gm = static_cast<uint8_t *>(gmeta);
    const uint64_t tg0 = token_offset / 4;
    const bool f8 = (odt == SSTE_E5M2), any = (ccols % 4) != 0;
#define SSTE_MVUE_LAUNCH(F8, ANY)                                                                                   \
    sste_launch(mvue_kernel<F8, ANY>, dim3(grid), dim3(EW_THREADS), 0, s, g, O, T, key0, key1, tensor_id, step, tg0, \
                ccols, F8 ? g_amax_dev : nullptr, gvals, gm, F8 ? dense_q_out : nullptr)
    if (f8) { if (any) SSTE_MVUE_LAUNCH(true, true); else SSTE_MVUE_LAUNCH(true, false); }
    else { if (any) SSTE_MVUE_LAUNCH(false, true); else SSTE_MVUE_LAUNCH(false, false); }
#undef SSTE_MVUE_LAUNCH
    return launch_result();
}

extern "C" sste_status sste_amax(sste_ctx *ctx, const void *x, size_t n, sste_dtype dt, float *amax_dev, void *stream)
{
    if (!ctx || !x || !amax_dev) return SSTE_ERR_INVALID_ARG;
    if (dt != SSTE_BF16) return SSTE_ERR_DTYPE;
    if (n == 0 || n % 8 != 0) return SSTE_ERR_SHAPE;
    if (!sste_aligned(x, 16) || !sste_aligned(amax_dev, 4)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_chunks = n / 8;
    SSTE_CUDA_TRY(cudaMemsetAsync(amax_dev, 0, sizeof(float), static_cast<cudaStream_t>(stream)));
    sste_launch(amax_kernel, dim3(grid_for(n_chunks, ctx->sm_count)), dim3(EW_THREADS), 0,
                static_cast<cudaStream_t>(stream), static_cast<const uint4 *>(x), n_chunks, amax_dev);
    return launch_result();
}

extern "C" sste_status sste_project_amax(sste_ctx *ctx, const void *W, int O, int I, sste_dtype wdt,
                                         const float *beta_dev, float *amax_dev, void *stream)
{
    if (!ctx || !W || !beta_dev || !amax_dev) return SSTE_ERR_INVALID_ARG;
    if (wdt != SSTE_BF16) return SSTE_ERR_DTYPE;
    if (!sste_mult128(O) || !sste_mult128(I)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(W, 16) || !sste_aligned(amax_dev, 4)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_chunks = static_cast<size_t>(O) * I / 8;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SSTE_CUDA_TRY(cudaMemsetAsync(amax_dev, 0, sizeof(float), s));
    sste_launch(project_amax_kernel, dim3(grid_for(n_chunks, ctx->sm_count)), dim3(EW_THREADS), 0, s,
                static_cast<const uint4 *>(W), n_chunks, beta_dev, amax_dev);
    return launch_result();
}

extern "C" sste_status sste_fp8_scale(sste_ctx *ctx, const float *amax_dev, sste_dtype odt, float *scale_dev,
                                      float *inv_scale_dev, void *stream)
{
    if (!ctx || !amax_dev || !scale_dev) return SSTE_ERR_INVALID_ARG;
    if (odt != SSTE_E4M3 && odt != SSTE_E5M2) return SSTE_ERR_DTYPE;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    sste_launch(fp8_scale_kernel, dim3(1), dim3(1), 0, static_cast<cudaStream_t>(stream), amax_dev,
                odt == SSTE_E4M3 ? 448.0f : 57344.0f, scale_dev, inv_scale_dev);
    return launch_result();
}

extern "C" sste_status sste_quantize_fp8(sste_ctx *ctx, const void *x, size_t n, const float *amax_dev,
                                         sste_dtype odt, void *q, void *stream)
{
    if (!ctx || !x || !amax_dev || !q) return SSTE_ERR_INVALID_ARG;
    if (odt != SSTE_E4M3 && odt != SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (n == 0 || n % 16 != 0) return SSTE_ERR_SHAPE;
    if (!sste_aligned(x, 16) || !sste_aligned(q, 16)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_chunks = n / 8;
    const int grid = grid_for(n_chunks, ctx->sm_count);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (odt == SSTE_E5M2)
        sste_launch(quantize_kernel<true>, dim3(grid), dim3(EW_THREADS), 0, s, static_cast<const uint4 *>(x),
                    n_chunks, amax_dev, static_cast<uint2 *>(q));
    else
        sste_launch(quantize_kernel<false>, dim3(grid), dim3(EW_THREADS), 0, s, static_cast<const uint4 *>(x),
                    n_chunks, amax_dev, static_cast<uint2 *>(q));
    return launch_result();
}

extern "C" sste_status sste_meta_to_canonical(sste_ctx *ctx, const void *meta, int rows, int k, sste_dtype dt,
                                              void *canonical_out, void *stream)
{
    if (!ctx || !meta || !canonical_out) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(rows) || !sste_mult128(k)) return SSTE_ERR_SHAPE;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t words = static_cast<size_t>(rows) * (k / 16);
    const int grid = grid_for(words, ctx->sm_count);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (dt == SSTE_BF16)
        sste_launch(meta_to_canonical_kernel<false>, dim3(grid), dim3(EW_THREADS), 0, s,
                    static_cast<const uint8_t *>(meta), rows, k, static_cast<uint16_t *>(canonical_out));
    else
        sste_launch(meta_to_canonical_kernel<true>, dim3(grid), dim3(EW_THREADS), 0, s,
                    static_cast<const uint8_t *>(meta), rows, k, static_cast<uint16_t *>(canonical_out));
    return launch_result();
}

extern "C" sste_status sste_flip_count(sste_ctx *ctx, const void *meta_prev, const void *meta_cur, int rows, int k,
                                       unsigned long long *count_dev, void *stream)
{
    if (!ctx || !meta_prev || !meta_cur || !count_dev) return SSTE_ERR_INVALID_ARG;
    if (!sste_mult128(rows) || !sste_mult128(k)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(meta_prev, 16) || !sste_aligned(meta_cur, 16) || !sste_aligned(count_dev, 8)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_vec = sste_meta_bytes(rows, k) / 16;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SSTE_CUDA_TRY(cudaMemsetAsync(count_dev, 0, sizeof(unsigned long long), s));
    sste_launch(flip_count_kernel, dim3(grid_for(n_vec, ctx->sm_count)), dim3(EW_THREADS), 0, s,
                static_cast<const uint4 *>(meta_prev), static_cast<const uint4 *>(meta_cur), n_vec, count_dev);
    return launch_result();
}

extern "C" sste_status sste_decompress(sste_ctx *ctx, const void *vals, const void *meta, int rows, int k, sste_dtype dt,
                                       void *dense_out, void *stream)
{
    if (!ctx || !vals || !meta || !dense_out) return SSTE_ERR_INVALID_ARG;
    if (dt != SSTE_BF16 && dt != SSTE_E4M3 && dt != SSTE_E5M2) return SSTE_ERR_DTYPE;
    if (!sste_mult128(rows) || !sste_mult128(k)) return SSTE_ERR_SHAPE;
    if (!sste_aligned(vals, 16) || !sste_aligned(meta, 16) || !sste_aligned(dense_out, 16)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const bool eight = (dt != SSTE_BF16);
    const size_t n_units = static_cast<size_t>(rows) * k / (eight ? 32 : 16);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (eight)
        sste_launch(decompress_kernel<true>, dim3(grid_for(n_units, ctx->sm_count)), dim3(EW_THREADS), 0, s,
                    static_cast<const uint4 *>(vals), static_cast<const uint8_t *>(meta), k, n_units,
                    static_cast<uint4 *>(dense_out));
    else
        sste_launch(decompress_kernel<false>, dim3(grid_for(n_units, ctx->sm_count)), dim3(EW_THREADS), 0, s,
                    static_cast<const uint4 *>(vals), static_cast<const uint8_t *>(meta), k, n_units,
                    static_cast<uint4 *>(dense_out));
    return launch_result();
}

extern "C" int sste_padded_dim(int n) { return n <= 0 ? 0 : (n + 127) / 128 * 128; }

extern "C" sste_status sste_pad_2d(sste_ctx *ctx, const void *src, int rows, int cols, void *dst, int rows_p, int cols_p,
                                   void *stream)
{
    if (!ctx || !src || !dst) return SSTE_ERR_INVALID_ARG;
    if (rows <= 0 || cols <= 0 || rows_p < rows || cols_p < cols || cols_p % 8 != 0) return SSTE_ERR_SHAPE;
    if (!sste_aligned(src, 2) || !sste_aligned(dst, 16)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n_vec = static_cast<size_t>(rows_p) * cols_p / 8;
    sste_launch(pad_2d_kernel, dim3(grid_for(n_vec, ctx->sm_count)), dim3(EW_THREADS), 0, static_cast<cudaStream_t>(stream),
                static_cast<const uint16_t *>(src), rows, cols, static_cast<uint4 *>(dst), cols_p, n_vec);
    return launch_result();
}

extern "C" sste_status sste_crop_2d(sste_ctx *ctx, const void *src, int rows_p, int cols_p, void *dst, int rows, int cols,
                                    void *stream)
{
    if (!ctx || !src || !dst) return SSTE_ERR_INVALID_ARG;
    if (rows <= 0 || cols <= 0 || rows_p < rows || cols_p < cols) return SSTE_ERR_SHAPE;
    if (!sste_aligned(src, 2) || !sste_aligned(dst, 2)) return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    const size_t n = static_cast<size_t>(rows) * cols;
    sste_launch(crop_2d_kernel, dim3(grid_for(n, ctx->sm_count)), dim3(EW_THREADS), 0, static_cast<cudaStream_t>(stream),
                static_cast<const uint16_t *>(src), cols_p, static_cast<uint16_t *>(dst), cols, n);
    return launch_result();
}

extern "C" sste_status sste_debug_mvue_groups(sste_ctx *ctx, const void *a, const void *k24, size_t n, void *pos_out,
                                              void *val_out, void *stream)
{
    if (!ctx || !a || !k24 || !pos_out || !val_out || n == 0) return SSTE_ERR_INVALID_ARG;
    if (!sste_aligned(a, 8) || !sste_aligned(k24, 4) || !sste_aligned(pos_out, 4) || !sste_aligned(val_out, 8))
        return SSTE_ERR_ALIGN;
    sste_device_guard guard(ctx->device);
    if (!guard.ok) return SSTE_ERR_CUDA;
    sste_launch(mvue_groups_kernel, dim3(grid_for(n, ctx->sm_count)), dim3(EW_THREADS), 0, static_cast<cudaStream_t>(stream),
                static_cast<const uint2 *>(a), static_cast<const uint32_t *>(k24), n, static_cast<uint32_t *>(pos_out),
                static_cast<float2 *>(val_out));
    return launch_result();
}
