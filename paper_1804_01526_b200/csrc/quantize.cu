// FP32 -> block-floating-point conversion kernels (the FP-to-BFP step of Sec. 4.1 / Sec. 5.3)
// and the inverse helpers used for inspection. HBM-bound: every FP32 element is read once,
// one (or two) mantissa bytes and 1/b exponent bytes are written.
//
// Kernels
//   quant_row_fast   blocks along contiguous rows, b in {32,64,128,256}: 8 elements per
//                    thread (two 128-bit loads, one Philox call in stochastic mode), block
//                    max by warp shuffles, exponents staged in shared memory so that the
//                    [kb][row] exponent array is written in full 32-byte sectors.
//   quant_row_flat   the same for row lengths that are not a multiple of 512 (K % b == 0): 8-element
//                    groups numbered through the whole matrix, no ragged last tile.
//   quant_col_tma    blocks down the columns, b in {32,64,128}, 16-byte aligned pitch: persistent
//                    CTAs stream 128 x 64 FP32 tiles through a TMA pipeline and write the packed,
//                    transposed tile with a swizzled TMA store (full lines in both directions).
//   quant_col_fast   blocks down the columns, any b <= 128 and any pitch: a (<=128) x 32 FP32
//                    panel is read with coalesced row loads into shared memory, reduced down the
//                    columns by four threads per column and written transposed.
//   tile_kernel      t x t weight tiles (t <= 128): one pass writes both packed views and
//                    the tile exponent grid.
//   exps_* / mant_generic   two-pass path for every other geometry (any b, any alignment).
#include "common.cuh"
#include "tc_ptx.cuh"

// This file is compiled twice. Part 1 (default) is the library's quantiser; part 2 holds only the launches of the
// full-tile kernel for tiles of 32 and 64, built with another ptxas level (see build.py): measured on 8192 x 8192,
// t = 64, the in-place update takes 111 instead of 129 us and the narrow views 48 instead of 56 us that way, while the
// same level costs tiles of 128 and the other kernels of this file time.
#ifndef HBFP_QUANT_PART
#define HBFP_QUANT_PART 1
#endif

namespace hbfp {
namespace {

// ------------------------------------------------------------------------------ arithmetic

struct QParams {
    int m;          // mantissa bits
    int qmax;       // 2^(m-1) - 1
    int exp_mode;
    int rounding;
    uint32_t key0, key1, stream_id;
};

__device__ __forceinline__ uint32_t abs_bits(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// Shared exponent (of the mantissa LSB) from the largest |x| of the block, given as its bit
// pattern: floor(log2 amax) + 1 is the biased exponent field minus 126.
__device__ __forceinline__ int block_exponent(uint32_t amax_bits, int m, int exp_mode) {
    int E = (int)(amax_bits >> 23);
    int e = E - 126;
    if (exp_mode == 1 && E != 0 && (amax_bits & 0x7fffffu) == 0u) e -= 1;
    int s = e - (m - 1);
    s = s < -63 ? -63 : s;
    return s > 127 ? 127 : s;
}

__device__ __forceinline__ float pow2f(int e) {   // 2^e for e in [-126, 127]
    return __uint_as_float((uint32_t)(e + 127) << 23);
}

__device__ __forceinline__ int clampq(int q, int qmax) { return max(-qmax, min(qmax, q)); }

// Bit pattern of max(m, |a|, |b|) for finite values, in one three-input instruction.
__device__ __forceinline__ uint32_t max3_abs_bits(uint32_t m, float a, float b) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(__uint_as_float(m)), "f"(fabsf(a)), "f"(fabsf(b)));
    return __float_as_uint(d);
}

// Stochastic rounding of two neighbours whose 16-bit draws are the halves of one word w: the
// floors of (Y + r) / 2^16 are the upper halfwords of the two sums, clamped as a signed pair.
// Returns the two mantissas as packed signed halfwords (element 0 in the low half).
__device__ __forceinline__ uint32_t round_sr_pair(float x0, float x1, float scale, uint32_t w, uint32_t qmax2, uint32_t nqmax2) {
    const int t0 = __float2int_rd(__fmul_rn(x0, scale)) + (int)(w & 0xFFFFu);
    const int t1 = __float2int_rd(__fmul_rn(x1, scale)) + (int)(w >> 16);
    const uint32_t h = __byte_perm((uint32_t)t0, (uint32_t)t1, 0x7632);
    return __vmaxs2(__vmins2(h, qmax2), nqmax2);
}

// The same for two values whose draws r0, r1 (16 bits each) come from different places.
__device__ __forceinline__ uint32_t round_sr_pair2(float x0, float x1, float scale, uint32_t r0, uint32_t r1, uint32_t qmax2, uint32_t nqmax2) {
    const int t0 = __float2int_rd(__fmul_rn(x0, scale)) + (int)r0;
    const int t1 = __float2int_rd(__fmul_rn(x1, scale)) + (int)r1;
    const uint32_t h = __byte_perm((uint32_t)t0, (uint32_t)t1, 0x7632);
    return __vmaxs2(__vmins2(h, qmax2), nqmax2);
}

// Nearest-even rounding of two values, clamped as a signed halfword pair (m <= 12: the unclamped
// value, at most 2^(m-1) in magnitude, fits a halfword).
__device__ __forceinline__ uint32_t round_rne_pair(float x0, float x1, float scale, uint32_t qmax2, uint32_t nqmax2) {
    const int q0 = __float2int_rn(__fmul_rn(x0, scale)), q1 = __float2int_rn(__fmul_rn(x1, scale));
    const uint32_t h = __byte_perm((uint32_t)q0, (uint32_t)q1, 0x5410);
    return __vmaxs2(__vmins2(h, qmax2), nqmax2);
}

__device__ __forceinline__ uint32_t qmax_pair(int qmax) { return (uint32_t)qmax * 0x10001u; }
__device__ __forceinline__ uint32_t neg_qmax_pair(int qmax) { return ((uint32_t)(-qmax) & 0xFFFFu) * 0x10001u; }

// Bytes of the mantissa planes from two halfword pairs (four mantissas): the 8-bit plane, or for
// two planes (q = 16 hi + lo) bits 4..11 and bits 0..3 of every halfword.
template <int PLANES>
__device__ __forceinline__ void pack4(uint32_t h01, uint32_t h23, uint32_t& hi, uint32_t& lo) {
    if (PLANES == 1) {
        hi = __byte_perm(h01, h23, 0x6420);
        lo = 0;
    } else {
        hi = __byte_perm((h01 >> 4) & 0x00FF00FFu, (h23 >> 4) & 0x00FF00FFu, 0x6420);
        lo = __byte_perm(h01 & 0x000F000Fu, h23 & 0x000F000Fu, 0x6420);
    }
}

// Largest |x| of eight values, as a bit pattern.
__device__ __forceinline__ uint32_t amax8_bits(const float (&e8)[8]) {
    uint32_t am = 0;
#pragma unroll
    for (int j = 0; j < 8; j += 2) am = max3_abs_bits(am, e8[j], e8[j + 1]);
    return am;
}

// Rounds eight consecutive values that share the exponent s (w: their eight 16-bit draws in
// stochastic mode) and packs the plane(s), eight bytes each.
template <bool SR, int PLANES>
__device__ __forceinline__ void quantize_pack8(const float (&e8)[8], int s, const QParams& p, uint4 w, uint2& hi, uint2& lo) {
    const uint32_t qm = qmax_pair(p.qmax), nqm = neg_qmax_pair(p.qmax);
    const float sc = pow2f(SR ? 16 - s : -s);
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    uint32_t h[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
        h[j] = SR ? round_sr_pair(e8[2 * j], e8[2 * j + 1], sc, ww[j], qm, nqm) : round_rne_pair(e8[2 * j], e8[2 * j + 1], sc, qm, nqm);
    pack4<PLANES>(h[0], h[1], hi.x, lo.x);
    pack4<PLANES>(h[2], h[3], hi.y, lo.y);
}

// round-half-even( x * 2^-s ), saturated
__device__ __forceinline__ int round_rne(float x, int s, int qmax) {
    float y = __fmul_rn(x, pow2f(-s));           // s >= -63 and s <= 126 for finite input, m >= 3
    return clampq(__float2int_rn(y), qmax);
}

// stochastic: floor( (floor(fl32(x * 2^(16-s))) + r) / 2^16 ), saturated
__device__ __forceinline__ int round_sr(float x, int s, int qmax, uint32_t r) {
    float y = __fmul_rn(x, pow2f(16 - s));
    int Y = __float2int_rd(y);
    return clampq((Y + (int)r) >> 16, qmax);
}

// Philox4x32-10 (Salmon et al., SC'11).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint4 draws_of_group(const QParams& p, uint64_t g) {
    return philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), p.stream_id, 0u, p.key0, p.key1);
}

__device__ __forceinline__ uint32_t draw_from(uint4 w, uint32_t lane8) {   // lane8 = L & 7
    uint32_t word = (lane8 >> 1) == 0 ? w.x : (lane8 >> 1) == 1 ? w.y : (lane8 >> 1) == 2 ? w.z : w.w;
    return (word >> (16u * (lane8 & 1u))) & 0xFFFFu;
}

__device__ __forceinline__ uint32_t draw_of_element(const QParams& p, uint64_t L) {
    return draw_from(draws_of_group(p, L >> 3), (uint32_t)(L & 7));
}

__device__ __forceinline__ int quantize_one(float x, int s, const QParams& p, uint64_t L) {
    if (p.rounding == 0) return round_rne(x, s, p.qmax);
    return round_sr(x, s, p.qmax, draw_of_element(p, L));
}

// ------------------------------------------------------------------------------ quant_row_fast

// LPB = lanes per block (b = 8 * LPB). CTA: 256 threads, tile 32 rows x 512 columns.
template <int LPB, bool SR, int PLANES>
__global__ void __launch_bounds__(256)
quant_row_fast(const float* __restrict__ x, int64_t rows, int64_t K, int64_t ld, QParams p,
               int8_t* __restrict__ mant, int64_t kst, int64_t plane_stride,
               int8_t* __restrict__ exps, int64_t rs, int64_t nkb, const int8_t* __restrict__ given = nullptr) {
    // given != nullptr: one exponent per row for the whole axis, computed beforehand (a block longer than the
    // tile); the kernel then only rounds and packs
    constexpr int B = 8 * LPB;
    constexpr int KB_PER_SPAN = 256 / B;            // blocks in one warp span of 256 columns
    constexpr int KB_PER_TILE = 512 / B;
    __shared__ int8_t s_exps[KB_PER_TILE][32];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t r0 = (int64_t)blockIdx.y * 32;
    const int64_t c0 = (int64_t)blockIdx.x * 512;

    for (int i = tid; i < KB_PER_TILE * 32; i += 256) (&s_exps[0][0])[i] = 0;
    __syncthreads();

    // warp w owns rows r0 + 4w .. +3, both spans: 8 items, in two batches of 4 rows.
#pragma unroll
    for (int span = 0; span < 2; ++span) {
        float4 v[4][2];
        const int64_t col = c0 + span * 256 + lane * 8;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t r = r0 + warp * 4 + i;
            if (r < rows && col < K) {
                const float4* src = reinterpret_cast<const float4*>(x + r * ld + col);
                v[i][0] = __ldcs(src);
                v[i][1] = __ldcs(src + 1);
            } else {
                v[i][0] = make_float4(0.f, 0.f, 0.f, 0.f);
                v[i][1] = v[i][0];
            }
        }
        // the draws do not depend on the data: they are made while the loads are in flight
        uint4 wd[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            wd[i] = make_uint4(0u, 0u, 0u, 0u);
            if (SR) wd[i] = draws_of_group(p, (uint64_t)((r0 + warp * 4 + i) * K + col) >> 3);   // a multiple of 8 on this path
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t r = r0 + warp * 4 + i;
            const float e8[8] = {v[i][0].x, v[i][0].y, v[i][0].z, v[i][0].w,
                                 v[i][1].x, v[i][1].y, v[i][1].z, v[i][1].w};
            uint32_t am = amax8_bits(e8);
#pragma unroll
            for (int off = 1; off < LPB; off <<= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
            const int s = given ? (r < rows ? (int)given[r] : -63) : block_exponent(am, p.m, p.exp_mode);
            const uint4 w = wd[i];
            uint2 hi, lo;
            quantize_pack8<SR, PLANES>(e8, s, p, w, hi, lo);
            if (r < rows && col < kst) {
                *reinterpret_cast<uint2*>(mant + r * kst + col) = hi;
                if (PLANES == 2) *reinterpret_cast<uint2*>(mant + plane_stride + r * kst + col) = lo;
            }
            if ((lane % LPB) == 0 && r < rows && col < K)
                s_exps[span * KB_PER_SPAN + lane / LPB][warp * 4 + i] = (int8_t)s;
        }
    }
    __syncthreads();
    if (given) return;
    // exponents: [kb][row], 32 rows of one block are 32 contiguous bytes.
    const int64_t kb0 = c0 / B;
    for (int i = tid; i < KB_PER_TILE * 8; i += 256) {
        const int kbl = i >> 3, part = i & 7;
        const int64_t kb = kb0 + kbl, r = r0 + part * 4;
        if (kb < nkb && r < rs)
            *reinterpret_cast<uint32_t*>(exps + kb * rs + r) =
                *reinterpret_cast<const uint32_t*>(&s_exps[kbl][part * 4]);
    }
}

// ------------------------------------------------------------------------------ quant_col_fast

// Blocks down the columns of x [K][R] (contract axis 0); output rows are the columns of x.
// CTA: 128 threads = 32 columns x 4 row slots; panel = G blocks of b <= 128 k-rows (G * padded b
// = 128) by 32 columns: 16 KB of shared memory, so a dozen CTAs fit an SM and cover the memory
// latency. Each thread keeps its 32 values in registers between the max and the rounding pass.
constexpr int COLT = 32;

template <int PLANES, int RQ>      // RQ = bp / 4: padded rows per thread and block (8, 16 or 32)
__global__ void __launch_bounds__(128)
quant_col_fast(const float* __restrict__ x, int64_t K, int64_t R, int64_t ld, int b, QParams p,
               int8_t* __restrict__ mant, int64_t kst, int64_t plane_stride,
               int8_t* __restrict__ exps, int64_t rs, int64_t nkb, int vec_ok) {
    constexpr int G = 32 / RQ;             // blocks per panel: G * bp = 128 padded rows
    constexpr int BP = 4 * RQ;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int krows = G * b;
    float* tile = reinterpret_cast<float*>(smem_raw);                      // [krows][COLT]
    uint32_t* pmax = reinterpret_cast<uint32_t*>(tile + (size_t)krows * COLT);   // [G][4][COLT]
    uint4* rnd = reinterpret_cast<uint4*>(pmax + (size_t)G * 4 * COLT);    // [krows][COLT/8] (stochastic only)

    const int tid = threadIdx.x, c = tid & 31, q = tid >> 5;
    const int64_t kb0 = (int64_t)blockIdx.y * G;
    const int64_t c0 = (int64_t)blockIdx.x * COLT;
    const int64_t k0 = kb0 * b;
    const int rows_here = (int)min((int64_t)krows, K - k0);

    // 1. coalesced load of the panel (zero beyond the matrix).
    if (vec_ok) {
        for (int i = tid; i < rows_here * (COLT / 4); i += 128) {
            const int kk = i >> 3, c4 = (i & 7) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c0 + c4 < R) v = __ldcs(reinterpret_cast<const float4*>(x + (k0 + kk) * ld + c0 + c4));   // R % 4 == 0 here
            *reinterpret_cast<float4*>(tile + kk * COLT + c4) = v;
        }
    } else {
        for (int i = tid; i < rows_here * COLT; i += 128) {
            const int kk = i >> 5, cc = i & 31;
            tile[kk * COLT + cc] = (c0 + cc < R) ? x[(k0 + kk) * ld + c0 + cc] : 0.f;
        }
    }
    // 2. stochastic mode: one Philox call per 8 consecutive source elements of a row.
    const bool group_ok = (R % 8) == 0;     // then L = k*R + col has L & 7 == col & 7 and groups align
    if (p.rounding == 1 && group_ok) {
        for (int i = tid; i < rows_here * (COLT / 8); i += 128) {
            const int kk = i >> 2, g8 = i & 3;
            const uint64_t L = (uint64_t)((k0 + kk) * R + c0 + g8 * 8);
            rnd[i] = draws_of_group(p, L >> 3);
        }
    }
    __syncthreads();

    // 3. thread (q, c) takes quarter q of every block of column c into registers.
    float v[G][RQ];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        uint32_t am = 0;
#pragma unroll
        for (int j = 0; j < RQ; ++j) {
            const int kk = g * b + q * RQ + j;
            const bool valid = q * RQ + j < b && kk < rows_here;
            v[g][j] = valid ? tile[kk * COLT + c] : 0.f;
            am = max(am, abs_bits(v[g][j]));
        }
        pmax[(g * 4 + q) * COLT + c] = am;
    }
    __syncthreads();

    const int64_t col = c0 + c;
    if (col >= R) return;
    const uint16_t* rnd16 = reinterpret_cast<const uint16_t*>(rnd);
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int64_t kb = kb0 + g;
        if (kb < nkb) {
            const uint32_t am = max(max(pmax[(g * 4 + 0) * COLT + c], pmax[(g * 4 + 1) * COLT + c]),
                                    max(pmax[(g * 4 + 2) * COLT + c], pmax[(g * 4 + 3) * COLT + c]));
            const int s = block_exponent(am, p.m, p.exp_mode);
            if (q == 0) exps[kb * rs + col] = (int8_t)s;
            int8_t* dst = mant + col * kst + kb * BP + q * RQ;
#pragma unroll
            for (int w0 = 0; w0 < RQ; w0 += 8) {
                uint32_t hi[2] = {0, 0}, lo[2] = {0, 0};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int kk = g * b + q * RQ + w0 + j;
                    int qv;
                    if (p.rounding == 0) qv = round_rne(v[g][w0 + j], s, p.qmax);
                    else if (group_ok) qv = round_sr(v[g][w0 + j], s, p.qmax, rnd16[((kk < rows_here ? kk : 0) * (COLT / 8) + (c >> 3)) * 8 + (c & 7)]);
                    else qv = round_sr(v[g][w0 + j], s, p.qmax, draw_of_element(p, (uint64_t)((k0 + kk) * R + col)));
                    if (!(q * RQ + w0 + j < b && kk < rows_here)) qv = 0;     // padding stays zero whatever the draw
                    if (PLANES == 1) {
                        hi[j >> 2] |= (uint32_t)(qv & 0xff) << (8 * (j & 3));
                    } else {
                        hi[j >> 2] |= (uint32_t)((qv >> 4) & 0xff) << (8 * (j & 3));
                        lo[j >> 2] |= (uint32_t)(qv & 15) << (8 * (j & 3));
                    }
                }
                *reinterpret_cast<uint2*>(dst + w0) = make_uint2(hi[0], hi[1]);
                if (PLANES == 2) *reinterpret_cast<uint2*>(dst + plane_stride + w0) = make_uint2(lo[0], lo[1]);
            }
            // zero the row tail [nkb*bp, kst) once
            if (kb == nkb - 1 && q == 0) {
                for (int64_t o = nkb * BP; o < kst; o += 16) {
                    *reinterpret_cast<uint4*>(mant + col * kst + o) = make_uint4(0, 0, 0, 0);
                    if (PLANES == 2) *reinterpret_cast<uint4*>(mant + plane_stride + col * kst + o) = make_uint4(0, 0, 0, 0);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------ weight tiles

// Writes one quantised t x t tile (qt: [tp][tp] int16, zero padded) into both packed views, with the
// tile's exponent s replicated over its rows and columns, and zeroes the row tails beyond the last tile.
// (u, v) = tile row / tile column; the tile covers hi x wj elements from (i0, j0).
struct TileViews {
    int8_t* mant_c0; int64_t kst0, ps0; int8_t* exps_c0; int64_t rs0, nkb0;
    int8_t* mant_c1; int64_t kst1, ps1; int8_t* exps_c1; int64_t rs1, nkb1;
};

// qt rows have a pitch of tp + 2 halfwords, so that the column reads of view c0 spread over the banks.
// sh: the views take the top bits of the words in qt (an arithmetic shift by sh bits); for wide storage qt
// holds the stored words, i.e. the mantissas plus half a narrow unit (see tile_kernel); sh = 0 copies.
template <int PLANES>
__device__ __forceinline__ void write_tile_views(const int16_t* qt, int tp, int hi, int wj, int64_t i0, int64_t j0,
                                                 int64_t u, int64_t v, int s, int sh, const TileViews& tv, int tid) {
    const int qp = tp + 2;
    const int lg = 31 - __clz(tp >> 2), gmask = (tp >> 2) - 1;       // tp is 32, 64 or 128
    int8_t* const mant_c0 = tv.mant_c0; int8_t* const mant_c1 = tv.mant_c1;
    int8_t* const exps_c0 = tv.exps_c0; int8_t* const exps_c1 = tv.exps_c1;
    const int64_t kst0 = tv.kst0, ps0 = tv.ps0, rs0 = tv.rs0, nkb0 = tv.nkb0;
    const int64_t kst1 = tv.kst1, ps1 = tv.ps1, rs1 = tv.rs1, nkb1 = tv.nkb1;
    // view c1: row i0+ii gets bytes [v*tp, v*tp+tp) = qt[ii][0..tp)
    if (mant_c1) for (int e = tid; e < hi * (tp / 4); e += 256) {
        const int ii = e >> lg, g = (e & gmask) * 4;
        uint32_t h = 0, l = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int q = qt[ii * qp + g + j] >> sh;
            if (PLANES == 1) h |= (uint32_t)(q & 0xff) << (8 * j);
            else { h |= (uint32_t)((q >> 4) & 0xff) << (8 * j); l |= (uint32_t)(q & 15) << (8 * j); }
        }
        int8_t* dst = mant_c1 + (i0 + ii) * kst1 + v * tp + g;
        *reinterpret_cast<uint32_t*>(dst) = h;
        if (PLANES == 2) *reinterpret_cast<uint32_t*>(dst + ps1) = l;
    }
    // view c0: row j0+jj gets bytes [u*tp, u*tp+tp) = qt[0..tp)[jj]
    // (neighbouring threads write neighbouring words of one output row)
    if (mant_c0) for (int e = tid; e < wj * (tp / 4); e += 256) {
        const int jj = e >> lg, g = (e & gmask) * 4;
        uint32_t h = 0, l = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int q = qt[(g + j) * qp + jj] >> sh;
            if (PLANES == 1) h |= (uint32_t)(q & 0xff) << (8 * j);
            else { h |= (uint32_t)((q >> 4) & 0xff) << (8 * j); l |= (uint32_t)(q & 15) << (8 * j); }
        }
        int8_t* dst = mant_c0 + (j0 + jj) * kst0 + u * tp + g;
        *reinterpret_cast<uint32_t*>(dst) = h;
        if (PLANES == 2) *reinterpret_cast<uint32_t*>(dst + ps0) = l;
    }
    // replicated exponents: exps_c1[v][i0+ii], exps_c0[u][j0+jj]
    if (exps_c1) for (int e = tid; e < hi; e += 256) exps_c1[v * rs1 + i0 + e] = (int8_t)s;
    if (exps_c0) for (int e = tid; e < wj; e += 256) exps_c0[u * rs0 + j0 + e] = (int8_t)s;
    // row tails beyond the last tile: zero them (last tile column / last tile row only)
    if (mant_c1 && v == nkb1 - 1)
        for (int64_t e = tid; e < (int64_t)hi * ((kst1 - nkb1 * tp) / 4); e += 256) {
            const int64_t per = (kst1 - nkb1 * tp) / 4, ii = e / per, o = nkb1 * tp + (e % per) * 4;
            *reinterpret_cast<uint32_t*>(mant_c1 + (i0 + ii) * kst1 + o) = 0;
            if (PLANES == 2) *reinterpret_cast<uint32_t*>(mant_c1 + ps1 + (i0 + ii) * kst1 + o) = 0;
        }
    if (mant_c0 && u == nkb0 - 1)
        for (int64_t e = tid; e < (int64_t)wj * ((kst0 - nkb0 * tp) / 4); e += 256) {
            const int64_t per = (kst0 - nkb0 * tp) / 4, jj = e / per, o = nkb0 * tp + (e % per) * 4;
            *reinterpret_cast<uint32_t*>(mant_c0 + (j0 + jj) * kst0 + o) = 0;
            if (PLANES == 2) *reinterpret_cast<uint32_t*>(mant_c0 + ps0 + (j0 + jj) * kst0 + o) = 0;
        }
}


// Stochastic rounding to 16 bits: x * 2^(16-s) reaches 2^31, so the floor form runs in 64 bits.
__device__ __forceinline__ int round_sr_wide(float x, int s, uint32_t r) {
    const long long Y = __float2ll_rd(__fmul_rn(x, pow2f(16 - s)));
    const long long q = (Y + (long long)r) >> 16;
    return (int)max(-32767ll, min(32767ll, q));
}

// Weight matrices with one exponent per t x t tile (Sec. 4.2 "Tiling", t <= 128) and their wide storage
// (Sec. 4.2 "Wide weight storage"): one CTA per tile of w [d0][d1], 256 threads.
//   MODE 3  quantise FP32 weights src (pitch ld) straight to p.m bits (no wide copy)
//   MODE 0  quantise FP32 weights src to wide storage: int16 mantissas `wide` (row-major, pitch d1) and
//           one exponent per tile in grid [tiles along d0][tiles along d1]
//   MODE 1  update: w = fl32(wide * 2^s + src) with src the FP32 update, re-quantised to 16 bits in place
//   MODE 2  read wide storage only
// In every mode, when view pointers are given, the tile goes to the two packed views
//   c1: rows = d0, contraction along d1 (the stored orientation);  c0: rows = d1, contraction along d0
// with, for the wide modes, the top p.m bits of the stored 16-bit words (the mantissa plus half a narrow
// unit: rounded to nearest, clamped to the symmetric range) under the exponent s + 16 - p.m.
// FAST: t, d1 multiples of 8, pitches and bases 16-byte aligned: a thread handles eight consecutive
// weights of a row at a time (two 128-bit loads, one Philox call, 128-bit store of the int16 mantissas).
template <int MODE, int PLANES, bool FAST>
__global__ void __launch_bounds__(256)
tile_kernel(const float* __restrict__ src, int64_t ld, int64_t d0, int64_t d1, int t, int tp, QParams p,
            int16_t* __restrict__ wide, int8_t* __restrict__ grid, int64_t grid_ld, TileViews tv) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int fp = FAST ? t + 4 : t + 1;                                   // pitch of the FP32 tile
    float* tile = reinterpret_cast<float*>(smem_raw);                      // [t][fp]
    const int qp = tp + 2;
    int16_t* qt = reinterpret_cast<int16_t*>(tile + (size_t)t * fp);       // [tp][tp + 2], zero padded
    __shared__ uint32_t s_am[8];
    __shared__ int s_exp;

    const int tid = threadIdx.x, lane = tid & 31, wrow = tid >> 5;
    const int64_t u = blockIdx.y, v = blockIdx.x;       // tile row (along d0), tile column (along d1)
    const int64_t i0 = u * t, j0 = v * t;
    const int hi = (int)min((int64_t)t, d0 - i0), wj = (int)min((int64_t)t, d1 - j0);
    const int G = wj >> 3;                              // FAST: groups of eight per tile row
    const int wbits = MODE == 3 ? p.m : 16, wqmax = MODE == 3 ? p.qmax : 32767;
    // Wide modes: qt holds the stored word the views are cut from: the mantissa plus half a narrow unit,
    // held inside the range whose top bits stay within +-qmax (so the shift alone rounds to nearest and
    // saturates symmetrically). MODE 3 copies (sh = 0).
    const int sh = MODE == 3 ? 0 : 16 - p.m;
    const int half = sh > 0 ? 1 << (sh - 1) : 0;
    const int w_hi = ((p.qmax + 1) << sh) - half - 1, w_lo = -(p.qmax << sh) - half;
    const uint32_t w_hi2 = ((uint32_t)w_hi & 0xFFFFu) * 0x10001u, w_lo2 = ((uint32_t)w_lo & 0xFFFFu) * 0x10001u;
    const uint32_t half2 = (uint32_t)half * 0x10001u;
    auto stored_pair = [&](uint32_t h) { return MODE == 3 ? h : __vadd2(__vmaxs2(__vmins2(h, w_hi2), w_lo2), half2); };
    auto stored_one = [&](int q) { return MODE == 3 ? q : max(w_lo, min(w_hi, q)) + half; };
    for (int e = tid; e < tp * qp / 2; e += 256) reinterpret_cast<uint32_t*>(qt)[e] = 0;
    int s;
    if (MODE == 2) {
        __syncthreads();
        s = grid[u * grid_ld + v];
        if (FAST) {
            for (int item = tid; item < hi * G; item += 256) {
                const int ii = item / G, gj = item - ii * G;
                const uint4 q8 = *reinterpret_cast<const uint4*>(wide + (i0 + ii) * d1 + j0 + 8 * gj);
                uint32_t* dst = reinterpret_cast<uint32_t*>(qt + ii * qp + 8 * gj);
                dst[0] = stored_pair(q8.x); dst[1] = stored_pair(q8.y); dst[2] = stored_pair(q8.z); dst[3] = stored_pair(q8.w);
            }
        } else {
            for (int ii = wrow; ii < hi; ii += 8)
                for (int jj = lane; jj < wj; jj += 32) qt[ii * qp + jj] = (int16_t)stored_one(wide[(i0 + ii) * d1 + j0 + jj]);
        }
    } else {
        const float old_scale = MODE == 1 ? pow2f(grid[u * grid_ld + v]) : 0.f;
        uint32_t am = 0;
        if (FAST) {
            for (int item = tid; item < hi * G; item += 256) {
                const int ii = item / G, gj = item - ii * G;
                const float4* sp = reinterpret_cast<const float4*>(src + (i0 + ii) * ld + j0 + 8 * gj);
                float4 a = __ldcs(sp), b = __ldcs(sp + 1);
                if (MODE == 1) {
                    const uint4 q8 = *reinterpret_cast<const uint4*>(wide + (i0 + ii) * d1 + j0 + 8 * gj);
                    a.x = __fadd_rn(__fmul_rn((float)(int16_t)(q8.x & 0xFFFFu), old_scale), a.x);
                    a.y = __fadd_rn(__fmul_rn((float)(int16_t)(q8.x >> 16), old_scale), a.y);
                    a.z = __fadd_rn(__fmul_rn((float)(int16_t)(q8.y & 0xFFFFu), old_scale), a.z);
                    a.w = __fadd_rn(__fmul_rn((float)(int16_t)(q8.y >> 16), old_scale), a.w);
                    b.x = __fadd_rn(__fmul_rn((float)(int16_t)(q8.z & 0xFFFFu), old_scale), b.x);
                    b.y = __fadd_rn(__fmul_rn((float)(int16_t)(q8.z >> 16), old_scale), b.y);
                    b.z = __fadd_rn(__fmul_rn((float)(int16_t)(q8.w & 0xFFFFu), old_scale), b.z);
                    b.w = __fadd_rn(__fmul_rn((float)(int16_t)(q8.w >> 16), old_scale), b.w);
                }
                float4* tp4 = reinterpret_cast<float4*>(tile + ii * fp + 8 * gj);
                tp4[0] = a; tp4[1] = b;
                const float e8[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                am = max(am, amax8_bits(e8));
            }
        } else {
            for (int ii = wrow; ii < hi; ii += 8)
                for (int jj = lane; jj < wj; jj += 32) {
                    float val = src[(i0 + ii) * ld + j0 + jj];
                    if (MODE == 1) val = __fadd_rn(__fmul_rn((float)wide[(i0 + ii) * d1 + j0 + jj], old_scale), val);
                    tile[ii * fp + jj] = val;
                    am = max(am, abs_bits(val));
                }
        }
        for (int off = 16; off > 0; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
        if (lane == 0) s_am[wrow] = am;
        __syncthreads();
        if (tid == 0) {
            uint32_t a = 0;
            for (int i = 0; i < 8; ++i) a = max(a, s_am[i]);
            s_exp = block_exponent(a, wbits, p.exp_mode);
            if (grid) grid[u * grid_ld + v] = (int8_t)s_exp;
        }
        __syncthreads();
        s = s_exp;
        if (FAST) {
            const uint32_t qm = qmax_pair(wqmax), nqm = neg_qmax_pair(wqmax);
            for (int item = tid; item < hi * G; item += 256) {
                const int ii = item / G, gj = item - ii * G;
                const float4* tp4 = reinterpret_cast<const float4*>(tile + ii * fp + 8 * gj);
                const float4 a = tp4[0], b = tp4[1];
                const float e8[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                uint4 w = make_uint4(0u, 0u, 0u, 0u);
                if (p.rounding == 1) w = draws_of_group(p, (uint64_t)((i0 + ii) * d1 + j0 + 8 * gj) >> 3);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
                uint32_t h[4];
                if (MODE == 3) {
                    // at most 12 bits: the packed halfword forms
                    const float sc = pow2f(p.rounding == 1 ? 16 - s : -s);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        h[j] = p.rounding == 1 ? round_sr_pair(e8[2 * j], e8[2 * j + 1], sc, ww[j], qm, nqm)
                                               : round_rne_pair(e8[2 * j], e8[2 * j + 1], sc, qm, nqm);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        int q0, q1;
                        if (p.rounding == 0) {
                            q0 = round_rne(e8[2 * j], s, 32767);
                            q1 = round_rne(e8[2 * j + 1], s, 32767);
                        } else {
                            q0 = round_sr_wide(e8[2 * j], s, ww[j] & 0xFFFFu);
                            q1 = round_sr_wide(e8[2 * j + 1], s, ww[j] >> 16);
                        }
                        h[j] = ((uint32_t)q0 & 0xFFFFu) | ((uint32_t)q1 << 16);
                    }
                }
                uint32_t* dst = reinterpret_cast<uint32_t*>(qt + ii * qp + 8 * gj);
                dst[0] = stored_pair(h[0]); dst[1] = stored_pair(h[1]); dst[2] = stored_pair(h[2]); dst[3] = stored_pair(h[3]);
                if (MODE != 3) *reinterpret_cast<uint4*>(wide + (i0 + ii) * d1 + j0 + 8 * gj) = make_uint4(h[0], h[1], h[2], h[3]);
            }
        } else {
            for (int ii = wrow; ii < hi; ii += 8)
                for (int jj = lane; jj < wj; jj += 32) {
                    const float val = tile[ii * fp + jj];
                    const uint64_t L = (uint64_t)((i0 + ii) * d1 + j0 + jj);
                    int q;
                    if (MODE == 3) q = quantize_one(val, s, p, L);
                    else if (p.rounding == 0) q = round_rne(val, s, 32767);
                    else q = round_sr_wide(val, s, draw_of_element(p, L));
                    qt[ii * qp + jj] = (int16_t)stored_one(q);
                    if (MODE != 3) wide[(i0 + ii) * d1 + j0 + jj] = (int16_t)q;
                }
        }
    }
    if (tv.mant_c0 == nullptr && tv.mant_c1 == nullptr) return;
    __syncthreads();
    write_tile_views<PLANES>(qt, tp, hi, wj, i0, j0, u, v, s + sh, sh, tv, tid);
}

// Full tiles of 32, 64 or 128 (the tile is its own padded width), aligned rows: the same arithmetic as
// tile_kernel with far fewer instructions per weight. A thread keeps its groups of eight weights in registers
// between the maximum and the rounding pass (no FP32 tile in shared memory); the rounded words go to a 16-bit
// tile in shared memory once, from which view c1 leaves as 8-byte pieces cut by byte permutes and view c0 as
// the byte-transposes of 4 x 4 blocks (eight permutes per block) instead of one shared-memory load, shift and
// mask per byte. ROWS4 = 4 x 4 blocks stacked per thread for view c0 (wider stores per output row).
template <int MODE, int PLANES, int TP>
__global__ void __launch_bounds__(256)
tile_kernel_full(const float* __restrict__ src, int64_t ld, int64_t d0, int64_t d1, QParams p,
                 int16_t* __restrict__ wide, int8_t* __restrict__ grid, int64_t grid_ld, TileViews tv) {
    constexpr int G = TP / 8;                          // groups of eight per tile row
    constexpr int NITEMS = TP * G;                     // groups per tile
    constexpr int ITEMS = (NITEMS + 255) / 256;        // per thread
    constexpr int QP = TP + 8;                         // halfword pitch of qt: rows stay 16-byte aligned
    __shared__ __align__(16) int16_t qt[TP * QP];
    __shared__ uint32_t s_am[8];
    __shared__ int s_exp;
    const int tid = threadIdx.x, lane = tid & 31, wrow = tid >> 5;
    const int64_t u = blockIdx.y, v = blockIdx.x;
    const int64_t i0 = u * TP, j0 = v * TP;
    const int wbits = MODE == 3 ? p.m : 16, wqmax = MODE == 3 ? p.qmax : 32767;
    const int sh = MODE == 3 ? 0 : 16 - p.m;
    const int half = sh > 0 ? 1 << (sh - 1) : 0;
    const int w_hi = ((p.qmax + 1) << sh) - half - 1, w_lo = -(p.qmax << sh) - half;
    const uint32_t w_hi2 = ((uint32_t)w_hi & 0xFFFFu) * 0x10001u, w_lo2 = ((uint32_t)w_lo & 0xFFFFu) * 0x10001u;
    const uint32_t half2 = (uint32_t)half * 0x10001u;
    auto stored_pair = [&](uint32_t h) { return MODE == 3 ? h : __vadd2(__vmaxs2(__vmins2(h, w_hi2), w_lo2), half2); };
    int s;
    if (MODE == 2) {
        s = grid[u * grid_ld + v];
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            const int item = tid + 256 * k;
            if (NITEMS % 256 == 0 || item < NITEMS) {
                const int ii = item / G, gj = item - ii * G;
                const uint4 q8 = *reinterpret_cast<const uint4*>(wide + (i0 + ii) * d1 + j0 + 8 * gj);
                *reinterpret_cast<uint4*>(qt + ii * QP + 8 * gj) = make_uint4(stored_pair(q8.x), stored_pair(q8.y), stored_pair(q8.z), stored_pair(q8.w));
            }
        }
    } else {
        const float old_scale = MODE == 1 ? pow2f(grid[u * grid_ld + v]) : 0.f;
        // the FP32 groups of the tile are requested before anything waits for them; for an update the wide
        // words follow, combined as fl32(wide * 2^s + delta) with one rounding
        float4 a[ITEMS], b[ITEMS];
        uint32_t am = 0;
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            const int item = tid + 256 * k;
            a[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            b[k] = a[k];
            if (NITEMS % 256 == 0 || item < NITEMS) {
                const int ii = item / G, gj = item - ii * G;
                const float4* sp = reinterpret_cast<const float4*>(src + (i0 + ii) * ld + j0 + 8 * gj);
                a[k] = __ldcs(sp);
                b[k] = __ldcs(sp + 1);
            }
        }
        if (MODE == 1) {
#pragma unroll
            for (int k = 0; k < ITEMS; ++k) {
                const int item = tid + 256 * k;
                if (NITEMS % 256 == 0 || item < NITEMS) {
                    const int ii = item / G, gj = item - ii * G;
                    const uint4 q8 = *reinterpret_cast<const uint4*>(wide + (i0 + ii) * d1 + j0 + 8 * gj);
                    a[k].x = __fadd_rn(__fmul_rn((float)(int16_t)(q8.x & 0xFFFFu), old_scale), a[k].x);
                    a[k].y = __fadd_rn(__fmul_rn((float)(int16_t)(q8.x >> 16), old_scale), a[k].y);
                    a[k].z = __fadd_rn(__fmul_rn((float)(int16_t)(q8.y & 0xFFFFu), old_scale), a[k].z);
                    a[k].w = __fadd_rn(__fmul_rn((float)(int16_t)(q8.y >> 16), old_scale), a[k].w);
                    b[k].x = __fadd_rn(__fmul_rn((float)(int16_t)(q8.z & 0xFFFFu), old_scale), b[k].x);
                    b[k].y = __fadd_rn(__fmul_rn((float)(int16_t)(q8.z >> 16), old_scale), b[k].y);
                    b[k].z = __fadd_rn(__fmul_rn((float)(int16_t)(q8.w & 0xFFFFu), old_scale), b[k].z);
                    b[k].w = __fadd_rn(__fmul_rn((float)(int16_t)(q8.w >> 16), old_scale), b[k].w);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            const float e8[8] = {a[k].x, a[k].y, a[k].z, a[k].w, b[k].x, b[k].y, b[k].z, b[k].w};
            am = max(am, amax8_bits(e8));
        }
        for (int off = 16; off > 0; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
        if (lane == 0) s_am[wrow] = am;
        __syncthreads();
        if (tid == 0) {
            uint32_t m8 = 0;
            for (int i = 0; i < 8; ++i) m8 = max(m8, s_am[i]);
            s_exp = block_exponent(m8, wbits, p.exp_mode);
            if (grid) grid[u * grid_ld + v] = (int8_t)s_exp;
        }
        __syncthreads();
        s = s_exp;
        const uint32_t qm = qmax_pair(wqmax), nqm = neg_qmax_pair(wqmax);
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            const int item = tid + 256 * k;
            if (NITEMS % 256 == 0 || item < NITEMS) {
                const int ii = item / G, gj = item - ii * G;
                const float e8[8] = {a[k].x, a[k].y, a[k].z, a[k].w, b[k].x, b[k].y, b[k].z, b[k].w};
                uint4 w = make_uint4(0u, 0u, 0u, 0u);
                if (p.rounding == 1) w = draws_of_group(p, (uint64_t)((i0 + ii) * d1 + j0 + 8 * gj) >> 3);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
                uint32_t h[4];
                if (MODE == 3) {
                    const float sc = pow2f(p.rounding == 1 ? 16 - s : -s);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        h[j] = p.rounding == 1 ? round_sr_pair(e8[2 * j], e8[2 * j + 1], sc, ww[j], qm, nqm)
                                               : round_rne_pair(e8[2 * j], e8[2 * j + 1], sc, qm, nqm);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        int q0, q1;
                        if (p.rounding == 0) {
                            q0 = round_rne(e8[2 * j], s, 32767);
                            q1 = round_rne(e8[2 * j + 1], s, 32767);
                        } else {
                            q0 = round_sr_wide(e8[2 * j], s, ww[j] & 0xFFFFu);
                            q1 = round_sr_wide(e8[2 * j + 1], s, ww[j] >> 16);
                        }
                        h[j] = ((uint32_t)q0 & 0xFFFFu) | ((uint32_t)q1 << 16);
                    }
                }
                *reinterpret_cast<uint4*>(qt + ii * QP + 8 * gj) = make_uint4(stored_pair(h[0]), stored_pair(h[1]), stored_pair(h[2]), stored_pair(h[3]));
                if (MODE != 3) *reinterpret_cast<uint4*>(wide + (i0 + ii) * d1 + j0 + 8 * gj) = make_uint4(h[0], h[1], h[2], h[3]);
            }
        }
    }
    if (tv.mant_c0 == nullptr && tv.mant_c1 == nullptr) return;
    __syncthreads();
    // Bytes of the views from pairs of stored halfwords: plane 0 takes bits [sh + 4 (PLANES - 1), + 8) of each
    // halfword, plane 1 the four bits below; the masks remove what a 32-bit shift drags across the halfwords.
    const int sh_hi = sh + (PLANES == 2 ? 4 : 0);
    auto bytes4 = [&](uint32_t w0, uint32_t w1, int k, uint32_t mask) {
        return __byte_perm((w0 >> k) & mask, (w1 >> k) & mask, 0x6420);
    };
    const int s_view = s + sh;
    // view c1: row i0 + ii, bytes [v TP + 8 gj, + 8)
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        const int item = tid + 256 * k;
        if (NITEMS % 256 == 0 || item < NITEMS) {
            const int ii = item / G, gj = item - ii * G;
            const uint4 q8 = *reinterpret_cast<const uint4*>(qt + ii * QP + 8 * gj);
            int8_t* dst = tv.mant_c1 + (i0 + ii) * tv.kst1 + v * TP + 8 * gj;
            *reinterpret_cast<uint2*>(dst) = make_uint2(bytes4(q8.x, q8.y, sh_hi, 0x00ff00ffu), bytes4(q8.z, q8.w, sh_hi, 0x00ff00ffu));
            if (PLANES == 2)
                *reinterpret_cast<uint2*>(dst + tv.ps1) = make_uint2(bytes4(q8.x, q8.y, sh, 0x000f000fu), bytes4(q8.z, q8.w, sh, 0x000f000fu));
        }
    }
    // view c0: row j0 + jj, bytes [u TP + g, ...): blocks of 4 columns x (4 ROWS4) rows of qt, byte-transposed
    constexpr int ROWS4 = TP >= 64 ? 4 : 1;                            // 16- or 4-byte stores
    constexpr int NBLK = (TP / 4) * (TP / (4 * ROWS4));
#pragma unroll
    for (int k = 0; k < (NBLK + 255) / 256; ++k) {
        const int e = tid + 256 * k;
        if (NBLK % 256 == 0 || e < NBLK) {
            const int jj = (e % (TP / 4)) * 4, g = (e / (TP / 4)) * 4 * ROWS4;
            uint32_t out[PLANES][4][ROWS4];
#pragma unroll
            for (int rb = 0; rb < ROWS4; ++rb) {
                uint2 r[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = *reinterpret_cast<const uint2*>(qt + (g + 4 * rb + i) * QP + jj);
#pragma unroll
                for (int pl = 0; pl < PLANES; ++pl) {
                    const int kk = pl == 0 ? sh_hi : sh;
                    const uint32_t mask = pl == 0 ? 0x00ff00ffu : 0x000f000fu;
                    const uint32_t R0 = bytes4(r[0].x, r[0].y, kk, mask), R1 = bytes4(r[1].x, r[1].y, kk, mask);
                    const uint32_t R2 = bytes4(r[2].x, r[2].y, kk, mask), R3 = bytes4(r[3].x, r[3].y, kk, mask);
                    const uint32_t t0 = __byte_perm(R0, R1, 0x5140), t1 = __byte_perm(R2, R3, 0x5140);
                    const uint32_t t2 = __byte_perm(R0, R1, 0x7362), t3 = __byte_perm(R2, R3, 0x7362);
                    out[pl][0][rb] = __byte_perm(t0, t1, 0x5410);
                    out[pl][1][rb] = __byte_perm(t0, t1, 0x7632);
                    out[pl][2][rb] = __byte_perm(t2, t3, 0x5410);
                    out[pl][3][rb] = __byte_perm(t2, t3, 0x7632);
                }
            }
#pragma unroll
            for (int pl = 0; pl < PLANES; ++pl)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    int8_t* dst = tv.mant_c0 + pl * tv.ps0 + (j0 + jj + c) * tv.kst0 + u * TP + g;
                    if (ROWS4 == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(out[pl][c][0], out[pl][c][1], out[pl][c][2 % ROWS4], out[pl][c][3 % ROWS4]);
                    else if (ROWS4 == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(out[pl][c][0], out[pl][c][1 % ROWS4]);
                    else *reinterpret_cast<uint32_t*>(dst) = out[pl][c][0];
                }
        }
    }
    // replicated exponents, and the row tails beyond the last tile
    if (tid < TP) {
        tv.exps_c1[v * tv.rs1 + i0 + tid] = (int8_t)s_view;
        tv.exps_c0[u * tv.rs0 + j0 + tid] = (int8_t)s_view;
    }
    if (v == tv.nkb1 - 1)
        for (int64_t e = tid; e < (int64_t)TP * ((tv.kst1 - tv.nkb1 * TP) / 4); e += 256) {
            const int64_t per = (tv.kst1 - tv.nkb1 * TP) / 4, ii = e / per, o = tv.nkb1 * TP + (e % per) * 4;
            *reinterpret_cast<uint32_t*>(tv.mant_c1 + (i0 + ii) * tv.kst1 + o) = 0;
            if (PLANES == 2) *reinterpret_cast<uint32_t*>(tv.mant_c1 + tv.ps1 + (i0 + ii) * tv.kst1 + o) = 0;
        }
    if (u == tv.nkb0 - 1)
        for (int64_t e = tid; e < (int64_t)TP * ((tv.kst0 - tv.nkb0 * TP) / 4); e += 256) {
            const int64_t per = (tv.kst0 - tv.nkb0 * TP) / 4, jj = e / per, o = tv.nkb0 * TP + (e % per) * 4;
            *reinterpret_cast<uint32_t*>(tv.mant_c0 + (j0 + jj) * tv.kst0 + o) = 0;
            if (PLANES == 2) *reinterpret_cast<uint32_t*>(tv.mant_c0 + tv.ps0 + (j0 + jj) * tv.kst0 + o) = 0;
        }
}

// ------------------------------------------------------------------------------ generic two-pass path

// Element (r, kk) of the operand view: r = line, kk = position along the contraction axis.
__device__ __forceinline__ float view_at(const float* x, int64_t ld, int axis, int64_t r, int64_t kk) {
    return axis == 1 ? x[r * ld + kk] : x[kk * ld + r];
}

// Pass 1a, blocks along rows: one warp per (line, block).
__global__ void exps_axis1(const float* __restrict__ x, int64_t rows, int64_t K, int64_t ld, int64_t b,
                           int64_t nkb, QParams p, int8_t* __restrict__ exps, int64_t rs) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t item = warp; item < rows * nkb; item += nwarps) {
        const int64_t r = item / nkb, kb = item % nkb;
        const int64_t k1 = min(K, (kb + 1) * b);
        uint32_t am = 0;
        for (int64_t kk = kb * b + lane; kk < k1; kk += 32) am = max(am, abs_bits(x[r * ld + kk]));
        for (int off = 16; off > 0; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
        if (lane == 0) exps[kb * rs + r] = (int8_t)block_exponent(am, p.m, p.exp_mode);
    }
}

// One exponent per whole row (block = 0, "BFP without tiles", Sec. 6) for rows of 2048 G elements: a CTA per row
// keeps the row in registers (eight elements per thread and step, G steps) between the maximum and the rounding,
// so the tensor is read once.
template <int G, bool SR, int PLANES>
__global__ void __launch_bounds__(256)
quant_row_whole(const float* __restrict__ x, int64_t ld, int64_t d1, QParams p, int8_t* __restrict__ mant, int64_t kst,
                int64_t plane_stride, int8_t* __restrict__ exps) {
    __shared__ uint32_t part[8];
    const int tid = threadIdx.x;
    const int64_t r = blockIdx.x;
    const float4* src = reinterpret_cast<const float4*>(x + r * ld);
    float e[G][8];
    uint32_t am = 0;
#pragma unroll
    for (int i = 0; i < G; ++i) {
        const int g = tid + 256 * i;
        const float4 a = __ldg(src + 2 * g), b = __ldg(src + 2 * g + 1);
        e[i][0] = a.x; e[i][1] = a.y; e[i][2] = a.z; e[i][3] = a.w;
        e[i][4] = b.x; e[i][5] = b.y; e[i][6] = b.z; e[i][7] = b.w;
    }
#pragma unroll
    for (int i = 0; i < G; ++i) am = max(am, amax8_bits(e[i]));
    for (int off = 16; off > 0; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
    if ((tid & 31) == 0) part[tid >> 5] = am;
    __syncthreads();
    am = part[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) am = max(am, part[i]);
    const int s = block_exponent(am, p.m, p.exp_mode);
    if (tid == 0) exps[r] = (int8_t)s;
#pragma unroll
    for (int i = 0; i < G; ++i) {
        const int g = tid + 256 * i;
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (SR) w = draws_of_group(p, (uint64_t)(r * d1 + 8 * (int64_t)g) >> 3);
        uint2 hi, lo;
        quantize_pack8<SR, PLANES>(e[i], s, p, w, hi, lo);
        *reinterpret_cast<uint2*>(mant + r * kst + 8 * g) = hi;
        if (PLANES == 2) *reinterpret_cast<uint2*>(mant + plane_stride + r * kst + 8 * g) = lo;
    }
}

// Pass 1b, blocks down columns: one thread per (block, line); neighbouring threads read
// neighbouring addresses.
__global__ void exps_axis0(const float* __restrict__ x, int64_t rows, int64_t K, int64_t ld, int64_t b,
                           int64_t nkb, QParams p, int8_t* __restrict__ exps, int64_t rs) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * nkb) return;
    const int64_t kb = i / rows, r = i % rows;
    const int64_t k1 = min(K, (kb + 1) * b);
    uint32_t am = 0;
    for (int64_t kk = kb * b; kk < k1; ++kk) am = max(am, abs_bits(x[kk * ld + r]));
    exps[kb * rs + r] = (int8_t)block_exponent(am, p.m, p.exp_mode);
}

// Pass 1c, t x t tiles of the stored matrix [d0][d1]: one warp per tile computes the tile's
// exponent and repeats it for every line of the view that crosses the tile.
__global__ void exps_tiles(const float* __restrict__ x, int64_t d0, int64_t d1, int64_t ld, int64_t t,
                           QParams p, int axis, int8_t* __restrict__ exps, int64_t rs, int64_t nu, int64_t nv) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp >= nu * nv) return;
    const int64_t u = warp / nv, v = warp % nv;
    const int64_t i1 = min(d0, (u + 1) * t), j1 = min(d1, (v + 1) * t);
    uint32_t am = 0;
    for (int64_t i = u * t; i < i1; ++i)
        for (int64_t j = v * t + lane; j < j1; j += 32) am = max(am, abs_bits(x[i * ld + j]));
    for (int off = 16; off > 0; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
    const int8_t s = (int8_t)block_exponent(am, p.m, p.exp_mode);
    // axis 1: lines are stored rows, block index is the tile column. axis 0: the transpose.
    if (axis == 1) for (int64_t i = u * t + lane; i < i1; i += 32) exps[v * rs + i] = s;
    else for (int64_t j = v * t + lane; j < j1; j += 32) exps[u * rs + j] = s;
}

// Pass 1d, convolution weights [taps * c_in][c_out] (Sec. 5.1: the two feature-map dimensions are tiled, the
// filter taps are not): one CTA per (input-map tile u, output-map tile v) takes the maximum over every tap
// (a warp per weight row, lanes along the output maps) and repeats the tile's exponent for every line and
// K-block of the two views that cross the tile.
constexpr int CONVW_THREADS = 512;
__global__ void __launch_bounds__(CONVW_THREADS)
exps_conv_tiles(const float* __restrict__ x, int64_t taps, int64_t c_in, int64_t c_out, int64_t ld, int64_t t, QParams p,
                int8_t* __restrict__ exps0, int64_t rs0, int8_t* __restrict__ exps1, int64_t rs1, int64_t nu, int64_t nv,
                int8_t* __restrict__ tile_exps, uint32_t* __restrict__ amax, bool fill) {
    __shared__ uint32_t part[CONVW_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t u = blockIdx.x / nv, v = blockIdx.x % nv;
    const int64_t j1 = min(c_out, (v + 1) * t);
    uint32_t am = 0;
    // with `amax` the rows are split over gridDim.y CTAs that merge their maxima there (exponents come from a
    // second launch with `fill`); without it this CTA scans the whole tile
    for (int64_t r = (int64_t)blockIdx.y * (CONVW_THREADS / 32) + warp; !fill && r < taps * t; r += (int64_t)gridDim.y * (CONVW_THREADS / 32)) {
        const int64_t tap = r / t, ci = u * t + r % t;
        for (int64_t j = v * t + lane; j < j1; j += 32) am = max(am, abs_bits(x[(tap * c_in + ci) * ld + j]));
    }
    for (int off = 16; off > 0; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
    if (lane == 0) part[warp] = am;
    __syncthreads();
    am = part[0];
    for (int i = 1; i < CONVW_THREADS / 32; ++i) am = max(am, part[i]);
    if (amax && !fill) {
        if (threadIdx.x == 0) atomicMax(amax + blockIdx.x, am);
        return;
    }
    if (fill) am = amax[blockIdx.x];
    const int8_t s = (int8_t)block_exponent(am, p.m, p.exp_mode);
    if (tile_exps && threadIdx.x == 0) tile_exps[u * nv + v] = s;
    // view c0 (forward): lines are output maps, K-block (tap, u). view c1: lines are (tap, ci), K-block v.
    if (exps0)
        for (int64_t i = threadIdx.x; i < taps * (j1 - v * t); i += CONVW_THREADS) {
            const int64_t tap = i / (j1 - v * t), j = v * t + i % (j1 - v * t);
            exps0[(tap * nu + u) * rs0 + j] = s;
        }
    if (exps1)
        for (int64_t i = threadIdx.x; i < taps * t; i += CONVW_THREADS) {
            const int64_t tap = i / t, ci = u * t + i % t;
            exps1[v * rs1 + tap * c_in + ci] = s;
        }
}

// Pass 2: one thread per 4 output bytes of a line; reads the exponent written by pass 1.
template <int PLANES>
__global__ void mant_generic(const float* __restrict__ x, int64_t d1, int64_t rows, int64_t K, int64_t ld,
                             int axis, int64_t b, int64_t bp, int64_t nkb, QParams p,
                             const int8_t* __restrict__ exps, int64_t rs, int8_t* __restrict__ mant,
                             int64_t kst, int64_t plane_stride) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t per = kst / 4;
    if (i >= rows * per) return;
    const int64_t r = i / per, o = (i % per) * 4;
    uint32_t h = 0, l = 0;
    const int64_t kb = o / bp;
    if (kb < nkb) {
        const int s = exps[kb * rs + r];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t within = o % bp + j, kk = kb * b + within;
            int q = 0;
            if (within < b && kk < K) {
                const uint64_t L = axis == 1 ? (uint64_t)(r * d1 + kk) : (uint64_t)(kk * d1 + r);
                q = quantize_one(view_at(x, ld, axis, r, kk), s, p, L);
            }
            if (PLANES == 1) h |= (uint32_t)(q & 0xff) << (8 * j);
            else { h |= (uint32_t)((q >> 4) & 0xff) << (8 * j); l |= (uint32_t)(q & 15) << (8 * j); }
        }
    }
    *reinterpret_cast<uint32_t*>(mant + r * kst + o) = h;
    if (PLANES == 2) *reinterpret_cast<uint32_t*>(mant + plane_stride + r * kst + o) = l;
}

// ------------------------------------------------------------------------------ packed im2col gather

// Convolution operand without the FP32 im2col matrix: with a block of c channels along the contraction
// (taps ordered (i, j, channel)) every block of an im2col row is the quantised channel vector of one input
// pixel, so the packed operand [n ho wo][kh kw c] is a gather of the packed per-pixel operand [n h w][c]:
// bp bytes of mantissas and one exponent per tap, zeros (exponent -63, as an all-zero block has) outside the
// image. One warp per output row, 16 bytes per lane and step (row tails beyond the last tap are zeroed too).
constexpr int IM2COL_MAX_TAPS = 64, IM2COL_ROWS = 64;

__global__ void __launch_bounds__(256)
im2col_gather(const int8_t* __restrict__ xm, const int8_t* __restrict__ xe, int kst_x, int64_t ps_x,
              int h, int w, int ho, int wo, int kh, int kw, int pad, int lg_bp, int planes,
              uint32_t rows_out, int kst_out, int64_t ps_out, int64_t rs_out,
              int8_t* __restrict__ om, int8_t* __restrict__ oe) {
    // A CTA takes 64 consecutive output rows, a warp eight of them; the lanes sweep a row 16 bytes at a
    // time. The filter offsets of the taps are tabulated once per CTA, the pixel coordinates once per row
    // (32-bit arithmetic: the host checks the sizes), and the exponents of the 64 rows are collected in
    // shared memory so that each tap's bytes leave as whole sectors.
    __shared__ int8_t s_e[IM2COL_MAX_TAPS][IM2COL_ROWS];
    __shared__ int8_t s_dy[IM2COL_MAX_TAPS], s_dx[IM2COL_MAX_TAPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t r0 = blockIdx.x * IM2COL_ROWS;
    const int taps = kh * kw, chunks = kst_out >> 4;
    if ((int)threadIdx.x < taps) {
        s_dy[threadIdx.x] = (int8_t)((int)threadIdx.x / kw - pad);
        s_dx[threadIdx.x] = (int8_t)((int)threadIdx.x % kw - pad);
    }
    __syncthreads();
    const uint32_t per_img = (uint32_t)(ho * wo);
    // four rows at a time, so that four independent loads are in flight per lane (eight were slower)
    for (int k = 0; k < IM2COL_ROWS / 8; k += 4) {
        int oy[4], ox[4];
        int64_t img_base[4];
        bool live[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t r = r0 + warp * (IM2COL_ROWS / 8) + k + q;
            live[q] = r < rows_out;
            const uint32_t rr = live[q] ? r : 0u;
            const uint32_t img = rr / per_img, rem = rr - img * per_img;
            oy[q] = (int)(rem / (uint32_t)wo);
            ox[q] = (int)(rem - (uint32_t)oy[q] * (uint32_t)wo);
            img_base[q] = (int64_t)img * h * w;
        }
        for (int ck = lane; ck < chunks; ck += 32) {
            const int o = ck << 4;                              // byte offset in the output row
            const int tap = o >> lg_bp, within = o - (tap << lg_bp);
            const int dy = tap < taps ? s_dy[tap] : 0, dx = tap < taps ? s_dx[tap] : 0;
            for (int pl = 0; pl < planes; ++pl) {
                int64_t src[4];
                uint4 v[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int iy = oy[q] + dy, ix = ox[q] + dx;
                    src[q] = (tap < taps && iy >= 0 && iy < h && ix >= 0 && ix < w) ? img_base[q] + iy * w + ix : -1;
                    v[q] = make_uint4(0u, 0u, 0u, 0u);
                    if (src[q] >= 0) v[q] = *reinterpret_cast<const uint4*>(xm + pl * ps_x + src[q] * kst_x + within);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int lr = warp * (IM2COL_ROWS / 8) + k + q;
                    if (live[q]) {
                        *reinterpret_cast<uint4*>(om + pl * ps_out + (int64_t)(r0 + lr) * kst_out + o) = v[q];
                        if (pl == 0 && within == 0 && tap < taps) s_e[tap][lr] = src[q] >= 0 ? xe[src[q]] : (int8_t)-63;
                    }
                }
            }
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < taps * IM2COL_ROWS; idx += 256) {
        const int tap = idx / IM2COL_ROWS, j = idx % IM2COL_ROWS;
        if (r0 + j < rows_out) oe[(int64_t)tap * rs_out + r0 + j] = s_e[tap][j];
    }
}

// Backward-weight operand of a convolution without the FP32 im2col matrix: dW = cols^T dY contracts over the
// output pixels, so cols^T [kh kw c][n h w] is quantised with blocks of b consecutive pixels along each
// (tap, channel) row. A block is a window of the image shifted by the tap, so nothing can be shared between
// taps except the loads: a CTA takes one block of b pixels (whole image rows: b % w == 0, h w % b == 0,
// output as large as the input) and stages the b / w + kh - 1 image rows it touches in shared memory once
// (zeros outside the image). Then, tap by tap and 64 channels at a time, thread (channel, quarter) keeps its
// quarter of the block's pixels in registers between the maximum (exchanged through shared memory) and the
// rounding, and writes its b / 4 mantissa bytes with 16-byte stores.
template <int PLANES, int NPX, bool SR>      // NPX = b / 4 pixels per thread: 4, 8, 16 or 32
__global__ void __launch_bounds__(256)
im2col_cols(const float* __restrict__ x, int h, int w, int lg_w, int c, int kh, int kw, int pad, QParams p,
            int64_t kst, int64_t plane_stride, int64_t rs, int8_t* __restrict__ mant, int8_t* __restrict__ exps) {
    constexpr int B = 4 * NPX;
    constexpr int BP = B <= 32 ? 32 : B <= 64 ? 64 : 128;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* img_rows = reinterpret_cast<float*>(smem_raw);        // [B / w + kh - 1][w][c]
    __shared__ uint32_t pmax[4][64];
    const int tid = threadIdx.x, chl = tid & 63, q = tid >> 6;
    const int64_t pb = blockIdx.x;                               // pixel block
    const int64_t p0 = pb * B;
    const int per_img = h * w;
    const int64_t img = p0 / per_img;
    const int oy0 = (int)((p0 - img * per_img) >> lg_w);
    const int srows = (B >> lg_w) + kh - 1;
    // stage the source rows oy0 - pad .. oy0 + B / w - 1 + (kh - 1 - pad)
    const int row_elems = w * c;
    for (int e = tid * 4; e < srows * row_elems; e += 256 * 4) {
        const int sr = e / row_elems, off = e - sr * row_elems;
        const int iy = oy0 - pad + sr;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (iy >= 0 && iy < h) v = __ldg(reinterpret_cast<const float4*>(x + ((img * h + iy) * (int64_t)w) * c + off));
        *reinterpret_cast<float4*>(img_rows + e) = v;
    }
    __syncthreads();
    const uint32_t qm = qmax_pair(p.qmax), nqm = neg_qmax_pair(p.qmax);
    const int taps = kh * kw;
    // this thread's pixels: column in the image row and offset in the staged rows, worked out once
    int ox_of[NPX], off_of[NPX];
#pragma unroll
    for (int j = 0; j < NPX; ++j) {
        const int px = q * NPX + j;
        ox_of[j] = px & (w - 1);
        off_of[j] = px * c;                                      // ((px >> lg_w) * w + ox) * c
    }
    for (int c0 = 0; c0 < c; c0 += 64) {
        const int ch = c0 + chl;
        const bool live = ch < c;
        for (int tap = 0; tap < taps; ++tap) {
            const int dy = tap / kw, dx = tap - dy * kw - pad;   // dy indexes the staged rows directly
            const float* tap_base = img_rows + (dy * w + dx) * c + (live ? ch : 0);
            float v[NPX];
            uint32_t am = 0;
#pragma unroll
            for (int j = 0; j < NPX; ++j)
                v[j] = (live && (unsigned)(ox_of[j] + dx) < (unsigned)w) ? tap_base[off_of[j]] : 0.f;
#pragma unroll
            for (int j = 0; j < NPX; j += 2) am = max3_abs_bits(am, v[j], v[j + 1]);
            pmax[q][chl] = am;
            __syncthreads();
            am = max(max(pmax[0][chl], pmax[1][chl]), max(pmax[2][chl], pmax[3][chl]));
            __syncthreads();                                     // pmax is rewritten by the next tap
            if (!live) continue;
            const int s = block_exponent(am, p.m, p.exp_mode);
            const int64_t row = (int64_t)tap * c + ch;
            if (q == 0) exps[pb * rs + row] = (int8_t)s;
            const float sc = pow2f(SR ? 16 - s : -s);
            uint32_t hi[NPX / 4], lo[NPX / 4];
#pragma unroll
            for (int wi = 0; wi < NPX / 4; ++wi) {
                uint32_t r[4] = {0u, 0u, 0u, 0u};
                if (SR) {
                    // stochastic rounding draws by the element's index in the activation tensor
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int px = q * NPX + 4 * wi + j, ry = px >> lg_w, ix = (px & (w - 1)) + dx;
                        const int iy = oy0 - pad + ry + dy;
                        if (ix >= 0 && ix < w && iy >= 0 && iy < h)
                            r[j] = draw_of_element(p, (uint64_t)(((img * h + iy) * (int64_t)w + ix) * c + ch));
                    }
                }
                uint32_t h01, h23;
                if (SR) {
                    h01 = round_sr_pair2(v[4 * wi], v[4 * wi + 1], sc, r[0], r[1], qm, nqm);
                    h23 = round_sr_pair2(v[4 * wi + 2], v[4 * wi + 3], sc, r[2], r[3], qm, nqm);
                } else {
                    h01 = round_rne_pair(v[4 * wi], v[4 * wi + 1], sc, qm, nqm);
                    h23 = round_rne_pair(v[4 * wi + 2], v[4 * wi + 3], sc, qm, nqm);
                }
                pack4<PLANES>(h01, h23, hi[wi], lo[wi]);
            }
            int8_t* dst = mant + row * kst + pb * BP + q * NPX;
            if (NPX >= 16) {
#pragma unroll
                for (int i = 0; i < NPX / 16; ++i) {
                    *reinterpret_cast<uint4*>(dst + 16 * i) = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
                    if (PLANES == 2) *reinterpret_cast<uint4*>(dst + plane_stride + 16 * i) = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < NPX / 4; ++i) {
                    *reinterpret_cast<uint32_t*>(dst + 4 * i) = hi[i];
                    if (PLANES == 2) *reinterpret_cast<uint32_t*>(dst + plane_stride + 4 * i) = lo[i];
                }
            }
            if (B < BP && q == 0) {                              // block padding (16-pixel blocks in 32 bytes)
#pragma unroll
                for (int px0 = B; px0 < BP; px0 += 4) {
                    *reinterpret_cast<uint32_t*>(mant + row * kst + pb * BP + px0) = 0u;
                    if (PLANES == 2) *reinterpret_cast<uint32_t*>(mant + plane_stride + row * kst + pb * BP + px0) = 0u;
                }
            }
        }
    }
}

// Filter operand of the backward-data convolution from view c1 of tiled convolution weights: row ci of the result
// is, tap by tap in reversed order, the c_out packed bytes of c1's row (tap, ci) (Sec. 5.1: backward-data is the
// convolution of the output gradient with the filters turned by 180 degrees and their feature-map roles swapped;
// the mantissas and tile exponents are the forward pass's own). One warp per (ci, tap), 16 bytes per lane.
__global__ void __launch_bounds__(256)
conv_dgrad_filters_kernel(const int8_t* __restrict__ m1, const int8_t* __restrict__ e1, int64_t kst1, int64_t ps1,
                          int64_t rs1, int taps, int64_t c_in, int64_t c_out, int t, int planes,
                          int8_t* __restrict__ mo, int8_t* __restrict__ eo, int64_t ksto, int64_t pso, int64_t rso) {
    const int lane = threadIdx.x & 31;
    const int64_t item = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (item >= c_in * taps) return;
    const int64_t ci = item / taps;
    const int tap = (int)(item - ci * taps);
    const int64_t src_row = (int64_t)(taps - 1 - tap) * c_in + ci;
    for (int pl = 0; pl < planes; ++pl)
        for (int64_t o = 16 * lane; o < c_out; o += 512)
            *reinterpret_cast<uint4*>(mo + pl * pso + ci * ksto + (int64_t)tap * c_out + o) =
                *reinterpret_cast<const uint4*>(m1 + pl * ps1 + src_row * kst1 + o);
    const int cb_n = (int)(c_out / t);
    for (int cb = lane; cb < cb_n; cb += 32) eo[((int64_t)tap * cb_n + cb) * rso + ci] = e1[(int64_t)cb * rs1 + src_row];
    // bytes of the row beyond the last tap (the row pitch is a multiple of 128)
    if (tap == taps - 1)
        for (int64_t o = (int64_t)taps * c_out + 16 * lane; o < ksto; o += 512)
            for (int pl = 0; pl < planes; ++pl) *reinterpret_cast<uint4*>(mo + pl * pso + ci * ksto + o) = make_uint4(0u, 0u, 0u, 0u);
}

// ------------------------------------------------------------------------------ inverse helpers

__global__ void unpack_kernel(const int8_t* __restrict__ mant, const int8_t* __restrict__ exps, int64_t rows,
                              int64_t K, int64_t b, int64_t bp, int64_t nkb, int64_t kst, int64_t plane_stride,
                              int planes, int64_t rs, int16_t* __restrict__ q, int8_t* __restrict__ s) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q && i < rows * K) {
        const int64_t r = i / K, kk = i % K, o = (kk / b) * bp + kk % b;
        int v = mant[r * kst + o];
        if (planes == 2) v = v * 16 + mant[plane_stride + r * kst + o];
        q[i] = (int16_t)v;
    }
    if (s && i < rows * nkb) {
        const int64_t r = i / nkb, kb = i % nkb;
        s[i] = exps[kb * rs + r];
    }
}

__global__ void dequant_kernel(const int8_t* __restrict__ mant, const int8_t* __restrict__ exps, int64_t rows,
                               int64_t K, int64_t b, int64_t bp, int64_t kst, int64_t plane_stride, int planes,
                               int64_t rs, float* __restrict__ out, int64_t ld) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * K) return;
    const int64_t r = i / K, kk = i % K, kb = kk / b, o = kb * bp + kk % b;
    int v = mant[r * kst + o];
    if (planes == 2) v = v * 16 + mant[plane_stride + r * kst + o];
    out[r * ld + kk] = ldexpf((float)v, (int)exps[kb * rs + r]);
}

// ------------------------------------------------------------------------------ quant_row_flat

// Blocks along contiguous rows for row lengths that are not a multiple of the 512-column tile of
// quant_row_fast (K % b == 0, e.g. im2col matrices with K = 576 or 1152): the packed rows, padding
// included, are cut into 8-element groups that are numbered through the whole matrix, and a warp takes
// 32 consecutive groups wherever the row boundaries fall, so no lane idles on a ragged last tile.
// CTA: 256 threads x ITEMS groups each (256 ITEMS consecutive groups).
template <int LPB, bool SR, int PLANES, int ITEMS>
__global__ void __launch_bounds__(256)
quant_row_flat(const float* __restrict__ x, int64_t rows, int64_t K, int64_t ld, QParams p,
               int8_t* __restrict__ mant, int64_t kst, int64_t plane_stride,
               int8_t* __restrict__ exps, int64_t rs, uint32_t gpr, uint32_t total_groups) {
    constexpr int B = 8 * LPB;
    const int tid = threadIdx.x, lane = tid & 31;
    const uint32_t g0 = blockIdx.x * (256u * ITEMS) + tid;
    // (row, group in row) of this thread's first group; the next ones are 256 groups further on each
    uint32_t row = g0 / gpr, cg = g0 - row * gpr;
    const uint32_t q256 = 256u / gpr, r256 = 256u - q256 * gpr;
    float4 v[ITEMS][2];
    uint32_t rw[ITEMS], cc[ITEMS];
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        rw[j] = row;
        cc[j] = cg * 8;
        const bool in = g0 + j * 256u < total_groups && cc[j] < K;
        if (in) {
            const float4* src = reinterpret_cast<const float4*>(x + (int64_t)row * ld + cc[j]);
            v[j][0] = __ldcs(src);
            v[j][1] = __ldcs(src + 1);
        } else {
            v[j][0] = make_float4(0.f, 0.f, 0.f, 0.f);
            v[j][1] = v[j][0];
        }
        row += q256;
        cg += r256;
        if (cg >= gpr) { cg -= gpr; ++row; }
    }
    // the draws do not depend on the data: they are made while the loads are in flight
    uint4 wd[ITEMS];
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        wd[j] = make_uint4(0u, 0u, 0u, 0u);
        if (SR) wd[j] = draws_of_group(p, ((uint64_t)rw[j] * (uint64_t)K + cc[j]) >> 3);     // a multiple of 8 on this path
    }
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const bool live = g0 + j * 256u < total_groups;      // uniform over the LPB lanes of a block
        const float e8[8] = {v[j][0].x, v[j][0].y, v[j][0].z, v[j][0].w, v[j][1].x, v[j][1].y, v[j][1].z, v[j][1].w};
        uint32_t am = amax8_bits(e8);
#pragma unroll
        for (int off = 1; off < LPB; off <<= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
        const int s = block_exponent(am, p.m, p.exp_mode);
        const uint4 w = wd[j];
        uint2 hi, lo;
        quantize_pack8<SR, PLANES>(e8, s, p, w, hi, lo);
        if (live) {
            int8_t* dst = mant + (int64_t)rw[j] * kst + cc[j];
            *reinterpret_cast<uint2*>(dst) = hi;
            if (PLANES == 2) *reinterpret_cast<uint2*>(dst + plane_stride) = lo;
            // blocks that lie in the padding beyond K have no exponent
            if ((lane % LPB) == 0 && cc[j] < K) exps[(int64_t)(cc[j] / B) * rs + rw[j]] = (int8_t)s;
        }
    }
}

template <int LPB, int ITEMS>
int launch_row_flat_items(const float* x, int64_t rows, int64_t K, int64_t ld, const QParams& p, const Layout& L,
                          int8_t* mant, int8_t* exps, cudaStream_t st) {
    const uint32_t gpr = (uint32_t)(L.kst / 8), total = (uint32_t)(rows * (L.kst / 8));
    const unsigned grid = (total + 256u * ITEMS - 1u) / (256u * ITEMS);
    if (p.rounding == 1) {
        if (L.planes == 1) quant_row_flat<LPB, true, 1, ITEMS><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, gpr, total);
        else quant_row_flat<LPB, true, 2, ITEMS><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, gpr, total);
    } else {
        if (L.planes == 1) quant_row_flat<LPB, false, 1, ITEMS><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, gpr, total);
        else quant_row_flat<LPB, false, 2, ITEMS><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, gpr, total);
    }
    return launch_status();
}

// Groups per thread: more of them amortise the index arithmetic, fewer keep the register footprint small
// and more loads in flight. Measured on 131072 x 576 (b = 64): eight 68 us, four 58 us, two 61 us with
// nearest-even rounding; 91 / 84 / 82 us with stochastic rounding (the Philox state of every group in flight
// is live). Narrow rows (one or two 128-byte units, e.g. one block of 64 channels per pixel, half of whose
// groups are padding that loads nothing) do best with two.
template <int LPB>
int launch_row_flat(const float* x, int64_t rows, int64_t K, int64_t ld, const QParams& p, const Layout& L,
                    int8_t* mant, int8_t* exps, cudaStream_t st) {
    if (L.kst > 256 && p.rounding == 0) return launch_row_flat_items<LPB, 4>(x, rows, K, ld, p, L, mant, exps, st);
    return launch_row_flat_items<LPB, 2>(x, rows, K, ld, p, L, mant, exps, st);
}

// ------------------------------------------------------------------------------ quant_col_tma

// Blocks down the columns of x [K][R] for b in {32, 64, 128}, the layout of the B operand of a
// forward GEMM. Persistent CTAs stream 128 (k) x 64 (columns) FP32 tiles through a two-stage TMA
// pipeline; thread (column n, quarter q) keeps 32 consecutive k of its column in registers between
// the block maximum and the rounding pass, and the packed tile (64 output rows x 128 mantissa bytes,
// contraction-major) goes back to global memory as one 128B-swizzled TMA store per plane, so both
// directions move full lines whatever the matrix pitch.
constexpr int QC_COLS = 64, QC_ROWS = 128, QC_STAGES = 2, QC_THREADS = 256;
constexpr int QC_IN_BYTES = QC_ROWS * QC_COLS * 4;          // 32 KB
constexpr int QC_OUT_BYTES = QC_COLS * QC_ROWS;             // 8 KB per plane

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int c0, int c1, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1) : "memory");
}

template <int PLANES, int LB, bool SR>      // b = 128 >> LB
__global__ void __launch_bounds__(QC_THREADS)
quant_col_tma(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapM0,
              const __grid_constant__ CUtensorMap mapM1, QParams p, int8_t* __restrict__ exps, int64_t rs,
              int64_t nkb, int64_t K, int64_t R, int tiles_n, int total_tiles, int32_t* status,
              const int8_t* __restrict__ given) {
    // given != nullptr: one exponent per column for the whole axis, computed beforehand (blocks longer than a
    // tile); the kernel then only rounds and packs
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    // [out planes | in stages | draws (stochastic) | block maxima | barriers]
    constexpr int OFF_IN = PLANES * QC_OUT_BYTES;
    constexpr int OFF_RND = OFF_IN + QC_STAGES * QC_IN_BYTES;
    constexpr int OFF_PMAX = OFF_RND + (SR ? QC_ROWS * QC_COLS * 2 : 0);
    constexpr int OFF_BAR = OFF_PMAX + 4 * QC_COLS * 4;
    const float* in = reinterpret_cast<const float*>(base_ptr + OFF_IN);
    uint4* rnd = reinterpret_cast<uint4*>(base_ptr + OFF_RND);
    uint32_t* pmax = reinterpret_cast<uint32_t*>(base_ptr + OFF_PMAX);
    const uint32_t full_bar = base + OFF_BAR;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + OFF_BAR + 8 * QC_STAGES);

    const int tid = threadIdx.x, n = tid & (QC_COLS - 1), q = tid >> 6;
    if (tid == 0) {
        for (int s = 0; s < QC_STAGES; ++s) mbar_init(full_bar + 8 * s, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int first = blockIdx.x, step = gridDim.x;
    if (tid == 0) {
        for (int s = 0; s < QC_STAGES; ++s) {
            const int t = first + s * step;
            if (t < total_tiles) {
                mbar_expect_tx(full_bar + 8 * s, QC_IN_BYTES);
                tma_load_2d(base + OFF_IN + s * QC_IN_BYTES, &mapX, (t % tiles_n) * (QC_COLS * 4), (t / tiles_n) * QC_ROWS, full_bar + 8 * s);
            }
        }
    }
    uint32_t s = 0, ph = 0;
    bool stores_pending = false;
    for (int t = first; t < total_tiles; t += step) {
        const int nt = t % tiles_n, kt = t / tiles_n;
        const int64_t col = (int64_t)nt * QC_COLS + n;
        if (SR) {
            // one Philox call per eight consecutive source elements of a row (R % 8 == 0 here); the draws
            // do not depend on the data, so they are made while the tile may still be in flight (the
            // previous tile's readers of the table are past the barrier that precedes its store)
            for (int i = tid; i < QC_ROWS * (QC_COLS / 8); i += QC_THREADS) {
                const uint64_t L = (uint64_t)((int64_t)kt * QC_ROWS + (i >> 3)) * (uint64_t)R + (uint64_t)(nt * QC_COLS + (i & 7) * 8);
                rnd[i] = draws_of_group(p, L >> 3);
            }
        }
        // (uniform verdict: a wait that gave up in some threads only would split the CTA barriers below)
        if (!__syncthreads_and(mbar_wait(full_bar + 8 * s, ph, abort_flag, status, 601))) break;
        const float* tile = in + (size_t)s * (QC_IN_BYTES / 4);
        float v[32];
        uint32_t am = 0;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            v[j] = tile[(q * 32 + j) * QC_COLS + n];
            v[j + 1] = tile[(q * 32 + j + 1) * QC_COLS + n];
            am = max3_abs_bits(am, v[j], v[j + 1]);
        }
        if (LB < 2) pmax[q * QC_COLS + n] = am;
        // the packed tile of the previous iteration must have left shared memory before it is rewritten
        if (tid == 0 && stores_pending) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncthreads();
        // every thread holds its values in registers now: refill this stage with the tile after next
        if (tid == 0) {
            const int t2 = t + QC_STAGES * step;
            if (t2 < total_tiles) {
                mbar_expect_tx(full_bar + 8 * s, QC_IN_BYTES);
                tma_load_2d(base + OFF_IN + s * QC_IN_BYTES, &mapX, (t2 % tiles_n) * (QC_COLS * 4), (t2 / tiles_n) * QC_ROWS, full_bar + 8 * s);
            }
        }
        if (LB == 0) am = max(max(pmax[n], pmax[QC_COLS + n]), max(pmax[2 * QC_COLS + n], pmax[3 * QC_COLS + n]));
        if (LB == 1) am = max(pmax[(q & 2) * QC_COLS + n], pmax[((q & 2) + 1) * QC_COLS + n]);
        const int sexp = given ? (col < R ? (int)given[col] : -63) : block_exponent(am, p.m, p.exp_mode);
        const int64_t kb = ((int64_t)kt << LB) + (q >> (2 - LB));
        if (!given && (q & ((4 >> LB) - 1)) == 0 && kb < nkb && col < R) exps[kb * rs + col] = (int8_t)sexp;

        uint32_t hi[8], lo[8];
        const uint16_t* rnd16 = reinterpret_cast<const uint16_t*>(rnd);
        const uint32_t qm = qmax_pair(p.qmax), nqm = neg_qmax_pair(p.qmax);
        const float sc = pow2f(SR ? 16 - sexp : -sexp);
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            uint32_t h[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int j = 4 * w + 2 * k;
                if (SR) {
                    // the draws of two vertical neighbours belong to different rows: two table entries
                    h[k] = round_sr_pair2(v[j], v[j + 1], sc, rnd16[(q * 32 + j) * QC_COLS + n], rnd16[(q * 32 + j + 1) * QC_COLS + n], qm, nqm);
                } else {
                    h[k] = round_rne_pair(v[j], v[j + 1], sc, qm, nqm);
                }
            }
            pack4<PLANES>(h[0], h[1], hi[w], lo[w]);
        }
        // 128B swizzle of the store tile: 16-byte chunk c of row n sits at chunk position c ^ (n % 8)
        unsigned char* orow = base_ptr + (n >> 3) * 1024 + (n & 7) * 128;
        const int c0 = ((2 * q) ^ (n & 7)) << 4, c1 = ((2 * q + 1) ^ (n & 7)) << 4;
        *reinterpret_cast<uint4*>(orow + c0) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(orow + c1) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        if (PLANES == 2) {
            *reinterpret_cast<uint4*>(orow + QC_OUT_BYTES + c0) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            *reinterpret_cast<uint4*>(orow + QC_OUT_BYTES + c1) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            tma_store_2d(&mapM0, kt * QC_ROWS, nt * QC_COLS, base);
            if (PLANES == 2) tma_store_2d(&mapM1, kt * QC_ROWS, nt * QC_COLS, base + QC_OUT_BYTES);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        stores_pending = true;
        if (++s == QC_STAGES) { s = 0; ph ^= 1u; }
    }
    // the stores must be complete when the CTA leaves (a load still in flight after an abandoned
    // wait has had the whole wait budget, seconds, to land)
    if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Whole-axis blocks down the columns (one exponent per column of the stored matrix): pass 1 of 2. Each CTA takes
// 256 columns and a band of rows, reads rows coalesced and folds its band's maxima into one word per column.
constexpr int CMAX_ROWS = 128;
__global__ void __launch_bounds__(256)
col_amax_kernel(const float* __restrict__ x, int64_t K, int64_t R, int64_t ld, uint32_t* __restrict__ amax) {
    const int64_t col = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (col >= R) return;
    const int64_t k0 = (int64_t)blockIdx.y * CMAX_ROWS, k1 = min(K, k0 + CMAX_ROWS);
    uint32_t am = 0;
#pragma unroll 8
    for (int64_t k = k0; k < k1; ++k) am = max(am, abs_bits(__ldg(x + k * ld + col)));
    atomicMax(amax + col, am);
}
__global__ void col_exps_kernel(const uint32_t* __restrict__ amax, int64_t R, QParams p, int8_t* __restrict__ exps) {
    const int64_t col = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (col < R) exps[col] = (int8_t)block_exponent(amax[col], p.m, p.exp_mode);
}

template <int PLANES, int LB, bool SR>
int launch_col_tma(const float* x, int64_t K, int64_t rows, int64_t ld, const QParams& p, const Layout& L,
                   int8_t* mant, int8_t* exps, cudaStream_t st, const int8_t* given = nullptr) {
    CUtensorMap mX, mM0, mM1;
    int rc = make_map(&mX, x, (uint64_t)rows * 4, (uint64_t)K, (uint64_t)ld * 4, QC_COLS * 4, QC_ROWS, false);
    if (rc) return rc;
    rc = make_map(&mM0, mant, (uint64_t)L.kst, (uint64_t)rows, (uint64_t)L.kst, QC_ROWS, QC_COLS, true);
    if (rc) return rc;
    mM1 = mM0;
    if (PLANES == 2) {
        rc = make_map(&mM1, mant + L.plane_stride, (uint64_t)L.kst, (uint64_t)rows, (uint64_t)L.kst, QC_ROWS, QC_COLS, true);
        if (rc) return rc;
    }
    constexpr int smem = 1024 + PLANES * QC_OUT_BYTES + QC_STAGES * QC_IN_BYTES + (SR ? QC_ROWS * QC_COLS * 2 : 0) +
                         4 * QC_COLS * 4 + 64;
    // attribute and occupancy belong to the device: cached per device ordinal
    static int ctas_per_sm_dev[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return HBFP_ERR_CUDA;
    if (!ctas_per_sm_dev[dev]) {
        HBFP_CUDA_OK(cudaFuncSetAttribute(quant_col_tma<PLANES, LB, SR>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        int nb = 0;
        HBFP_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, quant_col_tma<PLANES, LB, SR>, QC_THREADS, smem));
        ctas_per_sm_dev[dev] = nb > 0 ? nb : 1;
    }
    const int ctas_per_sm = ctas_per_sm_dev[dev];
    int32_t* status = device_status_word();
    if (!status) return HBFP_ERR_CUDA;
    const int64_t tiles_n = (rows + QC_COLS - 1) / QC_COLS, tiles_k = L.kst / QC_ROWS;
    const int64_t total = tiles_n * tiles_k;
    const int64_t cap = (int64_t)sm_count() * ctas_per_sm;
    const int grid = (int)(total < cap ? total : cap);
    quant_col_tma<PLANES, LB, SR><<<grid, QC_THREADS, smem, st>>>(mX, mM0, mM1, p, exps, L.rs, L.nkb, K, rows, (int)tiles_n,
                                                              (int)total, status, given);
    return launch_status();
}

QParams make_params(const hbfp_format* f) {
    QParams p;
    p.m = f->mant_bits;
    p.qmax = (1 << (f->mant_bits - 1)) - 1;
    p.exp_mode = f->exp_mode;
    p.rounding = f->rounding;
    p.key0 = (uint32_t)f->seed;
    p.key1 = (uint32_t)(f->seed >> 32);
    p.stream_id = f->stream_id;
    return p;
}

inline unsigned blocks_for(int64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

template <int LPB>
int launch_row_fast(const float* x, int64_t rows, int64_t K, int64_t ld, const QParams& p, const Layout& L,
                    int8_t* mant, int8_t* exps, cudaStream_t st) {
    dim3 grid((unsigned)((L.kst + 511) / 512), (unsigned)((rows + 31) / 32));
    // the last column tile must also cover the exponent rows of blocks that start before K
    if (p.rounding == 1) {
        if (L.planes == 1) quant_row_fast<LPB, true, 1><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, L.nkb);
        else quant_row_fast<LPB, true, 2><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, L.nkb);
    } else {
        if (L.planes == 1) quant_row_fast<LPB, false, 1><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, L.nkb);
        else quant_row_fast<LPB, false, 2><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, L.nkb);
    }
    return launch_status();
}

}  // namespace

// Launch of the full-tile kernel for tiles of 32 and 64 (defined in part 2 of this file). The parameter blocks are
// passed as opaque bytes: their types live in this file's unnamed namespace, which every part compiles alike.
int launch_tile_full_small(int mode, int planes, int t, unsigned gx, unsigned gy, const float* src, int64_t ld, int64_t d0,
                           int64_t d1, const void* qparams, int16_t* wide, int8_t* grid, int64_t grid_ld,
                           const void* tileviews, cudaStream_t st);

#if HBFP_QUANT_PART == 2

int launch_tile_full_small(int mode, int planes, int t, unsigned gx, unsigned gy, const float* src, int64_t ld, int64_t d0,
                           int64_t d1, const void* qparams, int16_t* wide, int8_t* grid, int64_t grid_ld,
                           const void* tileviews, cudaStream_t st) {
    QParams p;
    TileViews tv;
    memcpy(&p, qparams, sizeof(p));
    memcpy(&tv, tileviews, sizeof(tv));
    const dim3 grid_dim(gx, gy);
#define HBFP_TILE_FULL_SMALL(MODE, PLANES, TP) tile_kernel_full<MODE, PLANES, TP><<<grid_dim, 256, 0, st>>>(src, ld, d0, d1, p, wide, grid, grid_ld, tv)
#define HBFP_TILE_FULL_MODE(MODE)                                                                     \
    do {                                                                                              \
        if (planes == 1) { if (t == 32) HBFP_TILE_FULL_SMALL(MODE, 1, 32); else HBFP_TILE_FULL_SMALL(MODE, 1, 64); } \
        else { if (t == 32) HBFP_TILE_FULL_SMALL(MODE, 2, 32); else HBFP_TILE_FULL_SMALL(MODE, 2, 64); }             \
    } while (0)
    if (t != 32 && t != 64) return HBFP_ERR_INVALID_ARG;
    if (mode == 0) HBFP_TILE_FULL_MODE(0);
    else if (mode == 1) HBFP_TILE_FULL_MODE(1);
    else if (mode == 2) HBFP_TILE_FULL_MODE(2);
    else if (mode == 3) HBFP_TILE_FULL_MODE(3);
    else return HBFP_ERR_INVALID_ARG;
#undef HBFP_TILE_FULL_MODE
#undef HBFP_TILE_FULL_SMALL
    return launch_status();
}

#else   // part 1: everything else

// ------------------------------------------------------------------------------ launchers

int launch_quantize(const float* x, int64_t d0, int64_t d1, int64_t ld, int axis, const hbfp_format* f,
                    int8_t* mant, int8_t* exps, cudaStream_t st) {
    const int64_t K = axis == 1 ? d1 : d0, rows = axis == 1 ? d0 : d1;
    Layout L;
    int rc = make_layout(rows, K, f, &L);
    if (rc) return rc;
    if (rows == 0) return HBFP_OK;
    const QParams p = make_params(f);
    if (K == 0) {
        HBFP_CUDA_OK(cudaMemsetAsync(mant, 0, (size_t)L.mant_bytes, st));
        HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
        return HBFP_OK;
    }
    const bool aligned = ((reinterpret_cast<uintptr_t>(x) & 15) == 0) && (ld % 4 == 0);
    if (rows * L.kst >= (int64_t)1 << 40) return HBFP_ERR_UNSUPPORTED;

    // row lengths that the 512-column tiles of quant_row_fast would leave ragged
    if (f->tile == 0 && axis == 1 && aligned && L.b == L.bp && L.b <= 128 && K % L.b == 0 && L.kst % 512 != 0 &&
        rows * (L.kst / 8) < (1ll << 32) - 4096) {
        // exponent padding bytes (rows .. rs of every block line) are documented as zero
        if (L.rs != rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
        switch (L.b) {
            case 32: return launch_row_flat<4>(x, rows, K, ld, p, L, mant, exps, st);
            case 64: return launch_row_flat<8>(x, rows, K, ld, p, L, mant, exps, st);
            case 128: return launch_row_flat<16>(x, rows, K, ld, p, L, mant, exps, st);
            default: break;
        }
    }
    // one block per row over the whole axis, longer than the fast kernel's tile: row maxima first (one warp per row),
    // then the fast kernel with the exponents given
    if (f->tile == 0 && axis == 1 && aligned && d1 % 8 == 0 && L.nkb == 1 && L.b == K && K > 256) {
        if (L.rs != rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
        // rows of 2048, 4096, 8192 or 16384 elements stay in a CTA's registers: one pass
        if ((K == 2048 || K == 4096 || K == 8192 || K == 16384) && L.kst == K && rows < (1ll << 31)) {
#define HBFP_QROW_WHOLE2(GV, SRV, PL) quant_row_whole<GV, SRV, PL><<<(unsigned)rows, 256, 0, st>>>(x, ld, d1, p, mant, L.kst, L.plane_stride, exps)
#define HBFP_QROW_WHOLE(GV)                                                                          \
    do {                                                                                             \
        if (p.rounding == 1) { if (L.planes == 1) HBFP_QROW_WHOLE2(GV, true, 1); else HBFP_QROW_WHOLE2(GV, true, 2); }   \
        else { if (L.planes == 1) HBFP_QROW_WHOLE2(GV, false, 1); else HBFP_QROW_WHOLE2(GV, false, 2); }                 \
    } while (0)
            if (K == 2048) HBFP_QROW_WHOLE(1); else if (K == 4096) HBFP_QROW_WHOLE(2); else if (K == 8192) HBFP_QROW_WHOLE(4); else HBFP_QROW_WHOLE(8);
#undef HBFP_QROW_WHOLE
#undef HBFP_QROW_WHOLE2
            return launch_status();
        }
        const int64_t want = (rows * 32 + 255) / 256;
        exps_axis1<<<(unsigned)(want < 148 * 16 ? want : 148 * 16), 256, 0, st>>>(x, rows, K, ld, L.b, L.nkb, p, exps, L.rs);
        if (launch_status()) return HBFP_ERR_CUDA;
        dim3 grid((unsigned)((L.kst + 511) / 512), (unsigned)((rows + 31) / 32));
#define HBFP_QROW_GIVEN(SRV, PL) quant_row_fast<16, SRV, PL><<<grid, 256, 0, st>>>(x, rows, K, ld, p, mant, L.kst, L.plane_stride, exps, L.rs, L.nkb, exps)
        if (p.rounding == 1) { if (L.planes == 1) HBFP_QROW_GIVEN(true, 1); else HBFP_QROW_GIVEN(true, 2); }
        else { if (L.planes == 1) HBFP_QROW_GIVEN(false, 1); else HBFP_QROW_GIVEN(false, 2); }
#undef HBFP_QROW_GIVEN
        return launch_status();
    }
    if (f->tile == 0 && axis == 1 && aligned && d1 % 8 == 0 && L.b == L.bp && L.b <= 256 &&
        rows <= 32ll * 65535) {
        switch (L.b) {
            case 32: return launch_row_fast<4>(x, rows, K, ld, p, L, mant, exps, st);
            case 64: return launch_row_fast<8>(x, rows, K, ld, p, L, mant, exps, st);
            case 128: return launch_row_fast<16>(x, rows, K, ld, p, L, mant, exps, st);
            case 256: return launch_row_fast<32>(x, rows, K, ld, p, L, mant, exps, st);
            default: break;
        }
    }
    // one block per column over the whole axis: column maxima first (scratch: the head of the mantissa buffer, which
    // the second pass overwrites), then the tile kernel with the exponents given
    if (f->tile == 0 && axis == 0 && aligned && L.nkb == 1 && L.b == K && K % QC_ROWS == 0 && L.kst == K && K > 128 &&
        (p.rounding == 0 || rows % 8 == 0) && (reinterpret_cast<uintptr_t>(mant) & 127) == 0 && rows < (1ll << 29) &&
        K < (1ll << 31) && (K + CMAX_ROWS - 1) / CMAX_ROWS <= 65535 && (int64_t)rows * 4 <= (int64_t)rows * L.kst &&
        ((rows + QC_COLS - 1) / QC_COLS) * (L.kst / QC_ROWS) < (1ll << 31)) {
        if (L.rs != rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
        uint32_t* amax = reinterpret_cast<uint32_t*>(mant);
        HBFP_CUDA_OK(cudaMemsetAsync(amax, 0, (size_t)rows * 4, st));
        const dim3 g1((unsigned)((rows + 255) / 256), (unsigned)((K + CMAX_ROWS - 1) / CMAX_ROWS));
        col_amax_kernel<<<g1, 256, 0, st>>>(x, K, rows, ld, amax);
        col_exps_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(amax, rows, p, exps);
        if (launch_status()) return HBFP_ERR_CUDA;
#define HBFP_QCOL_GIVEN(PL) (p.rounding ? launch_col_tma<PL, 0, true>(x, K, rows, ld, p, L, mant, exps, st, exps) \
                                        : launch_col_tma<PL, 0, false>(x, K, rows, ld, p, L, mant, exps, st, exps))
        return L.planes == 1 ? HBFP_QCOL_GIVEN(1) : HBFP_QCOL_GIVEN(2);
#undef HBFP_QCOL_GIVEN
    }
    if (f->tile == 0 && axis == 0 && aligned && L.b == L.bp && L.b <= 128 && (p.rounding == 0 || rows % 8 == 0) &&
        (reinterpret_cast<uintptr_t>(mant) & 127) == 0 && rows < (1ll << 29) && K < (1ll << 31) &&
        ((rows + QC_COLS - 1) / QC_COLS) * (L.kst / QC_ROWS) < (1ll << 31)) {
        // exponent padding bytes (lines >= rows) are documented as zero
        if (L.rs != rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
#define HBFP_QCOL_TMA(PL, LBV) (p.rounding ? launch_col_tma<PL, LBV, true>(x, K, rows, ld, p, L, mant, exps, st) \
                                           : launch_col_tma<PL, LBV, false>(x, K, rows, ld, p, L, mant, exps, st))
        const int lb = L.b == 128 ? 0 : L.b == 64 ? 1 : 2;
        if (L.planes == 1) return lb == 0 ? HBFP_QCOL_TMA(1, 0) : lb == 1 ? HBFP_QCOL_TMA(1, 1) : HBFP_QCOL_TMA(1, 2);
        return lb == 0 ? HBFP_QCOL_TMA(2, 0) : lb == 1 ? HBFP_QCOL_TMA(2, 1) : HBFP_QCOL_TMA(2, 2);
#undef HBFP_QCOL_TMA
    }
    if (f->tile == 0 && axis == 0 && L.b <= 128) {
        const int vec_ok = aligned && (rows % 4 == 0);
        const int G = (int)(128 / L.bp);                   // blocks per panel
        const int64_t gy = (L.nkb + G - 1) / G;
        if (gy <= 65535) {
            const size_t krows = (size_t)G * L.b;
            size_t smem = krows * COLT * sizeof(float) + (size_t)G * 4 * COLT * sizeof(uint32_t) +
                          (p.rounding ? krows * (COLT / 8) * sizeof(uint4) : 0);
            dim3 grid((unsigned)((rows + COLT - 1) / COLT), (unsigned)gy);
            // exponent padding bytes (lines >= rows) are documented as zero
            if (L.rs != rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
#define HBFP_QCOL(PL, RQ) quant_col_fast<PL, RQ><<<grid, 128, smem, st>>>(x, K, rows, ld, (int)L.b, p, mant, L.kst, L.plane_stride, exps, L.rs, L.nkb, vec_ok)
            if (L.planes == 1) { if (L.bp == 32) HBFP_QCOL(1, 8); else if (L.bp == 64) HBFP_QCOL(1, 16); else HBFP_QCOL(1, 32); }
            else { if (L.bp == 32) HBFP_QCOL(2, 8); else if (L.bp == 64) HBFP_QCOL(2, 16); else HBFP_QCOL(2, 32); }
#undef HBFP_QCOL
            return launch_status();
        }
    }
    if (f->tile > 0 && f->tile <= 128) {
        // single view of a tiled weight: the fused tile kernel with the other view switched off
        return axis == 0 ? launch_quantize_tiles(x, d0, d1, ld, f, mant, exps, nullptr, nullptr, nullptr, st)
                         : launch_quantize_tiles(x, d0, d1, ld, f, nullptr, nullptr, mant, exps, nullptr, st);
    }

    // generic two-pass path
    HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
    if (f->tile == 0) {
        if (axis == 1) {
            int64_t items = rows * L.nkb;
            int64_t want = (items + 7) / 8;
            unsigned blocks = (unsigned)(want < 148 * 32 ? want : 148 * 32);
            exps_axis1<<<blocks, 256, 0, st>>>(x, rows, K, ld, L.b, L.nkb, p, exps, L.rs);
        } else {
            exps_axis0<<<blocks_for(rows * L.nkb, 256), 256, 0, st>>>(x, rows, K, ld, L.b, L.nkb, p, exps, L.rs);
        }
    } else {
        const int64_t t = f->tile, nu = (d0 + t - 1) / t, nv = (d1 + t - 1) / t;
        exps_tiles<<<blocks_for(nu * nv * 32, 256), 256, 0, st>>>(x, d0, d1, ld, t, p, axis, exps, L.rs, nu, nv);
    }
    if (launch_status()) return HBFP_ERR_CUDA;
    if (L.planes == 1)
        mant_generic<1><<<blocks_for(rows * (L.kst / 4), 256), 256, 0, st>>>(x, d1, rows, K, ld, axis, L.b, L.bp, L.nkb, p, exps, L.rs, mant, L.kst, L.plane_stride);
    else
        mant_generic<2><<<blocks_for(rows * (L.kst / 4), 256), 256, 0, st>>>(x, d1, rows, K, ld, axis, L.b, L.bp, L.nkb, p, exps, L.rs, mant, L.kst, L.plane_stride);
    return launch_status();
}

namespace {

template <int MODE>
int launch_tiles(const float* src, int64_t ld, int64_t d0, int64_t d1, const hbfp_format* f, int16_t* wide,
                 int8_t* grid, int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1, cudaStream_t st) {
    if (f->tile <= 0 || f->tile != f->block) return HBFP_ERR_INVALID_ARG;
    if (f->tile > 128) return HBFP_ERR_UNSUPPORTED;
    Layout L0, L1;
    int rc = make_layout(d1, d0, f, &L0);     // view c0: rows = d1, k = d0
    if (rc) return rc;
    rc = make_layout(d0, d1, f, &L1);         // view c1: rows = d0, k = d1
    if (rc) return rc;
    if (d0 == 0 || d1 == 0) return HBFP_OK;
    const QParams p = make_params(f);
    const int t = f->tile, tp = (int)L0.bp;
    const int64_t nu = L0.nkb, nv = L1.nkb;   // tiles along d0, along d1
    if (nu > 65535) return HBFP_ERR_UNSUPPORTED;
    if (exps_c0 && L0.rs != d1) HBFP_CUDA_OK(cudaMemsetAsync(exps_c0, 0, (size_t)L0.exp_bytes, st));
    if (exps_c1 && L1.rs != d0) HBFP_CUDA_OK(cudaMemsetAsync(exps_c1, 0, (size_t)L1.exp_bytes, st));
    const TileViews tv{mant_c0, L0.kst, L0.plane_stride, exps_c0, L0.rs, L0.nkb, mant_c1, L1.kst, L1.plane_stride, exps_c1, L1.rs, L1.nkb};
    const bool fast = (t % 8) == 0 && (d1 % 8) == 0 &&
                      (MODE == 2 || ((ld % 4) == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0)) &&
                      (MODE == 3 || (reinterpret_cast<uintptr_t>(wide) & 15) == 0);
    const size_t smem = (size_t)t * (t + 4) * sizeof(float) + (size_t)tp * (tp + 2) * sizeof(int16_t);
    const dim3 grid_dim((unsigned)nv, (unsigned)nu);
    // full tiles of 32 / 64 / 128, both views or none, narrow bits cut by 32-bit shifts (see tile_kernel_full)
    const int sh_full = MODE == 3 ? 0 : 16 - p.m;
    const bool full = fast && t == tp && (d0 % t) == 0 && (d1 % t) == 0 && ((mant_c0 != nullptr) == (mant_c1 != nullptr)) &&
                      (!mant_c0 || (exps_c0 && exps_c1)) && sh_full + (L0.planes == 2 ? 4 : 0) <= 8;
    if (full) {
#define HBFP_TILE_FULL(PLANES, TP) tile_kernel_full<MODE, PLANES, TP><<<grid_dim, 256, 0, st>>>(src, ld, d0, d1, p, wide, grid, nv, tv)
        if (t != 128)
            return launch_tile_full_small(MODE, (int)L0.planes, t, grid_dim.x, grid_dim.y, src, ld, d0, d1, &p, wide, grid, nv, &tv, st);
        if (L0.planes == 1) HBFP_TILE_FULL(1, 128); else HBFP_TILE_FULL(2, 128);
#undef HBFP_TILE_FULL
        return launch_status();
    }
#define HBFP_TILE_LAUNCH(PLANES, FAST)                                                                                       \
    do {                                                                                                                     \
        HBFP_CUDA_OK(cudaFuncSetAttribute(tile_kernel<MODE, PLANES, FAST>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        tile_kernel<MODE, PLANES, FAST><<<grid_dim, 256, smem, st>>>(src, ld, d0, d1, t, tp, p, wide, grid, nv, tv);         \
    } while (0)
    if (L0.planes == 1) {
        if (fast) HBFP_TILE_LAUNCH(1, true); else HBFP_TILE_LAUNCH(1, false);
    } else {
        if (fast) HBFP_TILE_LAUNCH(2, true); else HBFP_TILE_LAUNCH(2, false);
    }
#undef HBFP_TILE_LAUNCH
    return launch_status();
}

}  // namespace

int launch_quantize_tiles(const float* w, int64_t d0, int64_t d1, int64_t ld, const hbfp_format* f,
                          int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1,
                          int8_t* tile_exps, cudaStream_t st) {
    return launch_tiles<3>(w, ld, d0, d1, f, nullptr, tile_exps, mant_c0, exps_c0, mant_c1, exps_c1, st);
}

// Convolution weights w [taps * c_in][c_out] with one exponent per (t input maps) x (t output maps) tile over
// all taps: view c0 (rows = c_out, k = taps * c_in) and / or view c1 (rows = taps * c_in, k = c_out).
int launch_quantize_conv_weights(const float* w, int64_t taps, int64_t c_in, int64_t c_out, int64_t ld,
                                 const hbfp_format* f, int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1,
                                 int8_t* tile_exps, cudaStream_t st) {
    const int64_t t = f->tile;
    if (t <= 0 || f->block != t || taps <= 0 || c_in <= 0 || c_out <= 0) return HBFP_ERR_INVALID_ARG;
    if (c_in % t != 0) return HBFP_ERR_UNSUPPORTED;               // a K-block must not straddle two taps
    const int64_t d0 = taps * c_in, d1 = c_out, nu = c_in / t, nv = (c_out + t - 1) / t;
    const QParams p = make_params(f);
    if (nu * nv >= (1ll << 31)) return HBFP_ERR_UNSUPPORTED;
    Layout L[2];
    for (int axis = 0; axis < 2; ++axis) {
        int8_t* exps = axis == 0 ? exps_c0 : exps_c1;
        if (!(axis == 0 ? mant_c0 : mant_c1)) continue;
        int rc = make_layout(axis == 0 ? d1 : d0, axis == 0 ? d0 : d1, f, &L[axis]);
        if (rc) return rc;
        if (L[axis].rs != L[axis].rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L[axis].exp_bytes, st));   // padding lines are zero
    }
    if (!mant_c0 && !mant_c1 && !tile_exps) return HBFP_OK;
    // few tiles: split each tile's rows over several CTAs, maxima merged in the head of a mantissa buffer (the
    // mantissa pass that follows overwrites it)
    int8_t* const scratch_buf = mant_c1 ? mant_c1 : mant_c0;
    const int64_t scratch_room = !scratch_buf ? 0 : (mant_c1 ? L[1].mant_bytes : L[0].mant_bytes);
    int64_t splits = (2 * 148 + nu * nv - 1) / (nu * nv);
    splits = std::min<int64_t>(splits, (taps * t + CONVW_THREADS / 32 - 1) / (CONVW_THREADS / 32));
    for (int pass = 0; pass < 2; ++pass) {
        uint32_t* amax = nullptr;
        if (splits > 1 && nu * nv * 4 <= scratch_room) amax = reinterpret_cast<uint32_t*>(scratch_buf);
        if (pass == 1 && !amax) break;
        if (pass == 0 && amax) HBFP_CUDA_OK(cudaMemsetAsync(amax, 0, (size_t)(nu * nv * 4), st));
        const dim3 grid((unsigned)(nu * nv), pass == 0 && amax ? (unsigned)splits : 1u);
        exps_conv_tiles<<<grid, CONVW_THREADS, 0, st>>>(w, taps, c_in, c_out, ld, t, p, mant_c0 ? exps_c0 : nullptr,
                                                        mant_c0 ? L[0].rs : 0, mant_c1 ? exps_c1 : nullptr,
                                                        mant_c1 ? L[1].rs : 0, nu, nv, tile_exps, amax, pass == 1);
        if (launch_status()) return HBFP_ERR_CUDA;
    }
    for (int axis = 0; axis < 2; ++axis) {
        int8_t* mant = axis == 0 ? mant_c0 : mant_c1;
        const int8_t* exps = axis == 0 ? exps_c0 : exps_c1;
        if (!mant) continue;
        const Layout& A = L[axis];
        if (A.planes == 1)
            mant_generic<1><<<blocks_for(A.rows * (A.kst / 4), 256), 256, 0, st>>>(w, d1, A.rows, A.k, ld, axis, A.b, A.bp, A.nkb, p, exps, A.rs, mant, A.kst, A.plane_stride);
        else
            mant_generic<2><<<blocks_for(A.rows * (A.kst / 4), 256), 256, 0, st>>>(w, d1, A.rows, A.k, ld, axis, A.b, A.bp, A.nkb, p, exps, A.rs, mant, A.kst, A.plane_stride);
        if (launch_status()) return HBFP_ERR_CUDA;
    }
    return HBFP_OK;
}

int launch_wide(int mode, const float* src, int64_t ld, int64_t d0, int64_t d1, const hbfp_format* f,
                int16_t* wide, int8_t* wide_exps, int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1,
                cudaStream_t st) {
    if (mode == 0) return launch_tiles<0>(src, ld, d0, d1, f, wide, wide_exps, mant_c0, exps_c0, mant_c1, exps_c1, st);
    if (mode == 1) return launch_tiles<1>(src, ld, d0, d1, f, wide, wide_exps, mant_c0, exps_c0, mant_c1, exps_c1, st);
    return launch_tiles<2>(nullptr, d1, d0, d1, f, wide, wide_exps, mant_c0, exps_c0, mant_c1, exps_c1, st);
}

int launch_im2col_packed(const int8_t* xm, const int8_t* xe, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw,
                         int pad, const hbfp_format* f, int8_t* om, int8_t* oe, cudaStream_t st) {
    if (f->tile != 0 || f->block != c) return HBFP_ERR_INVALID_ARG;      // one block per pixel
    if (c > 128) return HBFP_ERR_UNSUPPORTED;
    const int64_t ho = h + 2 * pad - kh + 1, wo = w + 2 * pad - kw + 1;
    if (ho <= 0 || wo <= 0) return HBFP_ERR_INVALID_ARG;
    Layout Lx, Lo;
    int rc = make_layout(n * h * w, c, f, &Lx);
    if (rc) return rc;
    rc = make_layout(n * ho * wo, (int64_t)kh * kw * c, f, &Lo);
    if (rc) return rc;
    if (h > (1 << 20) || w > (1 << 20) || Lo.kst > (1ll << 30)) return HBFP_ERR_UNSUPPORTED;
    if (n == 0) return HBFP_OK;
    HBFP_CUDA_OK(cudaMemsetAsync(oe, 0, (size_t)Lo.exp_bytes, st));
    const int lg_bp = Lo.bp == 32 ? 5 : Lo.bp == 64 ? 6 : 7;
    if (kh * kw > IM2COL_MAX_TAPS || kh > 100 || kw > 100 || pad > 100) return HBFP_ERR_UNSUPPORTED;
    if (Lo.rows >= (1ll << 31) || Lx.rows >= (1ll << 31)) return HBFP_ERR_UNSUPPORTED;
    im2col_gather<<<blocks_for(Lo.rows, IM2COL_ROWS), 256, 0, st>>>(xm, xe, (int)Lx.kst, Lx.plane_stride, (int)h, (int)w, (int)ho, (int)wo,
                                                                   kh, kw, pad, lg_bp, (int)Lo.planes, (uint32_t)Lo.rows, (int)Lo.kst,
                                                                   Lo.plane_stride, Lo.rs, om, oe);
    return launch_status();
}

int launch_im2col_cols(const float* x, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw, int pad,
                       const hbfp_format* f, int8_t* mant, int8_t* exps, cudaStream_t st) {
    if (f->tile != 0 || f->block <= 0) return HBFP_ERR_INVALID_ARG;
    const int64_t b = f->block;
    // Under stochastic rounding every entry takes the draw of the activation it is a copy of (its index in
    // x [n][h][w][c]): the matrix this operand is the conversion of never exists.
    // same-size output, blocks of whole image rows that do not straddle images
    if (2 * pad != kh - 1 || 2 * pad != kw - 1) return HBFP_ERR_UNSUPPORTED;
    if (!(b == 16 || b == 32 || b == 64 || b == 128) || b % w != 0 || w < 4 || (w & (w - 1)) != 0 || (h * w) % b != 0 ||
        c % 4 != 0 || (reinterpret_cast<uintptr_t>(x) & 15))
        return HBFP_ERR_UNSUPPORTED;
    Layout L;
    int rc = make_layout((int64_t)kh * kw * c, n * h * w, f, &L);
    if (rc) return rc;
    if (n == 0) return HBFP_OK;
    if (h > 32768 || c > 4096 || L.nkb >= (1ll << 31)) return HBFP_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(b / w + kh - 1) * w * c * sizeof(float);
    if (smem > 200 * 1024) return HBFP_ERR_UNSUPPORTED;
    const QParams p = make_params(f);
    if (L.rs != L.rows) HBFP_CUDA_OK(cudaMemsetAsync(exps, 0, (size_t)L.exp_bytes, st));
    if (L.kst != L.nkb * L.bp) HBFP_CUDA_OK(cudaMemsetAsync(mant, 0, (size_t)L.mant_bytes, st));     // row tails
    int lg_w = 0;
    while ((1 << lg_w) < w) ++lg_w;
#define HBFP_COLS_LAUNCH2(PL, NPX, SRV)                                                                                       \
    do {                                                                                                                       \
        HBFP_CUDA_OK(cudaFuncSetAttribute(im2col_cols<PL, NPX, SRV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));   \
        im2col_cols<PL, NPX, SRV><<<(unsigned)L.nkb, 256, smem, st>>>(x, (int)h, (int)w, lg_w, (int)c, kh, kw, pad, p, L.kst,     \
                                                                     L.plane_stride, L.rs, mant, exps);                        \
    } while (0)
#define HBFP_COLS_LAUNCH(PL, NPX)                                                 \
    do {                                                                          \
        if (p.rounding) HBFP_COLS_LAUNCH2(PL, NPX, true);                         \
        else HBFP_COLS_LAUNCH2(PL, NPX, false);                                   \
    } while (0)
    if (L.planes == 1) {
        if (b == 16) HBFP_COLS_LAUNCH(1, 4); else if (b == 32) HBFP_COLS_LAUNCH(1, 8); else if (b == 64) HBFP_COLS_LAUNCH(1, 16); else HBFP_COLS_LAUNCH(1, 32);
    } else {
        if (b == 16) HBFP_COLS_LAUNCH(2, 4); else if (b == 32) HBFP_COLS_LAUNCH(2, 8); else if (b == 64) HBFP_COLS_LAUNCH(2, 16); else HBFP_COLS_LAUNCH(2, 32);
    }
#undef HBFP_COLS_LAUNCH2
#undef HBFP_COLS_LAUNCH
    return launch_status();
}

int launch_conv_dgrad_filters(const Packed& c1, int taps, int64_t c_in, int64_t c_out, int t, int8_t* mant_out,
                              int8_t* exps_out, const Layout& Lo, cudaStream_t st) {
    if (c_in == 0) return HBFP_OK;
    if (Lo.rs != c_in) HBFP_CUDA_OK(cudaMemsetAsync(exps_out, 0, (size_t)Lo.exp_bytes, st));   // padding lines are zero
    const int64_t warps = c_in * taps;
    conv_dgrad_filters_kernel<<<blocks_for(warps * 32, 256), 256, 0, st>>>(c1.mant, c1.exps, c1.L.kst, c1.L.plane_stride, c1.L.rs,
                                                                          taps, c_in, c_out, t, (int)c1.L.planes, mant_out, exps_out,
                                                                          Lo.kst, Lo.plane_stride, Lo.rs);
    return launch_status();
}

int launch_unpack(const Packed& p, int16_t* q, int8_t* s, cudaStream_t st) {
    const Layout& L = p.L;
    int64_t n = L.rows * (L.k > L.nkb ? L.k : L.nkb);
    if (n == 0) return HBFP_OK;
    unpack_kernel<<<blocks_for(n, 256), 256, 0, st>>>(p.mant, p.exps, L.rows, L.k, L.b, L.bp, L.nkb, L.kst,
                                                     L.plane_stride, (int)L.planes, L.rs, q, s);
    return launch_status();
}

// Value of wide weight storage, Eq. 1: out[i][j] = q16[i][j] * 2^s16[i/t][j/t] (exact in binary32: 16-bit mantissas).
__global__ void wide_dequant_kernel(const int16_t* __restrict__ wide, const int8_t* __restrict__ exps, int64_t d0,
                                    int64_t d1, int t, int64_t tiles1, float* __restrict__ out, int64_t ldo) {
    const int64_t n = d0 * d1;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / d1, c = i - r * d1;
        const int e = exps[(r / t) * tiles1 + c / t];
        out[r * ldo + c] = ldexpf((float)wide[i], e);
    }
}

int launch_wide_dequantize(const int16_t* wide, const int8_t* exps, int64_t d0, int64_t d1, int tile, float* out,
                           int64_t ldo, cudaStream_t st) {
    if (d0 * d1 == 0) return HBFP_OK;
    const int64_t tiles1 = (d1 + tile - 1) / tile;
    wide_dequant_kernel<<<blocks_for(d0 * d1, 256), 256, 0, st>>>(wide, exps, d0, d1, tile, tiles1, out, ldo);
    return launch_status();
}

int launch_dequantize(const Packed& p, float* out, int64_t ld, cudaStream_t st) {
    const Layout& L = p.L;
    if (L.rows * L.k == 0) return HBFP_OK;
    dequant_kernel<<<blocks_for(L.rows * L.k, 256), 256, 0, st>>>(p.mant, p.exps, L.rows, L.k, L.b, L.bp, L.kst,
                                                                 L.plane_stride, (int)L.planes, L.rs, out, ld);
    return launch_status();
}

#endif   // HBFP_QUANT_PART

}  // namespace hbfp
