// BFP GEMM for the smallest problems (a 256 or 512 cube: a few tens to hundreds of MOPs with a contraction of at
// most 512 bytes). The tensor-core kernels need several microseconds to set up their pipeline and, for outputs
// of a few tiles, a second launch to add split-K parts; here a plain tiled kernel finishes first (256 cube: 3.9
// against 6.0 us, 512 cube: 5.3 against 8.7 us), in one launch and without splitting K. It does not scale: on
// this part both dp4a and the warp-level int8 MMA it uses cost about 230 ns per 32-byte step of a 32 x 32 tile
// (the MLP's layers, 33-43 steps, take 10-12 us here against 9.6 us on the tensor-core path), so the dispatch
// keeps it to short contractions and grids of at most two CTAs per SM.
//
// One CTA per 32 x 32 tile of C, 256 threads, a 16 x 8 piece per warp. The packed mantissas of the tile's 32 rows
// of A and 32 rows of B come in 512-byte slices of K by asynchronous 16-byte copies into two shared-memory buffers
// (a slice is in flight while the previous one is multiplied); the exponents of all K-blocks of those rows are
// staged once. Per K-block: the exact int32 sum by mma.sync.m16n8k32 (Eq. 2), converted to binary32 and
// accumulated with one FMA by 2^(sA + sB), blocks in ascending order: bit for bit the sequential definition.
#include "common.cuh"

namespace hbfp {
namespace {

constexpr int SM_TILE = 32;                 // rows of A and rows of B (columns of C) per CTA
constexpr int SM_SLICE = 512;               // bytes of K per slice
constexpr int SM_PITCH = SM_SLICE + 16;     // row pitch in shared memory: rows 4 banks apart
constexpr int SM_BUF = 2 * SM_TILE * SM_PITCH;   // one slice of both operands
constexpr int SM_MAX_NKB = 1024;            // exponents staged per row
constexpr int SM_AUTO_BYTES = 512;          // automatic choice: contractions of at most one slice ...
constexpr int64_t SM_AUTO_CTAS = 2 * 148;   // ... and at most two CTAs per SM

// 2^e for any integer e the sum of two stored exponents can take; outside the normal range the slow exact route
__device__ __forceinline__ float scale_of(int e) {
    return (e >= -126 && e <= 127) ? __int_as_float((e + 127) << 23) : ldexpf(1.0f, e);
}
__device__ __forceinline__ void copy16_async(void* dst_shared, const void* src_global) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_shared)), "l"(src_global) : "memory");
}

__global__ void __launch_bounds__(256)
gemm_small_kernel(int64_t M, int64_t N, int nkb, int bp, const int8_t* __restrict__ mA, int64_t kstA,
                  const int8_t* __restrict__ eA, int64_t rsA, const int8_t* __restrict__ mB, int64_t kstB,
                  const int8_t* __restrict__ eB, int64_t rsB, float* __restrict__ C, int64_t ldc) {
    extern __shared__ __align__(16) unsigned char smem[];
    int8_t* xA = reinterpret_cast<int8_t*>(smem + 2 * SM_BUF);  // [nkb][32]
    int8_t* xB = xA + (size_t)nkb * SM_TILE;                    // [nkb][32]

    const int tid = threadIdx.x;
    const int64_t i0 = (int64_t)blockIdx.y * SM_TILE, j0 = (int64_t)blockIdx.x * SM_TILE;
    const int total_bytes = nkb * bp;                           // a multiple of 32, at most the row pitch of either operand
    const int slices = (total_bytes + SM_SLICE - 1) / SM_SLICE;
    // loader role: per slice, 16-byte pieces t, t + 256, ... of the 32 x 32 pieces of each operand (row = piece / 32)
    const int8_t* rowA[4];
    const int8_t* rowB[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int r = (tid + 256 * u) >> 5;
        rowA[u] = mA + min(i0 + r, M - 1) * kstA;               // rows beyond the matrix: the last valid row, never stored
        rowB[u] = mB + min(j0 + r, N - 1) * kstB;
    }
    auto issue = [&](int s) {
        unsigned char* buf = smem + (s & 1) * SM_BUF;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int r = (tid + 256 * u) >> 5, piece = (tid + 256 * u) & 31;
            const int off = s * SM_SLICE + 16 * piece;
            if (off < total_bytes) {
                copy16_async(buf + r * SM_PITCH + 16 * piece, rowA[u] + off);
                copy16_async(buf + SM_TILE * SM_PITCH + r * SM_PITCH + 16 * piece, rowB[u] + off);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    issue(0);
    // exponents of every K-block of the tile's rows
    for (int t = tid; t < nkb * SM_TILE; t += 256) {
        const int kb = t >> 5, r = t & 31;
        xA[t] = eA[(int64_t)kb * rsA + min(i0 + r, M - 1)];
        xB[t] = eB[(int64_t)kb * rsB + min(j0 + r, N - 1)];
    }

    // compute role: warp w owns the 16 x 8 piece of C at rows 16 (w & 1), columns 8 (w >> 1): one
    // mma.sync.m16n8k32 (s8 x s8 -> s32, exact) per 32-byte step. Fragment layout: this lane holds rows g and g + 8
    // of A (g = lane / 4) at k bytes 4 (lane % 4) and + 16, row g of B at the same bytes, and of C rows g, g + 8 at
    // columns 2 (lane % 4), + 1.
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, kq = 4 * (lane & 3);
    const int ra = 16 * (warp & 1) + g, rb = 8 * (warp >> 1) + g;
    const int cr0 = 16 * (warp & 1) + g, cc0 = 8 * (warp >> 1) + 2 * (lane & 3);
    const int steps_per_block = bp >> 5;                        // 32-byte steps per K-block
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int p0 = 0, p1 = 0, p2 = 0, p3 = 0;
    int step_in_block = 0, kb = 0;
    for (int s = 0; s < slices; ++s) {
        if (s + 1 < slices) {
            issue(s + 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();                                        // slice s (and, first, the exponents) visible to all
        const unsigned char* sA = smem + (s & 1) * SM_BUF + ra * SM_PITCH + kq;
        const unsigned char* sB = smem + (s & 1) * SM_BUF + SM_TILE * SM_PITCH + rb * SM_PITCH + kq;
        const int steps = min(SM_SLICE / 32, (total_bytes - s * SM_SLICE) >> 5);
        for (int q = 0; q < steps; ++q) {
            const uint32_t a0 = *reinterpret_cast<const uint32_t*>(sA + 32 * q);
            const uint32_t a1 = *reinterpret_cast<const uint32_t*>(sA + 8 * SM_PITCH + 32 * q);
            const uint32_t a2 = *reinterpret_cast<const uint32_t*>(sA + 32 * q + 16);
            const uint32_t a3 = *reinterpret_cast<const uint32_t*>(sA + 8 * SM_PITCH + 32 * q + 16);
            const uint32_t b0 = *reinterpret_cast<const uint32_t*>(sB + 32 * q);
            const uint32_t b1 = *reinterpret_cast<const uint32_t*>(sB + 32 * q + 16);
            asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                         : "+r"(p0), "+r"(p1), "+r"(p2), "+r"(p3) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
            if (++step_in_block == steps_per_block) {
                const int ea0 = xA[kb * SM_TILE + cr0], ea1 = xA[kb * SM_TILE + cr0 + 8];
                const int eb0 = xB[kb * SM_TILE + cc0], eb1 = xB[kb * SM_TILE + cc0 + 1];
                acc[0] = fmaf((float)p0, scale_of(ea0 + eb0), acc[0]);
                acc[1] = fmaf((float)p1, scale_of(ea0 + eb1), acc[1]);
                acc[2] = fmaf((float)p2, scale_of(ea1 + eb0), acc[2]);
                acc[3] = fmaf((float)p3, scale_of(ea1 + eb1), acc[3]);
                p0 = p1 = p2 = p3 = 0;
                step_in_block = 0;
                ++kb;
            }
        }
        __syncthreads();                                        // the buffer is free for the slice after the next
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            const int64_t i = i0 + cr0 + 8 * a, j = j0 + cc0 + b;
            if (i < M && j < N) C[i * ldc + j] = acc[2 * a + b];
        }
}

}  // namespace

// One-plane operands, at most SM_MAX_NKB K-blocks; unless any_size, a problem small enough that the tensor-core
// kernels' set-up time would dominate.
bool small_gemm_eligible(int64_t M, int64_t N, const Packed& a, const Packed& b, bool any_size) {
    if (a.L.planes != 1 || b.L.planes != 1) return false;
    if (a.L.bp != b.L.bp || a.L.nkb != b.L.nkb || a.L.b != b.L.b) return false;
    if (a.L.bp % 32 != 0 || a.L.nkb > SM_MAX_NKB || a.L.nkb * a.L.bp > (1 << 20)) return false;
    if (M <= 0 || N <= 0 || (M + SM_TILE - 1) / SM_TILE > 65535) return false;
    // the per-block sum must convert to binary32 exactly, as on the tensor-core path
    const int64_t qa = (1ll << (a.mant_bits - 1)) - 1, qb = (1ll << (b.mant_bits - 1)) - 1;
    if (qa * qb * a.L.b >= (1ll << 24)) return false;
    const int64_t ctas = ((M + SM_TILE - 1) / SM_TILE) * ((N + SM_TILE - 1) / SM_TILE);
    return any_size || (a.L.nkb * a.L.bp <= SM_AUTO_BYTES && ctas <= SM_AUTO_CTAS);
}

int launch_gemm_small(int64_t M, int64_t N, const Packed& a, const Packed& b, float* C, int64_t ldc, cudaStream_t st) {
    const int nkb = (int)a.L.nkb;
    const size_t smem = 2 * SM_BUF + 2 * (size_t)nkb * SM_TILE;          // at most 132 KB
    // the attribute belongs to the device: set once per device (same value from any thread)
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HBFP_ERR_CUDA;
    if (!attr_set[dev]) {
        HBFP_CUDA_OK(cudaFuncSetAttribute(gemm_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * SM_BUF + 2 * SM_MAX_NKB * SM_TILE));
        attr_set[dev] = true;
    }
    const dim3 grid((unsigned)((N + SM_TILE - 1) / SM_TILE), (unsigned)((M + SM_TILE - 1) / SM_TILE));
    gemm_small_kernel<<<grid, 256, smem, st>>>(M, N, nkb, (int)a.L.bp, a.mant, a.L.kst, a.exps, a.L.rs, b.mant, b.L.kst,
                                               b.exps, b.L.rs, C, ldc);
    return launch_status();
}

}  // namespace hbfp
