// Plain CUDA-core BFP GEMM: the reference GPU path. One thread per output element, dp4a over
// the packed int8 mantissas, one exact int32 sum per K-block (Eq. 2), FP32 accumulation of the
// scaled block sums in ascending block order. Handles every format the packed layout can
// express and can dump the per-block integer sums. Slow by design; the tensor-core kernel is
// the product path.
#include "common.cuh"

namespace hbfp {
namespace {

template <int PLANES_A, int PLANES_B>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(int64_t M, int64_t N, int64_t nkb, int64_t bp,
                 const int8_t* __restrict__ mA, int64_t kstA, int64_t psA, const int8_t* __restrict__ eA, int64_t rsA,
                 const int8_t* __restrict__ mB, int64_t kstB, int64_t psB, const int8_t* __restrict__ eB, int64_t rsB,
                 float* __restrict__ C, int64_t ldc, int32_t* __restrict__ P) {
    const int64_t j = (int64_t)blockIdx.x * 16 + (threadIdx.x & 15);
    const int64_t i = (int64_t)blockIdx.y * 16 + (threadIdx.x >> 4);
    if (i >= M || j >= N) return;
    const int* a0 = reinterpret_cast<const int*>(mA + i * kstA);
    const int* b0 = reinterpret_cast<const int*>(mB + j * kstB);
    const int* a1 = reinterpret_cast<const int*>(mA + psA + i * kstA);   // low planes (12-bit)
    const int* b1 = reinterpret_cast<const int*>(mB + psB + j * kstB);
    const int words = (int)(bp / 4);
    float acc = 0.f;
    for (int64_t kb = 0; kb < nkb; ++kb) {
        int hh = 0, mid = 0, ll = 0;
        const int64_t w0 = kb * words;
        for (int w = 0; w < words; ++w) {
            const int ah = __ldg(a0 + w0 + w), bh = __ldg(b0 + w0 + w);
            hh = __dp4a(ah, bh, hh);
            if (PLANES_A == 2) {
                const int al = __ldg(a1 + w0 + w);
                mid = __dp4a(al, bh, mid);
                if (PLANES_B == 2) ll = __dp4a(al, __ldg(b1 + w0 + w), ll);
            }
            if (PLANES_B == 2) mid = __dp4a(ah, __ldg(b1 + w0 + w), mid);
        }
        // q = 16*hi + lo on a two-plane operand, q = hi on a one-plane operand
        int p;
        if (PLANES_A == 2 && PLANES_B == 2) p = (int)(256u * (unsigned)hh + 16u * (unsigned)mid + (unsigned)ll);
        else if (PLANES_A == 2 || PLANES_B == 2) p = (int)(16u * (unsigned)hh + (unsigned)mid);
        else p = hh;
        if (P) P[(i * N + j) * nkb + kb] = p;
        const int e = (int)eA[kb * rsA + i] + (int)eB[kb * rsB + j];
        acc = __fadd_rn(acc, ldexpf((float)p, e));
    }
    if (C) C[i * ldc + j] = acc;
}

}  // namespace

int launch_gemm_simt(int64_t M, int64_t N, int64_t K, const Packed& a, const Packed& b, float* C,
                     int64_t ldc, int32_t* P, cudaStream_t st) {
    (void)K;
    if (M == 0 || N == 0) return HBFP_OK;
    if (a.L.bp != b.L.bp || a.L.nkb != b.L.nkb || a.L.b != b.L.b) return HBFP_ERR_INVALID_ARG;
    dim3 grid((unsigned)((N + 15) / 16), (unsigned)((M + 15) / 16));
    if (grid.y > 65535) return HBFP_ERR_UNSUPPORTED;
#define HBFP_SIMT(PA, PB)                                                                            \
    gemm_simt_kernel<PA, PB><<<grid, 256, 0, st>>>(M, N, a.L.nkb, a.L.bp, a.mant, a.L.kst,           \
                                                   a.L.plane_stride, a.exps, a.L.rs, b.mant, b.L.kst, \
                                                   b.L.plane_stride, b.exps, b.L.rs, C, ldc, P)
    if (a.L.planes == 1 && b.L.planes == 1) HBFP_SIMT(1, 1);
    else if (a.L.planes == 2 && b.L.planes == 1) HBFP_SIMT(2, 1);
    else if (a.L.planes == 1 && b.L.planes == 2) HBFP_SIMT(1, 2);
    else HBFP_SIMT(2, 2);
#undef HBFP_SIMT
    return launch_status();
}

}  // namespace hbfp
