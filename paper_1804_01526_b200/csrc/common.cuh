// Internal declarations shared by the CUDA translation units of the HBFP library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "hbfp.h"

namespace hbfp {

// ------------------------------------------------------------------------------ layout

struct Layout {
    int64_t rows, k, b, bp, nkb, kst, planes, plane_stride, rs, mant_bytes, exp_bytes;
};

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// Validates a format and computes the packed layout (see "Packed operand layout" in hbfp.h).
inline int make_layout(int64_t rows, int64_t k, const hbfp_format* f, Layout* L) {
    if (!f || !L || rows < 0 || k < 0) return HBFP_ERR_INVALID_ARG;
    if (f->struct_size != sizeof(hbfp_format)) return HBFP_ERR_INVALID_ARG;
    if (f->mant_bits < 3 || f->mant_bits > 12) return HBFP_ERR_UNSUPPORTED;
    if (f->block < 0 || f->tile < 0) return HBFP_ERR_INVALID_ARG;
    if (f->tile > 0 && f->tile != f->block) return HBFP_ERR_INVALID_ARG;
    if (f->rounding != 0 && f->rounding != 1) return HBFP_ERR_INVALID_ARG;
    if (f->exp_mode != 0 && f->exp_mode != 1) return HBFP_ERR_INVALID_ARG;
    int64_t b = f->block == 0 ? (k > 0 ? k : 1) : f->block;
    // The per-block integer sum must fit int32 (wide accumulators never overflow, Sec. 5.3).
    int64_t qmax = ((int64_t)1 << (f->mant_bits - 1)) - 1;
    if (qmax * qmax * b > 0x7fffffffll) return HBFP_ERR_UNSUPPORTED;
    L->rows = rows;
    L->k = k;
    L->b = b;
    L->bp = b <= 32 ? 32 : b <= 64 ? 64 : b <= 128 ? 128 : round_up(b, 128);
    L->nkb = (k + b - 1) / b;
    L->kst = round_up(L->nkb * L->bp, 128);
    if (L->kst == 0) L->kst = 128;
    L->planes = f->mant_bits <= 8 ? 1 : 2;
    L->plane_stride = round_up(rows * L->kst, 1024);
    if (L->plane_stride == 0) L->plane_stride = 1024;
    L->rs = round_up(rows > 0 ? rows : 1, 16);
    L->mant_bytes = L->planes * L->plane_stride;
    L->exp_bytes = round_up((L->nkb > 0 ? L->nkb : 1) * L->rs, 128);
    return HBFP_OK;
}

// ------------------------------------------------------------------------------ launch plumbing

#define HBFP_CUDA_OK(expr)                          \
    do {                                            \
        cudaError_t _e = (expr);                    \
        if (_e != cudaSuccess) return HBFP_ERR_CUDA; \
    } while (0)

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? HBFP_OK : HBFP_ERR_CUDA; }

// A packed operand as the kernels see it.
struct Packed {
    const int8_t* mant;   // plane 0
    const int8_t* exps;   // [nkb][rs]
    Layout L;
    int mant_bits;
};

// Quantiser launchers (quantize.cu).
int launch_quantize(const float* x, int64_t d0, int64_t d1, int64_t ld, int contract_axis,
                    const hbfp_format* f, int8_t* mant, int8_t* exps, cudaStream_t st);
int launch_quantize_tiles(const float* w, int64_t d0, int64_t d1, int64_t ld, const hbfp_format* f,
                          int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1,
                          int8_t* tile_exps, cudaStream_t st);
int launch_quantize_conv_weights(const float* w, int64_t taps, int64_t c_in, int64_t c_out, int64_t ld,
                                 const hbfp_format* f, int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1,
                                 int8_t* tile_exps, cudaStream_t st);
// Wide weight storage: mode 0 quantise FP32 weights, 1 apply an FP32 update in place, 2 read only; in every
// mode the packed narrow views are written when their pointers are given.
int launch_wide(int mode, const float* src, int64_t ld, int64_t d0, int64_t d1, const hbfp_format* f,
                int16_t* wide, int8_t* wide_exps, int8_t* mant_c0, int8_t* exps_c0, int8_t* mant_c1, int8_t* exps_c1,
                cudaStream_t st);
int launch_wide_dequantize(const int16_t* wide, const int8_t* exps, int64_t d0, int64_t d1, int tile, float* out,
                           int64_t ldo, cudaStream_t st);
// Packed convolution operand gathered from the packed per-pixel operand.
int launch_im2col_packed(const int8_t* xm, const int8_t* xe, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw,
                         int pad, const hbfp_format* f, int8_t* om, int8_t* oe, cudaStream_t st);
// Packed transposed convolution operand (blocks along the output pixels) straight from the FP32 activations.
int launch_im2col_cols(const float* x, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw, int pad,
                       const hbfp_format* f, int8_t* mant, int8_t* exps, cudaStream_t st);
int launch_unpack(const Packed& p, int16_t* q, int8_t* s, cudaStream_t st);
int launch_dequantize(const Packed& p, float* out, int64_t ld, cudaStream_t st);

// GEMM launchers. P (optional) receives the per-block integer sums [M][N][nkb].
int launch_gemm_simt(int64_t M, int64_t N, int64_t K, const Packed& a, const Packed& b, float* C,
                     int64_t ldc, int32_t* P, cudaStream_t st);

// Tiled dp4a kernel for small problems (gemm_small.cu): one-plane operands, one launch, no split-K.
bool small_gemm_eligible(int64_t M, int64_t N, const Packed& a, const Packed& b, bool any_size);
int launch_gemm_small(int64_t M, int64_t N, const Packed& a, const Packed& b, float* C, int64_t ldc, cudaStream_t st);

struct TensorPlan {
    int supported;      // 0: this case has no tensor-core kernel
    int n_tile;         // 64, 128 or 256
    int splits;         // split-K factor (1 = none)
    int64_t kb_per_split;
    size_t partial_bytes;  // split-K scratch
};
TensorPlan plan_gemm_tensor(int64_t M, int64_t N, int64_t K, const Layout& la, const Layout& lb,
                            int mant_bits_a, int mant_bits_b);
int launch_gemm_tensor(int64_t M, int64_t N, int64_t K, const Packed& a, const Packed& b, float* C,
                       int64_t ldc, int32_t* P, const TensorPlan& plan, void* partial,
                       cudaStream_t st);

// Paired-SM variant (two CTAs of a cluster per 256 x 256 tile): 8-bit mantissas, blocks up to 128,
// no split-K, enough tiles to occupy every SM pair.
bool pair_gemm_eligible(int64_t M, int64_t N, const Packed& a, const Packed& b, const TensorPlan& plan);
int launch_gemm_tensor_pair(int64_t M, int64_t N, const Packed& a, const Packed& b, float* C, int64_t ldc,
                            const TensorPlan& plan, void* partial, cudaStream_t st);

// Convolution forward as an implicit GEMM over the packed pixels (gemm_conv.cu).
int launch_conv_forward(const Packed& x, const Packed& wt, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw,
                        int pad, int64_t filters, float* Y, int64_t ldy, cudaStream_t st);

// One warp running the kernels' bounded barrier wait on a barrier nobody arrives on (test hook).
int launch_wait_probe(long long limit_cycles, int code, int* outcome, cudaStream_t st);
int launch_conv_dgrad_filters(const Packed& c1, int taps, int64_t c_in, int64_t c_out, int t, int8_t* mant_out,
                              int8_t* exps_out, const Layout& Lo, cudaStream_t st);
int pair_gemm_cycles(uint64_t* cycles);   // longest CTA of the last paired-SM GEMM launch on the current device, in SM cycles

// Device status word (bounded waits report here).
int32_t* device_status_word();   // device address, per current device
int read_clear_device_status(cudaStream_t st, int32_t* out);

}  // namespace hbfp
