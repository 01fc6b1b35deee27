/* hbfp.h - C ABI of the HBFP dot-product path for NVIDIA B200 (sm_100a).
 *
 * Hybrid block floating point (Drumond, Lin, Jaggi, Falsafi: "Training DNNs with Hybrid
 * Block Floating Point") performs every dot product of DNN training in block floating
 * point (BFP) and everything else in floating point. This library is that dot-product
 * path: FP32 -> BFP conversion and the BFP matrix products of a training step, as CUDA
 * kernels. All matrix pointers are DEVICE pointers unless a comment says "host"; all
 * matrices are row-major; every call is asynchronous on the caller's stream (a
 * cudaStream_t passed as void*, NULL = the legacy default stream), allocates nothing and
 * never synchronises unless stated. Functions return an hbfp_status code; on error the
 * outputs are unspecified but nothing is written out of bounds.
 *
 * ---- Number format (Eq. 1; Sec. 4.1; Sec. 5.3) -------------------------------------
 * A block of values shares one exponent; element i of the block is  q_i * 2^s  with an
 * integer mantissa q_i of m bits (sign + m-1 magnitude bits, |q_i| <= 2^(m-1)-1).
 *   amax = max |x_i| over the block;   e = floor(log2 amax) + 1   (exp_mode 0; equals
 *   ceil(log2 amax) except at exact powers of two, where it avoids saturating the maximum);
 *   s = max(e - (m-1), -63);  all-zero block: s = -63.
 *   rounding 0: q = clamp(round-half-even(x * 2^-s));
 *   rounding 1: stochastic, 16 random bits r per element:
 *               Y = floor(fl32(x * 2^(16-s))),  q = clamp(floor((Y + r) / 65536)).
 * The random bits come from Philox4x32-10 with key = (seed lo, seed hi) and counter =
 * (g lo, g hi, stream_id, 0), g = L >> 3, where L = i*d1 + j is the row-major index of
 * the element in the FP32 matrix AS PASSED (before any trans flag; independent of
 * blocking and layout). Of the four output words, element L takes 16-bit half (L & 1) of
 * word (L & 7) >> 1. The same (seed, stream_id, L) always gives the same draw.
 * Blocks are 1-D runs of `block` consecutive elements along the contraction axis of the
 * GEMM the operand feeds (block = 0: the whole axis, i.e. one exponent per row of A / per
 * column of B, Sec. 4), or, for weights, 2-D tile x tile squares of the stored matrix that
 * are shared by W and its transpose (Sec. 4.2 "Tiling"). Ragged last blocks share their
 * exponent among the elements that exist. Inputs must be finite.
 *
 * ---- Packed operand layout -----------------------------------------------------------
 * A quantised GEMM operand with `rows` non-contraction lines and contraction length k:
 *   b   = block (or k when block == 0),  nkb = ceil(k / b)
 *   bp  = padded block: 32, 64 or 128 for b <= 32, 64, 128; else b rounded up to 128
 *   kst = nkb*bp rounded up to a multiple of 128 (bytes per row)
 *   mantissas: `planes` planes of int8 [rows][kst]; block kb of a row occupies bytes
 *              [kb*bp, kb*bp + b), everything else in the row is zero. m <= 8: one plane
 *              holding q. 8 < m <= 12: plane 0 holds hi = q >> 4 (arithmetic), plane 1
 *              holds lo = q & 15, so q = 16*hi + lo exactly; planes are plane_stride bytes
 *              apart (rows*kst rounded up to 1024).
 *   exponents: int8 [nkb][rs], rs = rows rounded up to 16; entry [kb][r] is s of block kb
 *              of line r (bytes r >= rows are zero).
 * hbfp_packed_layout() returns these numbers; mantissa and exponent buffers must be
 * 256-byte and 128-byte aligned respectively (cudaMalloc/torch allocations are).
 */
#ifndef HBFP_H_
#define HBFP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define HBFP_API
#else
#define HBFP_API __attribute__((visibility("default")))
#endif

typedef enum hbfp_status {
    HBFP_OK = 0,
    HBFP_ERR_INVALID_ARG = 1, /* null pointer, negative size, ld too small, bad enum value   */
    HBFP_ERR_UNSUPPORTED = 2, /* a valid request this build has no kernel for                */
    HBFP_ERR_ALIGNMENT = 3,   /* a packed buffer or C is not aligned as documented           */
    HBFP_ERR_WORKSPACE = 4,   /* workspace pointer null or smaller than the query returned   */
    HBFP_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (launch, tensor map, ...)  */
    HBFP_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (see hbfp_device_status) */
    HBFP_ERR_STATIC_LIMIT = 7, /* hbfp_gemm_static: the problem needs more than the built-in scratch */
    HBFP_ERR_EXPONENT_RANGE = 8 /* hbfp_device_status: a tensor-core GEMM met block exponents outside its exact range */
} hbfp_status;

#define HBFP_ROUND_NEAREST_EVEN 0
#define HBFP_ROUND_STOCHASTIC 1

/* Format of one quantised operand. Set struct_size = sizeof(hbfp_format). */
typedef struct hbfp_format {
    uint32_t struct_size;
    int32_t mant_bits; /* m: 3..12 (sign included). 8 and 12 are the paper's design points     */
    int32_t block;     /* b: 1-D block length along the contraction axis; 0 = whole axis        */
    int32_t tile;      /* 0 = 1-D blocks; t > 0 = t x t tiles of the stored matrix (block == t)  */
    int32_t rounding;  /* HBFP_ROUND_NEAREST_EVEN or HBFP_ROUND_STOCHASTIC                       */
    int32_t exp_mode;  /* 0 = floor(log2 amax)+1 (default); 1 = literal ceil(log2 amax)          */
    uint32_t stream_id; /* third Philox counter word: distinct tensors use distinct ids          */
    uint32_t reserved;  /* must be 0                                                              */
    uint64_t seed;      /* Philox key                                                             */
} hbfp_format;

/* Geometry of a packed operand (all host-side numbers). */
typedef struct hbfp_layout {
    int64_t rows, k;       /* as passed                                     */
    int64_t b, bp, nkb;    /* block, padded block, number of blocks         */
    int64_t kst;           /* bytes per mantissa row                        */
    int64_t planes;        /* 1 or 2                                        */
    int64_t plane_stride;  /* bytes between mantissa planes                 */
    int64_t rs;            /* bytes per exponent row                        */
    int64_t mant_bytes;    /* planes * plane_stride                         */
    int64_t exp_bytes;     /* nkb * rs rounded up to 128                    */
} hbfp_layout;

/* Static, never-freed description of a status code (host). */
HBFP_API const char* hbfp_status_string(int status);

/* Host-only: layout and buffer sizes of a packed operand with `rows` lines of contraction
 * length `k` in format `fmt` (Eq. 1 storage; see "Packed operand layout"). */
HBFP_API int hbfp_packed_layout(int64_t rows, int64_t k, const hbfp_format* fmt, hbfp_layout* out);
HBFP_API int hbfp_packed_sizes(int64_t rows, int64_t k, const hbfp_format* fmt, size_t* mant_bytes,
                               size_t* exp_bytes);

/* FP32 -> BFP conversion, done ahead of each dot product with the shared exponent taken from the
 * block's largest magnitude (Sec. 4.1; the FP-to-BFP unit of Sec. 5.3).
 * x: FP32 [d0][d1], row stride ld >= d1 (elements). Blocks run along contract_axis (1 = along
 * rows of x, 0 = down its columns). Output: packed operand with rows = the other extent and
 * k = the extent of contract_axis (so contract_axis 0 writes the transposed, contraction-major
 * layout). With fmt->tile > 0 the exponents are those of tile x tile squares of x and each
 * entry [kb][r] repeats its tile's exponent. mant / exps: buffers of the sizes
 * hbfp_packed_sizes(rows, k) returns; fully overwritten. Any d0, d1 >= 0, any ld; the fastest
 * path needs x 16-byte aligned, ld % 4 == 0 and d1 % 8 == 0. */
HBFP_API int hbfp_quantize(const float* x, int64_t d0, int64_t d1, int64_t ld, int contract_axis,
                           const hbfp_format* fmt, void* mant, int8_t* exps, void* stream);

/* Weight conversion with shared tiles (Sec. 4.2 "Tiling"): one pass over w [d0][d1] that
 * writes BOTH packed views of the same mantissas - `*_c0` for GEMMs contracting over d0
 * (rows = d1, k = d0: forward Y = X W) and `*_c1` for GEMMs contracting over d1 (rows = d0,
 * k = d1: backward-data dX = dY W^T) - plus the tile exponent grid tile_exps
 * [ceil(d0/t)][ceil(d1/t)] (int8, may be NULL). Requires fmt->tile == fmt->block > 0,
 * tile <= 128. The backward pass therefore needs no re-quantisation. */
HBFP_API int hbfp_quantize_tiles(const float* w, int64_t d0, int64_t d1, int64_t ld,
                                 const hbfp_format* fmt, void* mant_c0, int8_t* exps_c0,
                                 void* mant_c1, int8_t* exps_c1, int8_t* tile_exps, void* stream);

/* Weights of a convolution layer with tiled feature-map dimensions (Sec. 5.1, last sentence). w: FP32
 * [taps * c_in][c_out] (taps = filter rows x filter columns, row index (tap, input map); pitch ld >=
 * c_out) - the matrix the convolution GEMM multiplies by. A tile is t input maps x t output maps and
 * spans every filter tap (fmt->tile == fmt->block == t, c_in % t == 0): the kh * kw * t * t weights of a
 * tile share one exponent, taken from their largest magnitude; the filter dimensions themselves are not
 * tiled. Writes view c0 (rows = c_out, k = taps * c_in: forward, hbfp_conv_forward) and / or view c1 (rows
 * = taps * c_in, k = c_out: backward-data) in the packed layout - either pair of pointers may be NULL -
 * and, if tile_exps is given, the grid [c_in / t][ceil(c_out / t)] of tile exponents (int8). Rounding,
 * seed and stream id as in hbfp_quantize (stochastic draws keyed by the index in w). Two passes over w
 * (weights are converted once per step). HBFP_ERR_UNSUPPORTED when c_in % t != 0. */
HBFP_API int hbfp_quantize_conv_weights(const float* w, int64_t taps, int64_t c_in, int64_t c_out, int64_t ld,
                                        const hbfp_format* fmt, void* mant_c0, int8_t* exps_c0, void* mant_c1,
                                        int8_t* exps_c1, int8_t* tile_exps, void* stream);

/* Filter operand of the backward-data convolution (Sec. 5.1: the backward pass of a convolution runs through
 * the same BFP dot products; Sec. 4.2: the weight tiles are shared between the passes). For a kh x kw filter,
 * stride 1, the gradient with respect to the input is the convolution of the output gradient with the
 * filters turned by 180 degrees and with the roles of input and output maps swapped:
 *   dX[p][ci] = sum over taps and co of dY[p + (pad' - tap')][co] * w[(taps - 1 - tap'), ci, co],  pad' = k - 1 - pad.
 * This call builds that operand, rows = c_in, contraction = taps x c_out, from view c1 of
 * hbfp_quantize_conv_weights (mant_c1 / exps_c1: rows = taps * c_in, contraction = c_out; device, 256-byte
 * aligned mantissas) by copying packed bytes and tile exponents: no value is converted again, so forward and
 * backward-data use the same mantissas. fmt: the format the weights were converted with (tile == block = t).
 * mant_out / exps_out: device buffers of the sizes hbfp_packed_sizes(c_in, taps * c_out, fmt) returns, mantissas
 * 256-byte aligned, fully overwritten. hbfp_conv_forward on the packed output gradient (block = c_out) with this
 * operand, `filters` = c_in and padding pad' then yields dX without the FP32 matrix of im2col-shaped gradients.
 * One launch, asynchronous on `stream`. Errors: HBFP_ERR_INVALID_ARG (null pointers, tile != block, sizes <= 0),
 * HBFP_ERR_UNSUPPORTED (t not 32, 64 or 128, or c_in or c_out not a multiple of t), HBFP_ERR_ALIGNMENT. */
HBFP_API int hbfp_conv_dgrad_filters(const void* mant_c1, const int8_t* exps_c1, int kh, int kw, int64_t c_in,
                                     int64_t c_out, const hbfp_format* fmt, void* mant_out, int8_t* exps_out,
                                     void* stream);

/* Wide weight storage (Sec. 4.2 "Wide weight storage": weights are kept with wider mantissas, only
 * weight updates use them, and the forward and backward passes read only the most significant bits).
 * The long-lived copy of w [d0][d1] is `wide`: int16 mantissas, row-major with pitch d1 (device,
 * 2-byte aligned, d0 * d1 elements), and `wide_exps`: one int8 exponent (of the 16-bit LSB) per
 * tile x tile square, [ceil(d0/t)][ceil(d1/t)] (device). fmt->tile == fmt->block = t in 1..128;
 * fmt->rounding, seed, stream_id and exp_mode govern the conversion to 16 bits (stochastic rounding
 * draws by the element's row-major index in w); fmt->mant_bits = m in 3..12 is the width of the narrow
 * copy: its mantissas are the top m bits of the wide mantissa after half a narrow unit has been added,
 * clamp(floor((q16 + 2^(15-m)) / 2^(16-m)), +-(2^(m-1) - 1)): the wide value rounded to nearest, ties
 * upward (plain truncation would leave every narrow weight half a narrow ULP low, a bias that adds up
 * over a dot product), under the exponent s16 + 16 - m. `wide` itself holds the bare mantissas q16. The narrow copy is
 * written as the two packed views of
 * hbfp_quantize_tiles (`*_c0`: rows = d1, k = d0; `*_c1`: rows = d0, k = d1; buffers of the sizes
 * hbfp_packed_sizes returns, fully overwritten); both mant_c0 and mant_c1 may be NULL to skip it, one
 * of them alone may not.
 *   hbfp_wide_quantize  w (FP32, pitch ld >= d1) -> wide storage (+ narrow views)
 *   hbfp_wide_update    wide <- 16-bit quantisation of fl32(wide * 2^s16 + delta) with fresh tile
 *                       exponents, in place; delta: FP32 [d0][d1], pitch ldd >= d1 (the update the
 *                       optimiser computed in FP32, Sec. 5.1) (+ narrow views of the new weights)
 *   hbfp_wide_narrow    wide storage -> narrow views only (reads 2 bytes per weight)
 * One launch, one CTA per tile; asynchronous on `stream`. Errors: HBFP_ERR_INVALID_ARG (null or
 * inconsistent arguments, tile != block), HBFP_ERR_UNSUPPORTED (tile > 128, m outside 3..12),
 * HBFP_ERR_ALIGNMENT (view buffers as for hbfp_quantize). */
HBFP_API int hbfp_wide_quantize(const float* w, int64_t d0, int64_t d1, int64_t ld, const hbfp_format* fmt,
                                int16_t* wide, int8_t* wide_exps, void* mant_c0, int8_t* exps_c0,
                                void* mant_c1, int8_t* exps_c1, void* stream);
HBFP_API int hbfp_wide_update(int16_t* wide, int8_t* wide_exps, const float* delta, int64_t d0, int64_t d1,
                              int64_t ldd, const hbfp_format* fmt, void* mant_c0, int8_t* exps_c0,
                              void* mant_c1, int8_t* exps_c1, void* stream);
HBFP_API int hbfp_wide_narrow(const int16_t* wide, const int8_t* wide_exps, int64_t d0, int64_t d1,
                              const hbfp_format* fmt, void* mant_c0, int8_t* exps_c0, void* mant_c1,
                              int8_t* exps_c1, void* stream);

/* Value of the wide copy as FP32 (Eq. 1): out[i][j] = wide[i][j] * 2^wide_exps[i/tile][j/tile], exact
 * (16-bit mantissas fit binary32). out: FP32 [d0][d1], pitch ldo >= d1 (device). What the FP32 parts
 * of training (the optimiser, regularisation: Sec. 4.1) see of the weights. Asynchronous on `stream`;
 * HBFP_ERR_INVALID_ARG for null pointers, tile <= 0 or ldo < d1. */
HBFP_API int hbfp_wide_dequantize(const int16_t* wide, const int8_t* wide_exps, int64_t d0, int64_t d1,
                                  int32_t tile, float* out, int64_t ldo, void* stream);

/* Convolution operand without the FP32 im2col matrix (the paper runs convolutions through the same
 * BFP dot products, Sec. 5.1). x is an activation tensor [n][h][w][c] (channels last) that was
 * converted once with hbfp_quantize(x as [n*h*w][c], contract_axis 1, block = c): one block, hence
 * one exponent, per pixel. The convolution with a kh x kw filter, stride 1 and `pad` zeros around the
 * image is the GEMM [n*ho*wo][kh*kw*c] x [kh*kw*c][filters], ho = h + 2 pad - kh + 1, columns ordered
 * (filter row, filter column, channel); each block of c columns of a row is the channel vector of one
 * input pixel, so the packed A operand is a gather of the packed pixels: this call writes it (rows =
 * n*ho*wo, k = kh*kw*c, format fmt with fmt->block == c, fmt->tile == 0, c <= 128; positions outside
 * the image hold zero mantissas and the exponent -63 of an all-zero block). It is bit-identical to
 * hbfp_quantize of the FP32 im2col matrix under nearest-even rounding (under stochastic rounding the
 * draws were keyed by the element's index in x, not in the im2col matrix). mant_x / exps_x: the
 * packed pixels; mant_out / exps_out: buffers of the sizes hbfp_packed_sizes(n*ho*wo, kh*kw*c)
 * returns, fully overwritten. All device pointers; asynchronous on `stream`. */
HBFP_API int hbfp_im2col_packed(const void* mant_x, const int8_t* exps_x, int64_t n, int64_t h, int64_t w,
                                int64_t c, int kh, int kw, int pad, const hbfp_format* fmt, void* mant_out,
                                int8_t* exps_out, void* stream);

/* Backward-weight operand of the same convolution: dW [kh*kw*c][filters] = cols^T dY contracts over
 * the n*h*w output pixels, so the A operand is cols^T with blocks of fmt->block consecutive pixels
 * along each (tap, channel) row. This call converts it straight from the FP32 activations x
 * [n][h][w][c] (16-byte aligned, c % 4 == 0): rows = kh*kw*c, k = n*h*w, bit-identical to
 * hbfp_quantize(im2col matrix, contract_axis 0) under nearest-even rounding; under stochastic rounding
 * every entry takes the draw of the activation it is a copy of (keyed by its index in x, as in
 * hbfp_im2col_packed). Supported: an output as
 * large as the input (2 pad == kh - 1 == kw - 1), blocks of whole image rows (block in {16, 32, 64,
 * 128}, block % w == 0, h*w % block == 0), w a power of two >= 4; anything else returns
 * HBFP_ERR_UNSUPPORTED (convert the im2col matrix instead). mant / exps: buffers of the
 * sizes hbfp_packed_sizes(kh*kw*c, n*h*w) returns, fully overwritten. */
HBFP_API int hbfp_im2col_packed_t(const float* x, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw,
                                  int pad, const hbfp_format* fmt, void* mant, int8_t* exps, void* stream);

/* Packed -> canonical arrays for inspection: q [rows][k] int16 mantissas and s [rows][nkb]
 * int8 exponents (either may be NULL). */
HBFP_API int hbfp_unpack(const void* mant, const int8_t* exps, int64_t rows, int64_t k,
                         const hbfp_format* fmt, int16_t* q, int8_t* s, void* stream);

/* Packed -> FP32 values q * 2^s (Eq. 1), out [rows][k] with row stride ld. */
HBFP_API int hbfp_dequantize(const void* mant, const int8_t* exps, int64_t rows, int64_t k,
                             const hbfp_format* fmt, float* out, int64_t ld, void* stream);

/* One GEMM operand: either an FP32 matrix that the call quantises, or a packed operand
 * produced earlier (weights live in BFP and are reused, Sec. 4.1). Set struct_size. */
#define HBFP_OPERAND_FP32 0
#define HBFP_OPERAND_PACKED 1
typedef struct hbfp_operand {
    uint32_t struct_size;
    int32_t kind;       /* HBFP_OPERAND_FP32 or HBFP_OPERAND_PACKED                                 */
    const void* data;   /* FP32: the matrix. PACKED: mantissas                                       */
    const int8_t* exps; /* PACKED only                                                               */
    int64_t ld;         /* FP32 only: row stride in elements                                         */
    int32_t trans;      /* FP32 only. A: 0 = stored [M][K], 1 = [K][M]. B: 0 = [K][N], 1 = [N][K]    */
    int32_t reserved;
    hbfp_format fmt;    /* FP32: format to quantise to. PACKED: format it was quantised with         */
} hbfp_operand;

#define HBFP_GEMM_AUTO 0u        /* smallest problems: tiled kernel; else a tensor-core kernel when it supports the case, else SIMT */
#define HBFP_GEMM_FORCE_SIMT 1u  /* plain dp4a kernel (reference path, any format)           */
#define HBFP_GEMM_FORCE_TENSOR 2u /* tcgen05 kernel or HBFP_ERR_UNSUPPORTED                  */
#define HBFP_GEMM_FORCE_TENSOR_1SM 3u  /* as FORCE_TENSOR, but never the paired-SM tile kernel */
#define HBFP_GEMM_FORCE_TENSOR_2SM 4u  /* paired-SM tile kernel or HBFP_ERR_UNSUPPORTED        */
#define HBFP_GEMM_FORCE_SMALL 5u       /* the tiled kernel that HBFP_GEMM_AUTO takes for the smallest problems (contraction
                                          of at most 512 bytes, at most 296 tiles of 32 x 32; one launch, no split-K,
                                          one-plane operands) at any size, or HBFP_ERR_UNSUPPORTED */

/* Host-only: bytes of workspace hbfp_gemm / hbfp_gemm_q need for this problem (packed copies
 * of FP32 operands, split-K partial tiles). Depends only on its arguments. */
HBFP_API int hbfp_gemm_workspace(int transA, int transB, int64_t M, int64_t N, int64_t K,
                                 const hbfp_format* fmtA, const hbfp_format* fmtB, size_t* bytes);
HBFP_API int hbfp_gemm_q_workspace(int64_t M, int64_t N, int64_t K, const hbfp_operand* a,
                                   const hbfp_operand* b, size_t* bytes);

/* BFP matrix product C = op(A) op(B) (Eq. 2 per block; blocks accumulated in FP32, Sec. 4):
 *   P[i][j][kb] = sum_{k in block kb} qA[i][k] * qB[k][j]        exact integers (int32)
 *   C[i][j]     = sum_kb  float(P[i][j][kb]) * 2^(sA[i][kb] + sB[kb][j])   in FP32
 * A: FP32 [M][K] (transA = 0) or [K][M] (transA = 1), row stride lda; B: FP32 [K][N] (transB =
 * 0) or [N][K] (transB = 1), row stride ldb; C: FP32 [M][N], row stride ldc, overwritten.
 * Both operands are first quantised along the contraction axis (fmtA, fmtB; their blocks must
 * coincide) into `workspace` (>= hbfp_gemm_workspace bytes, 256-byte aligned).
 * forward Y = X W is (0,0); backward-data dX = dY W^T is (0,1); backward-weight dW = X^T dY is
 * (1,0). Without split-K the blocks are accumulated in ascending order with one FP32 rounding
 * each; with split-K (chosen for small C and long K) each split does so and the splits are
 * summed in ascending order. Exactness of the scaled FP32 accumulation needs sA + sB in
 * [-126, 127] (else the true product is outside binary32). The tensor-core kernels split the scale
 * 2^(sA + sB) into two factors and need more: the paired-SM kernel chooses the split per K-block and
 * 128-row tile and fails only when that tile's row exponents span more than 104 within one block
 * (or the products leave binary32); the single-SM kernel's biased path needs sA <= 103 (|A| < 2^110
 * at 8-bit mantissas; sA <= 96 for 12-bit mantissas). A kernel that meets exponents outside its range does not depart silently: it
 * records a code in the device status word (hbfp_device_status then returns
 * HBFP_ERR_EXPONENT_RANGE) and the values of C it wrote for that call are unspecified;
 * HBFP_GEMM_FORCE_SIMT computes the same product without the restriction. */
HBFP_API int hbfp_gemm(int transA, int transB, int64_t M, int64_t N, int64_t K, const float* A,
                       int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                       const hbfp_format* fmtA, const hbfp_format* fmtB, void* workspace,
                       size_t workspace_bytes, uint32_t flags, void* stream);

/* Built-in scratch of hbfp_gemm_static, in bytes. */
#define HBFP_STATIC_WORKSPACE_BYTES (16u << 20)

/* hbfp_gemm for callers that cannot allocate device memory (the paper has no counterpart: this
 * is a property of the library, not of the method). Who they are: code that runs inside another
 * program's memory discipline - a plug-in whose host framework has taken the whole device for
 * its own pool, so that a cudaMalloc from the plug-in fails; a serving or real-time loop in which
 * an allocation is forbidden because it may synchronise the device and stall every stream.
 * Same arguments and result as hbfp_gemm, minus the workspace: the packed operands and the split-K
 * partial tiles live in a fixed HBFP_STATIC_WORKSPACE_BYTES array in device memory that belongs to
 * the library (every GPU that loads the library holds it until the process exits). The call
 * allocates and frees nothing. Problems whose hbfp_gemm_workspace() exceeds the array are
 * rejected with HBFP_ERR_STATIC_LIMIT and nothing is launched (at 8-bit mantissas roughly
 * M*K + N*K <= 15 million elements, e.g. every GEMM of the 784-1024-1024-10 MLP at batch 128).
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call outside any stream capture. All calls share the one
 * array and it keeps the previous call's contents: nothing in it needs clearing between calls,
 * but two calls that overlap on the GPU (different streams, or a captured graph replayed
 * concurrently) race on it - run them on one stream or order them yourself. */
HBFP_API int hbfp_gemm_static(int transA, int transB, int64_t M, int64_t N, int64_t K, const float* A,
                              int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                              const hbfp_format* fmtA, const hbfp_format* fmtB, uint32_t flags,
                              void* stream);

/* Same product with each operand either FP32 (quantised by the call) or already packed: the
 * steady state of training, where W is quantised once per step into shared tiles and used by
 * forward and backward-data (Sec. 4.1, Sec. 4.2). A packed A has rows = M, k = K; a packed B
 * has rows = N, k = K. */
HBFP_API int hbfp_gemm_q(int64_t M, int64_t N, int64_t K, const hbfp_operand* a,
                         const hbfp_operand* b, float* C, int64_t ldc, void* workspace,
                         size_t workspace_bytes, uint32_t flags, void* stream);

/* Convolution forward pass as one implicit GEMM (Sec. 5.1: convolutions run through the same BFP dot
 * products): Y [n*h*w][filters] = conv(x, filters), stride 1, `pad` zeros around the image, an output as
 * large as the input (2 pad == kh - 1 == kw - 1). x: the activations [n][h][w][c] converted once per
 * pixel - hbfp_quantize(x as [n*h*w][c], contract_axis 1, block = c, fmt_x) - given as mant_x / exps_x;
 * filters_op: a packed operand with rows = filters, k = kh*kw*c, block = c, K ordered (filter row, filter
 * column, channel), e.g. view c0 of hbfp_quantize_tiles / hbfp_wide_* of the [kh*kw*c][filters] matrix or
 * hbfp_quantize of it with contract_axis 0. The kernel reads every tap's channel vectors straight from
 * the packed pixels (one 4-D TMA box per tap and 128 output pixels; positions outside the image read as
 * zero mantissas): the packed im2col operand of hbfp_im2col_packed is never formed. The result equals
 * hbfp_gemm_q on that operand bit for bit (taps accumulated in ascending order, one FP32 rounding each).
 * Y: FP32, 16-byte aligned, row stride ldy >= filters, ldy % 4 == 0. Supported: c in {64, 128}, mantissas
 * up to 8 bits, w in {16, 32, 64, 128}, h a multiple of 128 / w, up to 256 filters, kh * kw <= 25; any
 * other case returns HBFP_ERR_UNSUPPORTED and leaves Y untouched (use hbfp_im2col_packed + hbfp_gemm_q).
 * Exponent range as for the paired-SM GEMM (hbfp_gemm). Asynchronous on `stream`, allocates nothing. */
HBFP_API int hbfp_conv_forward(const void* mant_x, const int8_t* exps_x, int64_t n, int64_t h, int64_t w, int64_t c,
                               int kh, int kw, int pad, const hbfp_format* fmt_x, const hbfp_operand* filters_op,
                               int64_t filters, float* Y, int64_t ldy, void* stream);

/* Inspection hook: the exact per-block integer sums P [M][N][nkb] (int32) of two packed
 * operands (Eq. 2's fixed-point dot product), for small shapes. `impl` selects the kernel that
 * produces them: HBFP_GEMM_FORCE_SIMT or HBFP_GEMM_FORCE_TENSOR. */
HBFP_API int hbfp_gemm_block_partials(int64_t M, int64_t N, int64_t K, const hbfp_operand* a,
                                      const hbfp_operand* b, int32_t* P, uint32_t impl,
                                      void* stream);

/* Host-only: name of the GEMM kernel that the calling thread's most recent hbfp_gemm, hbfp_gemm_q,
 * hbfp_gemm_static or hbfp_gemm_block_partials call launched ("gemm_tc2_kernel": two SMs per 256 x 256
 * tile; "gemm_tc_kernel": one SM per tile; "gemm_simt_kernel"; "conv_fwd_kernel" after hbfp_conv_forward),
 * "" before the first launch. For
 * measurement scripts that must name the kernel they timed (the paper has no counterpart). The
 * string is static storage. */
HBFP_API const char* hbfp_last_gemm_kernel(void);

/* Synchronises the current device, then writes to *cycles (host) the length, in SM clock cycles, of the
 * most recent launch of the paired-SM GEMM kernel ("gemm_tc2_kernel") on that device: every CTA reads the
 * cycle counter when it starts and when it ends, and the largest difference is reported (0 before the
 * first such launch). Cycles divided by the launch's duration is the clock the SMs really ran at, which
 * under the board's power cap is lower than the clock the driver reports; measurement scripts use it to
 * tell a change of the code from a change of the clock (the paper has no counterpart). Returns
 * HBFP_ERR_INVALID_ARG for a null pointer, HBFP_ERR_CUDA if the copy fails. */
HBFP_API int hbfp_last_gemm_cycles(uint64_t* cycles);

/* Synchronises `stream`, then returns and clears the device-side status word of the current
 * device in *status (host int): 0, or a code recorded by a kernel. Codes below 900: a bounded wait
 * on a barrier expired (the kernel then abandons its work and exits; HBFP_ERR_TIMEOUT is returned).
 * Codes 900-999: a tensor-core GEMM met block exponents outside the range in which its scaled
 * accumulation is exact (see hbfp_gemm; HBFP_ERR_EXPONENT_RANGE is returned). */
HBFP_API int hbfp_device_status(void* stream, int32_t* status);

/* Self-test of the bounded waits (the paper has no counterpart: failure behaviour of this
 * library). Launches one warp that waits, with the same wait routine and abort protocol the GEMM
 * kernels use, on a barrier nobody arrives on, with a budget of `limit_cycles` SM cycles (0 ..
 * 1e8) instead of the kernels' ~2 s. The wait runs out, the warp records `code` (1 .. 899) in the
 * device status word and returns; *outcome (device int32, may be null) receives 2 (abandoned, abort
 * flag raised; 1 would mean the barrier completed). A following hbfp_device_status returns
 * HBFP_ERR_TIMEOUT with `code`. Touches no tensor memory and issues no copy. Asynchronous on
 * `stream`. */
HBFP_API int hbfp_selftest_bounded_wait(int64_t limit_cycles, int32_t code, int32_t* outcome, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HBFP_H_ */
