// extern "C" entry points of the HBFP library: argument checks, workspace carving, dispatch.
#include "common.cuh"

#include <string.h>

namespace hbfp {

__device__ int32_t g_device_status;

int32_t* device_status_word() {
    int32_t* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_device_status) != cudaSuccess) return nullptr;
    return p;
}

int read_clear_device_status(cudaStream_t st, int32_t* out) {
    HBFP_CUDA_OK(cudaStreamSynchronize(st));
    int32_t v = 0, zero = 0;
    HBFP_CUDA_OK(cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v)));
    HBFP_CUDA_OK(cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)));
    *out = v;
    if (v == 0) return HBFP_OK;
    return v >= 900 && v < 1000 ? HBFP_ERR_EXPONENT_RANGE : HBFP_ERR_TIMEOUT;
}

namespace {

// Name of the GEMM kernel the calling thread's last hbfp_gemm* call launched (hbfp_last_gemm_kernel).
thread_local const char* t_last_gemm_kernel = "";

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct GemmPlan {
    Layout la, lb;
    size_t off_am, off_ae, off_bm, off_be, off_partial, total;
    TensorPlan tp;
};

int check_operand(const hbfp_operand* o) {
    if (!o || o->struct_size != sizeof(hbfp_operand)) return HBFP_ERR_INVALID_ARG;
    if (o->kind != HBFP_OPERAND_FP32 && o->kind != HBFP_OPERAND_PACKED) return HBFP_ERR_INVALID_ARG;
    return HBFP_OK;
}

int make_plan(int64_t M, int64_t N, int64_t K, const hbfp_operand* a, const hbfp_operand* b, GemmPlan* g) {
    if (M < 0 || N < 0 || K < 0) return HBFP_ERR_INVALID_ARG;
    int rc = check_operand(a);
    if (rc) return rc;
    rc = check_operand(b);
    if (rc) return rc;
    rc = make_layout(M, K, &a->fmt, &g->la);
    if (rc) return rc;
    rc = make_layout(N, K, &b->fmt, &g->lb);
    if (rc) return rc;
    if (g->la.b != g->lb.b) return HBFP_ERR_INVALID_ARG;   // the blocks of the two operands must coincide
    size_t off = 0;
    g->off_am = off; if (a->kind == HBFP_OPERAND_FP32) off += align_up((size_t)g->la.mant_bytes, 1024);
    g->off_ae = off; if (a->kind == HBFP_OPERAND_FP32) off += align_up((size_t)g->la.exp_bytes, 1024);
    g->off_bm = off; if (b->kind == HBFP_OPERAND_FP32) off += align_up((size_t)g->lb.mant_bytes, 1024);
    g->off_be = off; if (b->kind == HBFP_OPERAND_FP32) off += align_up((size_t)g->lb.exp_bytes, 1024);
    g->tp = plan_gemm_tensor(M, N, K, g->la, g->lb, a->fmt.mant_bits, b->fmt.mant_bits);
    g->off_partial = off;
    off += align_up(g->tp.partial_bytes, 1024);
    g->total = off;
    return HBFP_OK;
}

void fill_operand(hbfp_operand* o, const float* data, int64_t ld, int trans, const hbfp_format* f) {
    memset(o, 0, sizeof(*o));
    o->struct_size = sizeof(*o);
    o->kind = HBFP_OPERAND_FP32;
    o->data = data;
    o->ld = ld;
    o->trans = trans;
    if (f) o->fmt = *f;
}

// Quantises an FP32 operand into the workspace (or takes a packed one as is).
int resolve_operand(const hbfp_operand* o, bool is_a, int64_t rows, int64_t K, const Layout& L,
                    char* ws, size_t off_m, size_t off_e, Packed* out, cudaStream_t st) {
    out->L = L;
    out->mant_bits = o->fmt.mant_bits;
    if (o->kind == HBFP_OPERAND_PACKED) {
        if (!o->data || !o->exps) return HBFP_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(o->data) & 255) || (reinterpret_cast<uintptr_t>(o->exps) & 127))
            return HBFP_ERR_ALIGNMENT;
        out->mant = static_cast<const int8_t*>(o->data);
        out->exps = o->exps;
        return HBFP_OK;
    }
    if (!o->data && rows * K > 0) return HBFP_ERR_INVALID_ARG;
    int8_t* m = reinterpret_cast<int8_t*>(ws + off_m);
    int8_t* e = reinterpret_cast<int8_t*>(ws + off_e);
    out->mant = m;
    out->exps = e;
    const float* x = static_cast<const float*>(o->data);
    // A: trans 0 = stored [rows][K] (blocks along rows); trans 1 = stored [K][rows].
    // B: trans 0 = stored [K][rows] (blocks down columns); trans 1 = stored [rows][K].
    const bool k_contiguous = is_a ? (o->trans == 0) : (o->trans != 0);
    if (k_contiguous) {
        if (o->ld < K) return HBFP_ERR_INVALID_ARG;
        return launch_quantize(x, rows, K, o->ld, 1, &o->fmt, m, e, st);
    }
    if (o->ld < rows) return HBFP_ERR_INVALID_ARG;
    return launch_quantize(x, K, rows, o->ld, 0, &o->fmt, m, e, st);
}

int gemm_impl(int64_t M, int64_t N, int64_t K, const hbfp_operand* a, const hbfp_operand* b, float* C,
              int64_t ldc, void* workspace, size_t ws_bytes, uint32_t flags, int32_t* P, cudaStream_t st) {
    GemmPlan g;
    int rc = make_plan(M, N, K, a, b, &g);
    if (rc) return rc;
    if (flags > HBFP_GEMM_FORCE_SMALL) return HBFP_ERR_INVALID_ARG;
    if (P) {   // the inspection hook never splits K and needs no scratch
        g.total -= align_up(g.tp.partial_bytes, 1024);
        g.tp.partial_bytes = 0;
        g.tp.splits = 1;
        g.tp.kb_per_split = g.la.nkb;
    }
    if (M == 0 || N == 0) return HBFP_OK;
    if ((!C && !P) || ldc < N) return HBFP_ERR_INVALID_ARG;
    if (g.total > 0) {
        if (!workspace || ws_bytes < g.total) return HBFP_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(workspace) & 255) return HBFP_ERR_ALIGNMENT;
    }
    char* ws = static_cast<char*>(workspace);
    Packed pa, pb;
    rc = resolve_operand(a, true, M, K, g.la, ws, g.off_am, g.off_ae, &pa, st);
    if (rc) return rc;
    rc = resolve_operand(b, false, N, K, g.lb, ws, g.off_bm, g.off_be, &pb, st);
    if (rc) return rc;
    // a problem of a few hundred MOPs is over before a tensor-core kernel has filled its pipeline
    if (!P && (flags == HBFP_GEMM_AUTO || flags == HBFP_GEMM_FORCE_SMALL) &&
        small_gemm_eligible(M, N, pa, pb, flags == HBFP_GEMM_FORCE_SMALL)) {
        t_last_gemm_kernel = "gemm_small_kernel";
        return launch_gemm_small(M, N, pa, pb, C, ldc, st);
    }
    if (flags == HBFP_GEMM_FORCE_SMALL) return HBFP_ERR_UNSUPPORTED;
    const bool quad_rows = (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc % 4) == 0;
    const bool want_tensor = flags != HBFP_GEMM_FORCE_SIMT && g.tp.supported &&
                             (reinterpret_cast<uintptr_t>(C) & 3) == 0;
    if (want_tensor) {
        // With a short contraction (under 1 KiB of mantissas per row) a tile is bound by the write of
        // its C part, and the single-SM kernel, whose warps own wider row segments, is ~10 % faster.
        const bool long_k = g.la.nkb * g.la.bp >= 1024;
        const bool pair_ok = !P && quad_rows && flags != HBFP_GEMM_FORCE_TENSOR_1SM && pair_gemm_eligible(M, N, pa, pb, g.tp) &&
                             (long_k || flags == HBFP_GEMM_FORCE_TENSOR_2SM);
        if (pair_ok) {
            t_last_gemm_kernel = "gemm_tc2_kernel";
            return launch_gemm_tensor_pair(M, N, pa, pb, C, ldc, g.tp, ws ? ws + g.off_partial : nullptr, st);
        }
        if (flags == HBFP_GEMM_FORCE_TENSOR_2SM) return HBFP_ERR_UNSUPPORTED;
        t_last_gemm_kernel = "gemm_tc_kernel";
        return launch_gemm_tensor(M, N, K, pa, pb, C, ldc, P, g.tp, ws ? ws + g.off_partial : nullptr, st);
    }
    if (flags >= HBFP_GEMM_FORCE_TENSOR) return HBFP_ERR_UNSUPPORTED;
    t_last_gemm_kernel = "gemm_simt_kernel";
    return launch_gemm_simt(M, N, K, pa, pb, C, ldc, P, st);
}

}  // namespace
}  // namespace hbfp

using namespace hbfp;

extern "C" {

const char* hbfp_last_gemm_kernel(void) { return t_last_gemm_kernel; }

const char* hbfp_status_string(int status) {
    switch (status) {
        case HBFP_OK: return "ok";
        case HBFP_ERR_INVALID_ARG: return "invalid argument";
        case HBFP_ERR_UNSUPPORTED: return "unsupported format or size";
        case HBFP_ERR_ALIGNMENT: return "buffer not aligned as required";
        case HBFP_ERR_WORKSPACE: return "workspace missing or too small";
        case HBFP_ERR_CUDA: return "CUDA call failed";
        case HBFP_ERR_TIMEOUT: return "bounded device-side wait expired";
        case HBFP_ERR_EXPONENT_RANGE: return "operand exponents outside the tensor-core path's exact range";
        case HBFP_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of hbfp_gemm_static";
        default: return "unknown status";
    }
}

int hbfp_packed_layout(int64_t rows, int64_t k, const hbfp_format* fmt, hbfp_layout* out) {
    if (!out) return HBFP_ERR_INVALID_ARG;
    Layout L;
    int rc = make_layout(rows, k, fmt, &L);
    if (rc) return rc;
    out->rows = L.rows; out->k = L.k; out->b = L.b; out->bp = L.bp; out->nkb = L.nkb; out->kst = L.kst;
    out->planes = L.planes; out->plane_stride = L.plane_stride; out->rs = L.rs;
    out->mant_bytes = L.mant_bytes; out->exp_bytes = L.exp_bytes;
    return HBFP_OK;
}

int hbfp_packed_sizes(int64_t rows, int64_t k, const hbfp_format* fmt, size_t* mant_bytes, size_t* exp_bytes) {
    Layout L;
    int rc = make_layout(rows, k, fmt, &L);
    if (rc) return rc;
    if (mant_bytes) *mant_bytes = (size_t)L.mant_bytes;
    if (exp_bytes) *exp_bytes = (size_t)L.exp_bytes;
    return HBFP_OK;
}

int hbfp_quantize(const float* x, int64_t d0, int64_t d1, int64_t ld, int contract_axis,
                  const hbfp_format* fmt, void* mant, int8_t* exps, void* stream) {
    if (d0 < 0 || d1 < 0 || ld < d1 || (contract_axis != 0 && contract_axis != 1)) return HBFP_ERR_INVALID_ARG;
    if (!fmt) return HBFP_ERR_INVALID_ARG;
    if ((!x && d0 * d1 > 0) || !mant || !exps) return HBFP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mant) & 255) || (reinterpret_cast<uintptr_t>(exps) & 127)) return HBFP_ERR_ALIGNMENT;
    return launch_quantize(x, d0, d1, ld, contract_axis, fmt, static_cast<int8_t*>(mant), exps,
                           static_cast<cudaStream_t>(stream));
}

int hbfp_quantize_tiles(const float* w, int64_t d0, int64_t d1, int64_t ld, const hbfp_format* fmt,
                        void* mant_c0, int8_t* exps_c0, void* mant_c1, int8_t* exps_c1, int8_t* tile_exps,
                        void* stream) {
    if (d0 < 0 || d1 < 0 || ld < d1 || !fmt) return HBFP_ERR_INVALID_ARG;
    if ((!w && d0 * d1 > 0) || !mant_c0 || !exps_c0 || !mant_c1 || !exps_c1) return HBFP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mant_c0) & 255) || (reinterpret_cast<uintptr_t>(mant_c1) & 255) ||
        (reinterpret_cast<uintptr_t>(exps_c0) & 127) || (reinterpret_cast<uintptr_t>(exps_c1) & 127))
        return HBFP_ERR_ALIGNMENT;
    return launch_quantize_tiles(w, d0, d1, ld, fmt, static_cast<int8_t*>(mant_c0), exps_c0,
                                 static_cast<int8_t*>(mant_c1), exps_c1, tile_exps,
                                 static_cast<cudaStream_t>(stream));
}

int hbfp_quantize_conv_weights(const float* w, int64_t taps, int64_t c_in, int64_t c_out, int64_t ld,
                               const hbfp_format* fmt, void* mant_c0, int8_t* exps_c0, void* mant_c1, int8_t* exps_c1,
                               int8_t* tile_exps, void* stream) {
    if (!w || !fmt || taps <= 0 || c_in <= 0 || c_out <= 0 || ld < c_out) return HBFP_ERR_INVALID_ARG;
    if ((mant_c0 && !exps_c0) || (mant_c1 && !exps_c1) || (!mant_c0 && !mant_c1 && !tile_exps)) return HBFP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mant_c0) & 255) || (reinterpret_cast<uintptr_t>(mant_c1) & 255) ||
        (reinterpret_cast<uintptr_t>(exps_c0) & 127) || (reinterpret_cast<uintptr_t>(exps_c1) & 127))
        return HBFP_ERR_ALIGNMENT;
    return launch_quantize_conv_weights(w, taps, c_in, c_out, ld, fmt, static_cast<int8_t*>(mant_c0), exps_c0,
                                        static_cast<int8_t*>(mant_c1), exps_c1, tile_exps, static_cast<cudaStream_t>(stream));
}

static int wide_views_ok(void* mant_c0, int8_t* exps_c0, void* mant_c1, int8_t* exps_c1) {
    if (!mant_c0 && !mant_c1 && !exps_c0 && !exps_c1) return HBFP_OK;        // wide storage only
    if (!mant_c0 || !exps_c0 || !mant_c1 || !exps_c1) return HBFP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mant_c0) & 255) || (reinterpret_cast<uintptr_t>(mant_c1) & 255) ||
        (reinterpret_cast<uintptr_t>(exps_c0) & 127) || (reinterpret_cast<uintptr_t>(exps_c1) & 127))
        return HBFP_ERR_ALIGNMENT;
    return HBFP_OK;
}

int hbfp_wide_quantize(const float* w, int64_t d0, int64_t d1, int64_t ld, const hbfp_format* fmt, int16_t* wide,
                       int8_t* wide_exps, void* mant_c0, int8_t* exps_c0, void* mant_c1, int8_t* exps_c1, void* stream) {
    if (d0 < 0 || d1 < 0 || ld < d1 || !fmt) return HBFP_ERR_INVALID_ARG;
    if (d0 * d1 > 0 && (!w || !wide || !wide_exps)) return HBFP_ERR_INVALID_ARG;
    int rc = wide_views_ok(mant_c0, exps_c0, mant_c1, exps_c1);
    if (rc) return rc;
    return launch_wide(0, w, ld, d0, d1, fmt, wide, wide_exps, static_cast<int8_t*>(mant_c0), exps_c0,
                       static_cast<int8_t*>(mant_c1), exps_c1, static_cast<cudaStream_t>(stream));
}

int hbfp_wide_update(int16_t* wide, int8_t* wide_exps, const float* delta, int64_t d0, int64_t d1, int64_t ldd,
                     const hbfp_format* fmt, void* mant_c0, int8_t* exps_c0, void* mant_c1, int8_t* exps_c1, void* stream) {
    if (d0 < 0 || d1 < 0 || ldd < d1 || !fmt) return HBFP_ERR_INVALID_ARG;
    if (d0 * d1 > 0 && (!delta || !wide || !wide_exps)) return HBFP_ERR_INVALID_ARG;
    int rc = wide_views_ok(mant_c0, exps_c0, mant_c1, exps_c1);
    if (rc) return rc;
    return launch_wide(1, delta, ldd, d0, d1, fmt, wide, wide_exps, static_cast<int8_t*>(mant_c0), exps_c0,
                       static_cast<int8_t*>(mant_c1), exps_c1, static_cast<cudaStream_t>(stream));
}

int hbfp_wide_narrow(const int16_t* wide, const int8_t* wide_exps, int64_t d0, int64_t d1, const hbfp_format* fmt,
                     void* mant_c0, int8_t* exps_c0, void* mant_c1, int8_t* exps_c1, void* stream) {
    if (d0 < 0 || d1 < 0 || !fmt || (d0 * d1 > 0 && (!wide || !wide_exps))) return HBFP_ERR_INVALID_ARG;
    if (!mant_c0 || !mant_c1) return HBFP_ERR_INVALID_ARG;
    int rc = wide_views_ok(mant_c0, exps_c0, mant_c1, exps_c1);
    if (rc) return rc;
    return launch_wide(2, nullptr, d1, d0, d1, fmt, const_cast<int16_t*>(wide), const_cast<int8_t*>(wide_exps),
                       static_cast<int8_t*>(mant_c0), exps_c0, static_cast<int8_t*>(mant_c1), exps_c1,
                       static_cast<cudaStream_t>(stream));
}

int hbfp_wide_dequantize(const int16_t* wide, const int8_t* wide_exps, int64_t d0, int64_t d1, int32_t tile, float* out,
                         int64_t ldo, void* stream) {
    if (d0 < 0 || d1 < 0 || tile <= 0 || ldo < d1) return HBFP_ERR_INVALID_ARG;
    if (d0 * d1 > 0 && (!wide || !wide_exps || !out)) return HBFP_ERR_INVALID_ARG;
    return launch_wide_dequantize(wide, wide_exps, d0, d1, tile, out, ldo, static_cast<cudaStream_t>(stream));
}

int hbfp_im2col_packed(const void* mant_x, const int8_t* exps_x, int64_t n, int64_t h, int64_t w, int64_t c, int kh,
                       int kw, int pad, const hbfp_format* fmt, void* mant_out, int8_t* exps_out, void* stream) {
    if (!fmt || n < 0 || h <= 0 || w <= 0 || c <= 0 || kh <= 0 || kw <= 0 || pad < 0) return HBFP_ERR_INVALID_ARG;
    if (!mant_x || !exps_x || !mant_out || !exps_out) return HBFP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mant_x) & 255) || (reinterpret_cast<uintptr_t>(mant_out) & 255) ||
        (reinterpret_cast<uintptr_t>(exps_out) & 127))
        return HBFP_ERR_ALIGNMENT;
    return launch_im2col_packed(static_cast<const int8_t*>(mant_x), exps_x, n, h, w, c, kh, kw, pad, fmt,
                                static_cast<int8_t*>(mant_out), exps_out, static_cast<cudaStream_t>(stream));
}

int hbfp_conv_forward(const void* mant_x, const int8_t* exps_x, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw,
                      int pad, const hbfp_format* fmt_x, const hbfp_operand* filters_op, int64_t filters, float* Y,
                      int64_t ldy, void* stream) {
    if (!fmt_x || !filters_op || n < 0 || h <= 0 || w <= 0 || c <= 0 || kh <= 0 || kw <= 0 || pad < 0 || filters <= 0)
        return HBFP_ERR_INVALID_ARG;
    if (!mant_x || !exps_x || !Y || ldy < filters) return HBFP_ERR_INVALID_ARG;
    if (filters_op->struct_size != sizeof(hbfp_operand) || filters_op->kind != HBFP_OPERAND_PACKED || !filters_op->data ||
        !filters_op->exps)
        return HBFP_ERR_INVALID_ARG;
    if (fmt_x->block != c || fmt_x->tile != 0 || filters_op->fmt.block != c) return HBFP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(mant_x) & 255) || (reinterpret_cast<uintptr_t>(filters_op->data) & 255)) return HBFP_ERR_ALIGNMENT;
    Packed px, pw;
    int rc = make_layout(n * h * w, c, fmt_x, &px.L);
    if (rc) return rc;
    rc = make_layout(filters, (int64_t)kh * kw * c, &filters_op->fmt, &pw.L);
    if (rc) return rc;
    px.mant = static_cast<const int8_t*>(mant_x);
    px.exps = exps_x;
    px.mant_bits = fmt_x->mant_bits;
    pw.mant = static_cast<const int8_t*>(filters_op->data);
    pw.exps = static_cast<const int8_t*>(filters_op->exps);
    pw.mant_bits = filters_op->fmt.mant_bits;
    if (n == 0) return HBFP_OK;
    t_last_gemm_kernel = "conv_fwd_kernel";
    return launch_conv_forward(px, pw, n, h, w, c, kh, kw, pad, filters, Y, ldy, static_cast<cudaStream_t>(stream));
}

int hbfp_conv_dgrad_filters(const void* mant_c1, const int8_t* exps_c1, int kh, int kw, int64_t c_in, int64_t c_out,
                            const hbfp_format* fmt, void* mant_out, int8_t* exps_out, void* stream) {
    if (!fmt || kh <= 0 || kw <= 0 || c_in < 0 || c_out <= 0) return HBFP_ERR_INVALID_ARG;
    if (!mant_c1 || !exps_c1 || !mant_out || !exps_out) return HBFP_ERR_INVALID_ARG;
    const int64_t t = fmt->tile;
    if (t <= 0 || fmt->block != t) return HBFP_ERR_INVALID_ARG;
    // whole 16-byte pieces of unpadded blocks: tiles of 32, 64 or 128 output maps
    if ((t != 32 && t != 64 && t != 128) || c_out % t != 0 || c_in % t != 0) return HBFP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(mant_c1) & 255) || (reinterpret_cast<uintptr_t>(mant_out) & 255)) return HBFP_ERR_ALIGNMENT;
    const int64_t taps = (int64_t)kh * kw;
    Packed c1;
    Layout Lo;
    int rc = make_layout(taps * c_in, c_out, fmt, &c1.L);
    if (rc) return rc;
    rc = make_layout(c_in, taps * c_out, fmt, &Lo);
    if (rc) return rc;
    c1.mant = static_cast<const int8_t*>(mant_c1);
    c1.exps = exps_c1;
    c1.mant_bits = fmt->mant_bits;
    return launch_conv_dgrad_filters(c1, (int)taps, c_in, c_out, (int)t, static_cast<int8_t*>(mant_out), exps_out, Lo,
                                     static_cast<cudaStream_t>(stream));
}

int hbfp_im2col_packed_t(const float* x, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw, int pad,
                         const hbfp_format* fmt, void* mant, int8_t* exps, void* stream) {
    if (!fmt || n < 0 || h <= 0 || w <= 0 || c <= 0 || kh <= 0 || kw <= 0 || pad < 0) return HBFP_ERR_INVALID_ARG;
    if ((!x && n > 0) || !mant || !exps) return HBFP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mant) & 255) || (reinterpret_cast<uintptr_t>(exps) & 127)) return HBFP_ERR_ALIGNMENT;
    return launch_im2col_cols(x, n, h, w, c, kh, kw, pad, fmt, static_cast<int8_t*>(mant), exps,
                              static_cast<cudaStream_t>(stream));
}

int hbfp_unpack(const void* mant, const int8_t* exps, int64_t rows, int64_t k, const hbfp_format* fmt,
                int16_t* q, int8_t* s, void* stream) {
    Packed p;
    int rc = make_layout(rows, k, fmt, &p.L);
    if (rc) return rc;
    if (!mant || !exps) return HBFP_ERR_INVALID_ARG;
    p.mant = static_cast<const int8_t*>(mant);
    p.exps = exps;
    p.mant_bits = fmt->mant_bits;
    return launch_unpack(p, q, s, static_cast<cudaStream_t>(stream));
}

int hbfp_dequantize(const void* mant, const int8_t* exps, int64_t rows, int64_t k, const hbfp_format* fmt,
                    float* out, int64_t ld, void* stream) {
    Packed p;
    int rc = make_layout(rows, k, fmt, &p.L);
    if (rc) return rc;
    if (!mant || !exps || !out || ld < k) return HBFP_ERR_INVALID_ARG;
    p.mant = static_cast<const int8_t*>(mant);
    p.exps = exps;
    p.mant_bits = fmt->mant_bits;
    return launch_dequantize(p, out, ld, static_cast<cudaStream_t>(stream));
}

int hbfp_gemm_q_workspace(int64_t M, int64_t N, int64_t K, const hbfp_operand* a, const hbfp_operand* b,
                          size_t* bytes) {
    if (!bytes) return HBFP_ERR_INVALID_ARG;
    GemmPlan g;
    int rc = make_plan(M, N, K, a, b, &g);
    if (rc) return rc;
    *bytes = g.total;
    return HBFP_OK;
}

int hbfp_gemm_workspace(int transA, int transB, int64_t M, int64_t N, int64_t K, const hbfp_format* fmtA,
                        const hbfp_format* fmtB, size_t* bytes) {
    if (!fmtA || !fmtB) return HBFP_ERR_INVALID_ARG;
    hbfp_operand a, b;
    fill_operand(&a, nullptr, 0, transA, fmtA);
    fill_operand(&b, nullptr, 0, transB, fmtB);
    return hbfp_gemm_q_workspace(M, N, K, &a, &b, bytes);
}

int hbfp_gemm_q(int64_t M, int64_t N, int64_t K, const hbfp_operand* a, const hbfp_operand* b, float* C,
                int64_t ldc, void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
    if (!C && M * N > 0) return HBFP_ERR_INVALID_ARG;
    return gemm_impl(M, N, K, a, b, C, ldc, workspace, workspace_bytes, flags, nullptr,
                     static_cast<cudaStream_t>(stream));
}

int hbfp_gemm(int transA, int transB, int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
              const float* B, int64_t ldb, float* C, int64_t ldc, const hbfp_format* fmtA,
              const hbfp_format* fmtB, void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
    if (!fmtA || !fmtB) return HBFP_ERR_INVALID_ARG;
    hbfp_operand a, b;
    fill_operand(&a, A, lda, transA, fmtA);
    fill_operand(&b, B, ldb, transB, fmtB);
    return hbfp_gemm_q(M, N, K, &a, &b, C, ldc, workspace, workspace_bytes, flags, stream);
}

int hbfp_gemm_block_partials(int64_t M, int64_t N, int64_t K, const hbfp_operand* a, const hbfp_operand* b,
                             int32_t* P, uint32_t impl, void* stream) {
    if (!P || !a || !b) return HBFP_ERR_INVALID_ARG;
    if (a->kind != HBFP_OPERAND_PACKED || b->kind != HBFP_OPERAND_PACKED) return HBFP_ERR_INVALID_ARG;
    if (impl != HBFP_GEMM_FORCE_SIMT && impl != HBFP_GEMM_FORCE_TENSOR) return HBFP_ERR_INVALID_ARG;
    return gemm_impl(M, N, K, a, b, nullptr, N, nullptr, 0, impl, P, static_cast<cudaStream_t>(stream));
}

int hbfp_selftest_bounded_wait(int64_t limit_cycles, int32_t code, int32_t* outcome, void* stream) {
    return launch_wait_probe((long long)limit_cycles, (int)code, reinterpret_cast<int*>(outcome), static_cast<cudaStream_t>(stream));
}

int hbfp_last_gemm_cycles(uint64_t* cycles) {
    if (!cycles) return HBFP_ERR_INVALID_ARG;
    return pair_gemm_cycles(cycles);
}

int hbfp_device_status(void* stream, int32_t* status) {
    if (!status) return HBFP_ERR_INVALID_ARG;
    return read_clear_device_status(static_cast<cudaStream_t>(stream), status);
}

}  // extern "C"
