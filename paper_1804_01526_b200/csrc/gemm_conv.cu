// Convolution forward pass as an implicit BFP GEMM for sm_100a (Sec. 5.1: convolutions run through the
// same BFP dot products; Eq. 2 per filter tap, taps accumulated in FP32).
//
// The activations were converted once per pixel (one block of c channels, one exponent, per pixel),
// the filters once per (tap, filter) block. Row p of the GEMM is output pixel p, K-block t is filter
// tap t = (dy, dx), and the operand of (p, t) is the packed channel vector of input pixel
// (y + dy - pad, x + dx - pad): nothing has to be gathered into an im2col operand first. The producer
// warp issues, per tap, one 4-D TMA box per 128 output pixels straight from the packed pixels
// [n][h][w][c]; coordinates outside the image are filled with zero mantissas by the copy engine, which
// makes the padded taps contribute exactly +0 whatever exponent accompanies them.
//
// One CTA per SM, persistent over "super tiles" of RT x 128 output pixels x all filters (RT = 256 /
// N_TILE row tiles share one hand-over per tap, so that a hand-over always covers 128 x 256
// accumulator words). Roles as in the other tensor-core kernels: warp 0 producer, warp 1 MMA issuer and
// tensor-memory owner, warp 2 scale-table builder (it also gathers the pixel exponents of the taps),
// warps 4-11 rescale. Block sums: every tap starts with an MMA step of two constant all-255 operands
// taken as unsigned bytes, which overwrites the accumulator with OFFSET = 32 * 255 * 255; the tap's own
// steps land on top, a word read back is the positive pattern OFFSET + P, as binary32 the subnormal
// (OFFSET + P) * 2^-149, and two packed FMAs per pair of outputs finish Eq. 2 exactly (see gemm_tc2.cu).
// Every wait is bounded (tc_ptx.cuh); no copy is multicast and every tensor map covers this GPU's memory.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace hbfp {
namespace {

constexpr int CV_RESCALE_WARPS = 8, CV_CONTROL_WARPS = 4;
constexpr int CV_PRODUCER_WARP = 0, CV_MMA_WARP = 1, CV_TABLE_WARP = 2;
constexpr int CV_THREADS = 32 * (CV_CONTROL_WARPS + CV_RESCALE_WARPS);
constexpr int CV_REGS_RESCALE = 216, CV_REGS_CONTROL = 72;      // totals stay inside 384 threads x 168 registers
constexpr int CV_OFFSET = 32 * 255 * 255;
constexpr int CV_SHIFT = 86;
constexpr int CV_COLS = 256;          // accumulator columns per buffer: RT row tiles of N_TILE columns
constexpr int CV_BUFS = TMEM_COLS / CV_COLS;
constexpr int CV_TSLOTS = 2 * CV_BUFS;
constexpr int CV_MAX_TAPS = 25, CV_MAX_PAD = 2;
constexpr int CV_GRID_BYTES = 832;    // (R + 2 pad) rows of w + 32 pixel exponents of one row tile (data from column 16), pad <= 2

template <int C, int N_TILE>
struct ConvCfg {
    static constexpr int RT = CV_COLS / N_TILE;
    static constexpr int A_TILE = TILE_M * C;
    static constexpr int A_BYTES = RT * A_TILE;
    static constexpr int B_BYTES = N_TILE * C;
    static constexpr int STAGE = A_BYTES + B_BYTES;
    static constexpr int ONES_BYTES = 1024;
    static constexpr int SLOT_WORDS = N_TILE + RT * TILE_M;
    static constexpr int TABLE_BYTES = 4 * CV_TSLOTS * SLOT_WORDS;
    static constexpr int GRID_BYTES = RT * CV_GRID_BYTES;
    static constexpr int WEXP_BYTES = CV_MAX_TAPS * N_TILE;
    static constexpr int FIXED = 1024 /*align*/ + ONES_BYTES + TABLE_BYTES + GRID_BYTES + WEXP_BYTES + 1024 /*barriers*/;
    static constexpr int STAGES_RAW = (232448 - FIXED) / STAGE;
    static constexpr int STAGES = STAGES_RAW > 4 ? 4 : STAGES_RAW;
    static constexpr int SMEM = FIXED + STAGES * STAGE;
    static_assert(STAGES >= 2, "pipeline too shallow");
    static_assert(A_TILE % 1024 == 0 && B_BYTES % 1024 == 0, "tiles keep the swizzle atoms aligned");
    static_assert(GRID_BYTES % 16 == 0 && TABLE_BYTES % 16 == 0, "16-byte pieces");
};

struct ConvProblem {
    int n, h, w, kh, kw, pad, taps;
    int rows_per_tile;          // R = 128 / w image rows per row tile
    int tiles_per_image;        // h / R
    int row_tiles;              // n * h / R
    int super_tiles;
    int filters;
    const int8_t* exps_x;       // [n*h*w] pixel exponents
    const int8_t* exps_w;       // [taps][rs_w] filter exponents
    int64_t rs_w;
    float* Y;
    int64_t ldy;
    int32_t* status;
};

// ------------------------------------------------------------------------------ PTX

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// K-major tile whose rows are C bytes long, swizzled over C bytes (64B or 128B swizzle): 8-row groups
// 8 * C bytes apart; the start address advances by 32 bytes per K = 32 step.
template <int C>
__device__ __forceinline__ uint64_t smem_desc_rows(uint32_t addr, bool alias_groups = false) {
    const uint64_t sbo = alias_groups ? 0ull : (uint64_t)((8 * C) >> 4);
    const uint64_t layout = C == 128 ? 2ull : 4ull;        // 128-byte / 64-byte swizzle
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | (sbo << 32) | (1ull << 46) | (layout << 61);
}

template <int N_TILE>
__device__ __forceinline__ constexpr uint32_t idesc_conv(bool unsigned_ops) {
    return (2u << 4) | (unsigned_ops ? 0u : ((1u << 7) | (1u << 10))) | ((uint32_t)(N_TILE >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
}

__device__ __forceinline__ bool cv_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Poll first (a thread that try_wait has put to sleep wakes up late), then the bounded suspending wait.
__device__ __forceinline__ bool cv_wait_polled(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int code) {
    for (int i = 0; i < 4096; ++i)
        if (cv_test_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, abort_flag, status, code);
}

template <int N>
__device__ __forceinline__ void cv_ring_next(uint32_t& i, uint32_t& ph) {
    if (++i == N) { i = 0; ph ^= 1u; }
}

__device__ __forceinline__ uint32_t cv_scale_bits(int e, int sh) { return (uint32_t)(e + 127 + sh) << 23; }

// ------------------------------------------------------------------------------ kernel

template <int C, int N_TILE>
__global__ void __launch_bounds__(CV_THREADS, 1)
conv_fwd_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW, const ConvProblem p) {
    using G = ConvCfg<C, N_TILE>;
    constexpr int RT = G::RT, STAGES = G::STAGES;
    constexpr int HALF = N_TILE / 2;                 // columns of a row tile that one rescale warp owns
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t stage_base = base;                                        // STAGES x STAGE, 1024-aligned tiles
    const uint32_t ones_off = STAGES * G::STAGE;
    const uint32_t table_off = ones_off + G::ONES_BYTES;
    const uint32_t grid_off = table_off + G::TABLE_BYTES;
    const uint32_t wexp_off = grid_off + G::GRID_BYTES;
    const uint32_t bar_off = (wexp_off + G::WEXP_BYTES + 15u) & ~15u;
    uint32_t* tables = reinterpret_cast<uint32_t*>(base_ptr + table_off);     // [slot][N_TILE column scales | RT*128 row scales]
    int8_t* grid = reinterpret_cast<int8_t*>(base_ptr + grid_off);            // [row tile][(R + 2 pad) x (w + 2 pad)]
    int8_t* wexp = reinterpret_cast<int8_t*>(base_ptr + wexp_off);            // [tap][N_TILE]
    const uint32_t bars = base + bar_off;
    const uint32_t full_bar = bars;                          // stage landed
    const uint32_t empty_bar = full_bar + 8 * STAGES;        // stage consumed (MMA commit)
    const uint32_t tfull_bar = empty_bar + 8 * STAGES;       // tap sums complete (MMA commit) and scale table written
    const uint32_t tempty_bar = tfull_bar + 8 * CV_BUFS;     // buffer read by every rescale warp
    const uint32_t done_bar = tempty_bar + 8 * CV_BUFS;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + bar_off + 16 * STAGES + 16 * CV_BUFS + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int b = 0; b < CV_BUFS; ++b) {
            mbar_init(tfull_bar + 8 * b, 2);                 // MMA commit + table warp
            mbar_init(tempty_bar + 8 * b, CV_RESCALE_WARPS);
        }
        mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // constant operand of the offset step, and the filter exponents (the same for every tile)
    for (int i = threadIdx.x; i < G::ONES_BYTES / 4; i += CV_THREADS) reinterpret_cast<uint32_t*>(base_ptr + ones_off)[i] = 0xFFFFFFFFu;
    for (int i = threadIdx.x; i < p.taps * N_TILE; i += CV_THREADS) {
        const int t = i / N_TILE, j = i - t * N_TILE;
        wexp[i] = j < p.filters ? p.exps_w[(int64_t)t * p.rs_w + j] : (int8_t)0;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == CV_MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < CV_CONTROL_WARPS) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CV_REGS_CONTROL));
        if (warp == CV_PRODUCER_WARP) {
            // -------------------------------------------------------------- TMA producer
            if (lane == 0) {
                uint32_t s = 0, ph = 0, it = 0;
                bool ok = true;
                for (int st = blockIdx.x; ok && st < p.super_tiles; st += gridDim.x) {
                    for (int tap = 0; tap < p.taps; ++tap, ++it) {
                        if (!mbar_wait(empty_bar + 8 * s, ph ^ 1, abort_flag, p.status, 121)) { ok = false; break; }
                        const uint32_t fb = full_bar + 8 * s;
                        mbar_expect_tx(fb, (uint32_t)G::STAGE);
                        const uint32_t dst = stage_base + s * G::STAGE;
                        const int dy = tap / p.kw, dx = tap - dy * p.kw;
#pragma unroll
                        for (int r = 0; r < RT; ++r) {
                            // row tiles past the end lie in image n >= p.n: filled with zeros like any coordinate outside
                            const int rt = st * RT + r;
                            const int img = rt / p.tiles_per_image, y0 = (rt - img * p.tiles_per_image) * p.rows_per_tile;
                            tma_load_4d(dst + r * G::A_TILE, &mapX, 0, dx - p.pad, y0 + dy - p.pad, img, fb);
                        }
                        tma_load_2d(dst + G::A_BYTES, &mapW, tap * C, 0, fb);
                        cv_ring_next<STAGES>(s, ph);
                    }
                }
                const uint32_t back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;     // drain what is still in flight
                for (uint32_t k = 0; k < back; ++k) {
                    if (s == 0) { s = STAGES - 1; ph ^= 1u; } else { --s; }
                    mbar_wait(full_bar + 8 * s, ph, abort_flag, p.status, 122, false);
                }
            }
        } else if (warp == CV_MMA_WARP) {
            // -------------------------------------------------------------- MMA issuer
            if (lane == 0) {
                constexpr uint32_t idesc = idesc_conv<N_TILE>(false), idesc_ones = idesc_conv<N_TILE>(true);
                const uint64_t ones_desc = smem_desc_rows<C>(base + ones_off, true);
                uint32_t s = 0, ph = 0, b = 0, bph = 0;
                bool ok = true;
                for (int st = blockIdx.x; ok && st < p.super_tiles; st += gridDim.x) {
                    for (int tap = 0; tap < p.taps; ++tap) {
                        if (!mbar_wait(full_bar + 8 * s, ph, abort_flag, p.status, 221)) { ok = false; break; }
                        if (!cv_wait_polled(tempty_bar + 8 * b, bph, abort_flag, p.status, 222)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t src = stage_base + s * G::STAGE;
                        const uint64_t b_desc = smem_desc_rows<C>(src + G::A_BYTES);
#pragma unroll
                        for (int r = 0; r < RT; ++r) {
                            const uint32_t d = tmem_base + b * CV_COLS + r * N_TILE;
                            const uint64_t a_desc = smem_desc_rows<C>(src + r * G::A_TILE);
                            tc_mma_i8(d, ones_desc, ones_desc, idesc_ones, 0u);           // offset step: overwrites
#pragma unroll
                            for (int q = 0; q < C / 32; ++q) tc_mma_i8(d, a_desc + 2 * q, b_desc + 2 * q, idesc, 1u);
                        }
                        tc_commit(tfull_bar + 8 * b);
                        tc_commit(empty_bar + 8 * s);
                        cv_ring_next<CV_BUFS>(b, bph);
                        cv_ring_next<STAGES>(s, ph);
                    }
                }
                tc_commit(done_bar);
                mbar_wait(done_bar, 0, abort_flag, p.status, 223, false);
            }
        } else if (warp == CV_TABLE_WARP) {
            // -------------------------------------------------------------- scale-table builder
            // Per super tile it first lays out, for each row tile, the exponents of the input pixels that the
            // taps touch (the tile's image rows plus `pad` rows and columns around them; 127 marks a position
            // outside the image). The table of step k (tap by tap, across tiles) goes to slot k % 4 and its
            // arrival counts on tfull[k % 2]; it is written once the phase of step k - 2 on that barrier is
            // complete (see gemm_tc2.cu for why the slot's last readers are done by then).
            // Grid row gy holds image row y0 + gy - pad; its pixel x sits in column 16 + x, so that 16-byte pieces
            // of the exponent array land aligned; the columns next to the data stay at the mark for good.
            const int gw = p.w + 32, gh = p.rows_per_tile + 2 * p.pad;
            const int lw = 31 - __clz(p.w);                           // w is a power of two
            const int cpr = p.w >> 4;                                 // 16-byte pieces per image row
            for (int i = lane; i < RT * CV_GRID_BYTES; i += 32) grid[i] = (int8_t)127;
            __syncwarp();
            uint32_t b = 0, bph = 0, slot = 0;
            bool ok = true, out_of_range = false;
            for (int st = blockIdx.x; ok && st < p.super_tiles; st += gridDim.x) {
                // all the loads of a super tile are issued together: one trip to L2, not one per piece
                for (int i0 = 0; i0 < RT * gh * cpr; i0 += 64) {
                    uint4 val[2];
                    int dst[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int i = i0 + 32 * u + lane;
                        dst[u] = -1;
                        val[u] = make_uint4(0x7f7f7f7fu, 0x7f7f7f7fu, 0x7f7f7f7fu, 0x7f7f7f7fu);
                        if (i < RT * gh * cpr) {
                            const int r = i / (gh * cpr), j = i - r * (gh * cpr);
                            const int gy = j / cpr, xc = j - gy * cpr;
                            const int rt = st * RT + r;
                            const int img = rt / p.tiles_per_image, y0 = (rt - img * p.tiles_per_image) * p.rows_per_tile;
                            const int yy = y0 + gy - p.pad;
                            dst[u] = r * CV_GRID_BYTES + gy * gw + 16 + 16 * xc;
                            if (img < p.n && yy >= 0 && yy < p.h)
                                val[u] = *reinterpret_cast<const uint4*>(p.exps_x + (((int64_t)img * p.h + yy) << lw) + 16 * xc);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u)
                        if (dst[u] >= 0) *reinterpret_cast<uint4*>(grid + dst[u]) = val[u];
                }
                __syncwarp();
                for (int tap = 0; ok && tap < p.taps; ++tap) {
                    const int dy = tap / p.kw, dx = tap - dy * p.kw;
                    // this lane's 4 rows of every row tile and its N_TILE / 32 columns
                    int ea[RT][4];
                    int a_lo = 127, a_hi = -128;
#pragma unroll
                    for (int r = 0; r < RT; ++r)
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int row = 4 * lane + k;
                            const int yl = row >> lw, xl = row & (p.w - 1);
                            const int e = grid[r * CV_GRID_BYTES + (yl + dy) * gw + 16 + xl + dx - p.pad];
                            ea[r][k] = e;
                            if (e != 127) { a_lo = min(a_lo, e); a_hi = max(a_hi, e); }
                        }
                    constexpr int CPL = N_TILE / 32;
                    int eb[CPL];
                    int b_lo = 127, b_hi = -128;
#pragma unroll
                    for (int k = 0; k < CPL; ++k) {
                        eb[k] = wexp[tap * N_TILE + CPL * lane + k];
                        b_lo = min(b_lo, eb[k]); b_hi = max(b_hi, eb[k]);
                    }
                    a_lo = __reduce_min_sync(0xffffffffu, a_lo); a_hi = __reduce_max_sync(0xffffffffu, a_hi);
                    b_lo = __reduce_min_sync(0xffffffffu, b_lo); b_hi = __reduce_max_sync(0xffffffffu, b_hi);
                    if (a_lo > a_hi) a_lo = a_hi = 0;                 // every position of the tap lies outside the image
                    // split of the scale 2^(sA + sB) = 2^(sA + c) * 2^(sB + 149 - c): every factor and every
                    // P * 2^(sA + c - 149) a normal binary32 number (see gemm_tc2.cu)
                    const int c_lo = max(23 - a_lo, 22 + b_hi), c_hi = min(127 - a_hi, 275 + b_lo);
                    out_of_range |= c_lo > c_hi;
                    const int c = min(max(CV_SHIFT, c_lo), c_hi);
                    if (!mbar_wait_warp(tfull_bar + 8 * b, bph ^ 1, abort_flag, p.status, 421)) { ok = false; break; }
                    uint32_t* tb = tables + slot * G::SLOT_WORDS;
#pragma unroll
                    for (int k = 0; k < CPL; ++k) tb[CPL * lane + k] = cv_scale_bits(eb[k], 149 - c);
#pragma unroll
                    for (int r = 0; r < RT; ++r)
#pragma unroll
                        for (int k = 0; k < 4; ++k)      // outside the image the mantissas are zero: any finite scale gives +0
                            tb[N_TILE + r * TILE_M + 4 * lane + k] = cv_scale_bits(ea[r][k] == 127 ? a_lo : ea[r][k], c);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tfull_bar + 8 * b);
                    cv_ring_next<CV_BUFS>(b, bph);
                    slot = (slot + 1) & (CV_TSLOTS - 1);
                }
                __syncwarp();
            }
            if (out_of_range) atomicCAS(p.status, 0, STATUS_EXPONENT_RANGE);
        }
    } else {
        // ------------------------------------------------------------------ rescale warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(CV_REGS_RESCALE));
        const int rwarp = warp - CV_CONTROL_WARPS;
        const int quarter = warp & 3, half = rwarp >> 2;       // tensor-memory lanes follow warp % 4; half = column half
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + half * HALF;
        constexpr int CH = 8, NCH = HALF / CH;                 // chunks per row tile
        uint64_t acc2[RT][HALF / 2];
        if (lane == 0)
            for (int b = 0; b < CV_BUFS; ++b) mbar_arrive(tempty_bar + 8 * b);     // every buffer starts out free
        uint32_t b = 0, bph = 0, slot = 0;
        bool ok = true;
        for (int st = blockIdx.x; ok && st < p.super_tiles; st += gridDim.x) {
#pragma unroll
            for (int r = 0; r < RT; ++r)
#pragma unroll
                for (int k = 0; k < HALF / 2; ++k) acc2[r][k] = 0ull;
            for (int tap = 0; tap < p.taps; ++tap) {
                const uint32_t taddr = lane_addr + b * CV_COLS;
                uint32_t v[2][CH];
                {   // polled first: a warp that try_wait has put to sleep wakes up late
                    bool hit = false;
                    for (int i = 0; i < 2048 && !hit; ++i) hit = cv_test_wait(tfull_bar + 8 * b, bph);
                    if (!__all_sync(0xffffffffu, hit) && !mbar_wait_warp(tfull_bar + 8 * b, bph, abort_flag, p.status, 321)) { ok = false; break; }
                }
                tc_fence_after();
                tc_ld8(taddr, v[0]);
                const uint32_t* tab = tables + slot * G::SLOT_WORDS + half * HALF;
                const uint32_t* rowtab = tables + slot * G::SLOT_WORDS + N_TILE + row;
#pragma unroll
                for (int r = 0; r < RT; ++r) {
                    // x = (OFFSET + P) * 2^-149;  t = fma(x, 2^(sA + c), -OFFSET * 2^(sA + c - 149)) = P * 2^(sA + c - 149)
                    // (exact);  acc = fma(t, 2^(sB + 149 - c), acc)
                    const float sa_f = __uint_as_float(rowtab[r * TILE_M]);
                    const float ca_f = -__uint_as_float((uint32_t)CV_OFFSET) * sa_f;
                    const uint64_t sa2 = pack2(__float_as_uint(sa_f), __float_as_uint(sa_f));
                    const uint64_t ca2 = pack2(__float_as_uint(ca_f), __float_as_uint(ca_f));
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch) {
                        constexpr int TOTAL = RT * NCH;
                        const int idx = r * NCH + ch;                      // compile-time after unrolling
                        uint4 sbq[CH / 4];
#pragma unroll
                        for (int q = 0; q < CH; q += 4) sbq[q / 4] = *reinterpret_cast<const uint4*>(tab + ch * CH + q);
                        tc_wait_ld();
                        if (idx + 1 < TOTAL) {
                            const int r2 = (idx + 1) / NCH, ch2 = (idx + 1) - r2 * NCH;
                            tc_ld8(taddr + r2 * N_TILE + ch2 * CH, v[(idx + 1) & 1]);
                        } else {
                            // the whole buffer is in registers: hand it back before the last chunk's arithmetic
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(tempty_bar + 8 * b);
                        }
                        const uint32_t(&x)[CH] = v[idx & 1];
#pragma unroll
                        for (int q = 0; q < CH; q += 4) {
                            const uint4 sb = sbq[q / 4];
                            const uint64_t t01 = ffma2(pack2(x[q], x[q + 1]), sa2, ca2);
                            const uint64_t t23 = ffma2(pack2(x[q + 2], x[q + 3]), sa2, ca2);
                            acc2[r][(ch * CH + q) / 2] = ffma2(t01, pack2(sb.x, sb.y), acc2[r][(ch * CH + q) / 2]);
                            acc2[r][(ch * CH + q) / 2 + 1] = ffma2(t23, pack2(sb.z, sb.w), acc2[r][(ch * CH + q) / 2 + 1]);
                        }
                    }
                }
                cv_ring_next<CV_BUFS>(b, bph);
                slot = (slot + 1) & (CV_TSLOTS - 1);
            }
            if (!ok) break;
            // ---- store this warp's columns of every row tile: each lane owns an output pixel
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                const int rt = st * RT + r;
                if (rt < p.row_tiles) {
                    float* rowp = p.Y + ((int64_t)rt * TILE_M + row) * p.ldy + half * HALF;
                    const bool wide = (p.ldy & 7) == 0 && (reinterpret_cast<uintptr_t>(p.Y) & 31) == 0;
#pragma unroll
                    for (int col = 0; col < HALF; col += 4) {
                        const int gj = half * HALF + col;
                        if (wide && (col & 7) == 0 && gj + 7 < p.filters) {
                            st_global_256(rowp + col, acc2[r][col / 2], acc2[r][col / 2 + 1], acc2[r][col / 2 + 2], acc2[r][col / 2 + 3]);
                        } else if (wide && (col & 7) == 4 && gj + 3 < p.filters) {
                            // second half of a sector written above
                        } else if (gj + 3 < p.filters) {
                            *reinterpret_cast<ulonglong2*>(rowp + col) = make_ulonglong2(acc2[r][col / 2], acc2[r][col / 2 + 1]);
                        } else {
                            float e4[4];
                            unpack2(acc2[r][col / 2], e4[0], e4[1]);
                            unpack2(acc2[r][col / 2 + 1], e4[2], e4[3]);
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (gj + e < p.filters) rowp[col + e] = e4[e];
                        }
                    }
                }
            }
        }
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (warp == CV_MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// 4-D byte tensor of the packed pixels: [n][h][w][pitch bytes], of which the first c bytes of every pixel
// are copied; box = c bytes x w pixels x R image rows x 1 image.
int make_map_pixels(CUtensorMap* m, const void* ptr, int c, uint64_t pitch, int w, int h, int n, int rows_per_tile) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return HBFP_ERR_CUDA;
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {pitch, pitch * (uint64_t)w, pitch * (uint64_t)w * (uint64_t)h};
    cuuint32_t box[4] = {(cuuint32_t)c, (cuuint32_t)w, (cuuint32_t)rows_per_tile, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, c == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HBFP_OK : HBFP_ERR_CUDA;
}

// 2-D byte tensor of the packed filters [filters][kst]; box = c bytes of one tap x N_TILE filters.
int make_map_filters(CUtensorMap* m, const void* ptr, uint64_t kst, uint64_t rows, int c, int n_tile) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return HBFP_ERR_CUDA;
    cuuint64_t dims[2] = {kst, rows};
    cuuint64_t strides[1] = {kst};
    cuuint32_t box[2] = {(cuuint32_t)c, (cuuint32_t)n_tile};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, c == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HBFP_OK : HBFP_ERR_CUDA;
}

template <int C, int N_TILE>
int launch_conv_cfg(const CUtensorMap& mX, const CUtensorMap& mW, const ConvProblem& p, cudaStream_t st) {
    using G = ConvCfg<C, N_TILE>;
    static bool attr_set[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return HBFP_ERR_CUDA;
    if (!attr_set[dev]) {
        HBFP_CUDA_OK(cudaFuncSetAttribute(conv_fwd_kernel<C, N_TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM));
        attr_set[dev] = true;
    }
    const int grid = p.super_tiles < sm_count() ? p.super_tiles : sm_count();
    conv_fwd_kernel<C, N_TILE><<<grid, CV_THREADS, G::SMEM, st>>>(mX, mW, p);
    return launch_status();
}

}  // namespace

// x: packed pixels (rows = n*h*w, k = c, one block); wt: packed filters (rows = filters, k = kh*kw*c, blocks of c).
int launch_conv_forward(const Packed& x, const Packed& wt, int64_t n, int64_t h, int64_t w, int64_t c, int kh, int kw,
                        int pad, int64_t filters, float* Y, int64_t ldy, cudaStream_t st) {
    // what the kernel covers; everything else is the caller's gather + GEMM path
    if (c != 64 && c != 128) return HBFP_ERR_UNSUPPORTED;
    if (x.L.planes != 1 || wt.L.planes != 1 || x.L.bp != c || wt.L.bp != c || x.L.nkb != 1) return HBFP_ERR_UNSUPPORTED;
    if (kh * kw > CV_MAX_TAPS || pad > CV_MAX_PAD || 2 * pad != kh - 1 || 2 * pad != kw - 1) return HBFP_ERR_UNSUPPORTED;
    if (w < 16 || w > 128 || (128 % w) != 0 || (h % (128 / w)) != 0) return HBFP_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(x.exps) & 15) return HBFP_ERR_UNSUPPORTED;
    if (filters < 1 || filters > 256 || n * h * w > (1ll << 30)) return HBFP_ERR_UNSUPPORTED;
    const int64_t qa = (1ll << (x.mant_bits - 1)) - 1, qb = (1ll << (wt.mant_bits - 1)) - 1;
    if (qa * qb * c >= CV_OFFSET) return HBFP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(Y) & 15) || (ldy % 4) != 0) return HBFP_ERR_UNSUPPORTED;
    const int n_tile = filters <= 64 ? 64 : filters <= 128 ? 128 : 256;
    ConvProblem p{};
    p.n = (int)n; p.h = (int)h; p.w = (int)w; p.kh = kh; p.kw = kw; p.pad = pad; p.taps = kh * kw;
    p.rows_per_tile = 128 / (int)w;
    p.tiles_per_image = (int)h / p.rows_per_tile;
    p.row_tiles = (int)n * p.tiles_per_image;
    const int rt = CV_COLS / n_tile;
    p.super_tiles = (p.row_tiles + rt - 1) / rt;
    p.filters = (int)filters;
    p.exps_x = x.exps;
    p.exps_w = wt.exps;
    p.rs_w = wt.L.rs;
    p.Y = Y;
    p.ldy = ldy;
    p.status = device_status_word();
    if (!p.status) return HBFP_ERR_CUDA;
    if (p.super_tiles == 0) return HBFP_OK;
    CUtensorMap mX, mW;
    int rc = make_map_pixels(&mX, x.mant, (int)c, (uint64_t)x.L.kst, (int)w, (int)h, (int)n, p.rows_per_tile);
    if (rc) return rc;
    rc = make_map_filters(&mW, wt.mant, (uint64_t)wt.L.kst, (uint64_t)wt.L.rows, (int)c, n_tile);
    if (rc) return rc;
    if (c == 64) {
        if (n_tile == 64) return launch_conv_cfg<64, 64>(mX, mW, p, st);
        if (n_tile == 128) return launch_conv_cfg<64, 128>(mX, mW, p, st);
        return launch_conv_cfg<64, 256>(mX, mW, p, st);
    }
    if (n_tile == 64) return launch_conv_cfg<128, 64>(mX, mW, p, st);
    if (n_tile == 128) return launch_conv_cfg<128, 128>(mX, mW, p, st);
    return launch_conv_cfg<128, 256>(mX, mW, p, st);
}

}  // namespace hbfp
