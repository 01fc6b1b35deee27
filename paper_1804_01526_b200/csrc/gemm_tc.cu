// Tensor-core BFP GEMM for sm_100a: TMA -> shared memory -> tcgen05.mma kind::i8 -> int32 in
// tensor memory -> per-block rescale into FP32 registers (Eq. 2 per block, blocks accumulated in
// floating point, Sec. 4).
//
// One persistent CTA per SM, 12 warps (the control warps come first: the issue logic favours low
// warp ids, and a starved MMA issuer stalls everything):
//   warp 0     TMA producer: mantissa tiles (128B-swizzled, K-major) and exponent slices
//   warp 1     MMA issuer (one thread) and owner of the tensor-memory allocation
//   warp 2     scale-table builder: turns the int8 exponent slices of each block into 2^sA / 2^sB
//   warps 4-11 rescale: tcgen05.ld the int32 block sums, scale by 2^(sA+sB), accumulate in FP32
//              registers (128 rows x N_TILE columns per tile), store C
// A stage is 128 bytes of K for every row of the A (128 rows) and B (N_TILE rows) tiles, i.e. four
// K=32 MMA steps; a K-block of bp bytes is bp/32 consecutive steps accumulated into one fresh
// int32 accumulator group in tensor memory. Groups form a ring, so the MMA of the next block
// overlaps the rescale of the previous one. 12-bit mantissas (two int8 planes, q = 16 hi + lo): the
// hi and lo planes of the B tile lie back to back in a stage, so each A plane is multiplied by both
// in one MMA of width 2 N_TILE, the two results overlapping in the middle: three accumulators
// (hi*hi | hi*lo + lo*hi | lo*lo) that the rescale warps combine exactly in int32.
//
// Fast rescale (8-bit mantissas, blocks up to 256, so |P| < 2^22): integer-to-float conversion
// runs on a slow pipe and an integer add per element would land on the FP32 pipe, so the
// accumulator groups are armed with the integer 0x4B400000 and every MMA accumulates on top of it:
// what tcgen05.ld returns, read as binary32, is exactly 1.5*2^23 + P. Then
//   t   = fma(v, 2^sA, -1.5*2^23 * 2^sA)   = P * 2^sA          (exact)
//   acc = fma(t, 2^sB, acc)                = acc + P*2^(sA+sB) (one rounding, as the definition)
// both as packed two-wide FP32 FMAs; after reading a chunk the warp stores the bias back.
// 12-bit mantissas with blocks below 256 take the same route with three armed parts per group: one FMA per
// part removes the bias and applies the part's weight (256, 16, 1) and 2^sA exactly, two additions form
// float(P) * 2^sA with the single rounding of the definition, one FMA accumulates it times 2^sB.
// Longer blocks clear the accumulator with the first MMA of a block and convert with cvt.rn.f32.s32.
// The MMA thread and the rescale warps wait for their barriers with a few looks, then naps of at most 64 ns
// (a suspended wait of unbounded length wakes late; a spinning one takes issue slots from the rescale warps).
//
// Every wait on an mbarrier is bounded: when it expires the CTA records a code in the device
// status word, raises a shared abort flag, drains its own copies and MMAs (bounded again),
// releases tensor memory and returns.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace hbfp {
namespace {

constexpr int RESCALE_WARPS = 8;                   // two per sub-partition
constexpr int COL_GROUPS = RESCALE_WARPS / 4;      // warps sharing a lane quarter split the columns
// The control warps take the lowest warp ids: the issue logic favours them over the rescale
// warps of the same sub-partition, and a starved MMA issuer stalls the whole pipeline.
constexpr int CONTROL_WARPS = 4;      // one warpgroup: producer, MMA issuer, table builder, one spare
constexpr int PRODUCER_WARP = 0;
constexpr int MMA_WARP = 1;
constexpr int TABLE_WARP = 2;
constexpr int THREADS = 32 * (CONTROL_WARPS + RESCALE_WARPS);
// setmaxnreg totals must never exceed what the launch allocated (384 threads x 168 registers): a
// request the register file cannot satisfy blocks forever.
constexpr int REGS_RESCALE = 216, REGS_CONTROL = 72;
static_assert(128 * REGS_CONTROL + 32 * RESCALE_WARPS * REGS_RESCALE <= 384 * 168, "register split");

// TSTORE: the output tile leaves through shared memory and TMA stores (one 32 x 32 FP32 box per rescale warp
// and 32 columns, double-buffered) instead of per-lane stores from registers; takes 64 KB from the stages.
template <int N_TILE, int PLANES, bool TSTORE = false>
struct Cfg {
    // accumulator parts per group; two planes: [hi.hi | hi.lo + lo.hi | lo.lo], each N_TILE columns
    static constexpr int PARTS = PLANES == 1 ? 1 : 3;
    static constexpr int GROUPS_RAW = TMEM_COLS / (N_TILE * PARTS);
    static constexpr int GROUPS = GROUPS_RAW > 4 ? 4 : GROUPS_RAW;
    static constexpr int A_BYTES = TILE_M * STAGE_K;              // per plane
    static constexpr int B_BYTES = N_TILE * STAGE_K;              // per plane
    static constexpr int MANT_STAGE = PLANES * (A_BYTES + B_BYTES);
    static constexpr int EXP_A = 4 * TILE_M, EXP_B = 4 * N_TILE;
    static constexpr int EXP_STAGE = EXP_A + EXP_B;
    // scale tables: a ring of 2 * GROUPS blocks, each [N_TILE column scales][128 row scales], 32-bit
    static constexpr int TABLE_SLOTS = 2 * GROUPS;
    static constexpr int TABLE_SLOT_WORDS = N_TILE + TILE_M;
    static constexpr int TABLE_BYTES = 4 * TABLE_SLOTS * TABLE_SLOT_WORDS;
    static constexpr int OUT_BUF = 32 * 32 * 4;                    // one 32-row x 32-column FP32 box
    static constexpr int OUT_BYTES = TSTORE ? RESCALE_WARPS * 2 * OUT_BUF : 0;
    static constexpr int STAGES_RAW = (232448 - 2048 - TABLE_BYTES - OUT_BYTES - (TSTORE ? 1024 : 0)) / (MANT_STAGE + EXP_STAGE);
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr int SMEM = 1024 /*align slack*/ + STAGES * (MANT_STAGE + EXP_STAGE) + (TSTORE ? 1024 : 0) + OUT_BYTES + TABLE_BYTES + 1024 /*barriers*/;
    static constexpr uint32_t TX_BYTES = MANT_STAGE + EXP_STAGE;
    static_assert(GROUPS >= 2, "need two accumulator groups to overlap MMA and rescale");
    static_assert(STAGES >= 3, "pipeline too shallow");
};

// ------------------------------------------------------------------------------ work decomposition

struct Problem {
    int64_t M, N;
    int64_t nkb;            // K-blocks
    int bp;                 // padded block bytes: 32, 64, 128, or a multiple of 128
    int tiles_m, tiles_n;
    int splits;
    int64_t kb_per_split;
    float* C;
    int64_t ldc;
    float* partial;         // [splits][M][ldp] when splits > 1
    int64_t ldp;
    int32_t* P;             // optional dump of block sums [M][N][nkb]
    int32_t* status;
};

struct Work {
    int m0, nt, split;
    int kb0, nblk;          // first K-block and number of K-blocks of this item
};

// 32-bit arithmetic only (this runs in warps that have given most of their registers away);
// returned by value so that the fields stay in registers.
__device__ __forceinline__ Work get_work(const Problem& p, int w) {
    Work out;
    const int tiles = p.tiles_m * p.tiles_n;
    const int split = w / tiles;
    const int t = w - split * tiles;
    // groups of 16 tile rows share their B panels in L2 while a group sweeps across N
    const int G = 16;
    const int per_group = G * p.tiles_n;
    const int group = t / per_group;
    const int first_m = group * G;
    const int gsize = min(G, p.tiles_m - first_m);
    const int within = t - group * per_group;
    const int nt = within / gsize;
    out.m0 = (first_m + (within - nt * gsize)) * TILE_M;
    out.nt = nt;
    out.split = split;
    out.kb0 = split * (int)p.kb_per_split;
    out.nblk = min((int)p.nkb, out.kb0 + (int)p.kb_per_split) - out.kb0;
    return out;
}

// How the K-blocks of an item map onto 128-byte stages: blocks of 32 or 64 bytes share a stage
// (bps of them, spb MMA steps each); longer blocks span spk whole stages.
struct Shape {
    int lb, bps, spb, spk;  // log2(bps), blocks per stage, MMA steps per block inside a stage, stages per block
    bool lng;
};
__device__ __forceinline__ Shape make_shape(int bp) {
    Shape s;
    s.lng = bp >= STAGE_K;
    s.lb = bp == 32 ? 2 : bp == 64 ? 1 : 0;
    s.bps = 1 << s.lb;
    s.spb = 4 >> s.lb;
    s.spk = s.lng ? bp / STAGE_K : 1;       // (once per kernel)
    return s;
}
__device__ __forceinline__ int stages_of(const Shape& sh, int nblk) {
    return sh.lng ? nblk * sh.spk : (nblk + sh.bps - 1) >> sh.lb;
}

// Advances a ring position (stage, accumulator group or table slot) and its phase bit.
template <int N>
__device__ __forceinline__ void ring_next(uint32_t& i, uint32_t& ph) {
    if (++i == N) { i = 0; ph ^= 1u; }
}

// Non-blocking look at a barrier phase.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

__device__ __forceinline__ bool mbar_try_wait_ns(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// A few looks at the barrier, then naps of at most 64 ns (no issue slots taken from the arithmetic warps), then the
// bounded wait.
__device__ __forceinline__ bool mbar_wait_quick(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int code) {
    for (int i = 0; i < 32; ++i)
        if (mbar_test_wait(bar, parity)) return true;
    for (int i = 0; i < 1024; ++i)
        if (mbar_try_wait_ns(bar, parity, 64u)) return true;
    return mbar_wait(bar, parity, abort_flag, status, code);
}

// 2^e as binary32 bits (MAGIC) or the exponent shifted into the exponent field, e = signed byte i of
// a packed word of exponents.
__device__ __forceinline__ uint32_t exp_to_field(uint32_t packed, int i, int add) {
    const int e = (int)(int8_t)(packed >> (8 * i));
    return (uint32_t)(e + add) << 23;
}

// ------------------------------------------------------------------------------ MMA issuer

struct MmaArgs {
    uint32_t full_bar, empty_bar, tfull_bar, tempty_bar, done_bar, mant_base, tmem_base;
    int total_work;
    volatile int* abort_flag;
};

// The loop of the single MMA-issuing thread. LNG: blocks of 128 bytes or more (one block step set per
// stage, SPB = 4); otherwise 128 / (32 SPB) blocks of SPB steps share a stage.
template <int N_TILE, int PLANES, bool MAGIC, bool LNG, int SPB, bool TSTORE>
__device__ __forceinline__ void mma_issue_loop(const Problem& p, const Shape& sh, const MmaArgs& a) {
    using C = Cfg<N_TILE, PLANES, TSTORE>;      // the kernel's configuration: same ring sizes
    constexpr int STAGES = C::STAGES, GROUPS = C::GROUPS, PARTS = C::PARTS;
    constexpr int BPS = LNG ? 1 : 4 / SPB;
    // Two planes: the hi and lo planes of B lie back to back in a stage, so one MMA of twice the width
    // (idesc2) multiplies an A plane by both: A_hi gives [hi.hi | hi.lo] from column 0 of the group,
    // A_lo gives [lo.hi | lo.lo] from column N_TILE, so that the two cross terms add up in the middle
    // part. Only the first step of a block, which must overwrite hi.hi and lo.lo but accumulate the
    // second cross term, takes three MMAs.
    constexpr uint32_t idesc = idesc_i8<N_TILE>(), idesc2 = idesc_i8<2 * N_TILE>();
    uint32_t s = 0, ph = 0, g = 0, gph = 0, it = 0, blk = 0;
    // The barriers the next MMAs will need are polled (without blocking) just before the last MMA
    // step of a block or stage is issued, while earlier MMAs still occupy the tensor pipe; a
    // barrier found complete then is not waited on again.
    bool pre_full = false, pre_tempty = false;
    bool ok = true;
    for (int wi = blockIdx.x; ok && wi < a.total_work; wi += gridDim.x) {
        const Work w = get_work(p, wi);
        const int nst = stages_of(sh, w.nblk);
        int left = w.nblk, sib = 0;
        for (int si = 0; ok && si < nst; ++si, ++it) {
            if (pre_full) pre_full = false;
            else if (!mbar_wait_quick(a.full_bar + 8 * s, ph, a.abort_flag, p.status, 201)) { ok = false; break; }
            tc_fence_after();
            const uint32_t ms = a.mant_base + s * C::MANT_STAGE;
            const uint64_t a_hi = smem_desc_sw128(ms), b_hi = smem_desc_sw128(ms + PLANES * C::A_BYTES);
            const uint64_t a_lo = smem_desc_sw128(ms + C::A_BYTES);
            const uint64_t b_lo = smem_desc_sw128(ms + 2 * C::A_BYTES + C::B_BYTES);
            const int nb = LNG ? 1 : min(BPS, left);          // blocks that have steps in this stage
#pragma unroll
            for (int jb = 0; jb < BPS; ++jb) {
                if (jb < nb) {
                    const bool first = !LNG || sib == 0;              // the block starts in this stage
                    const bool last = !LNG || sib == sh.spk - 1;      // ... and ends in it
                    if (first) {
                        // the group was read (and, on the biased path, re-armed) by all rescale warps
                        if (pre_tempty) pre_tempty = false;
                        else if (!mbar_wait_quick(a.tempty_bar + 8 * g, gph, a.abort_flag, p.status, 202)) { ok = false; break; }
                        tc_fence_after();
                    }
                    const uint32_t d = a.tmem_base + g * PARTS * N_TILE;
#pragma unroll
                    for (int q = 0; q < SPB; ++q) {
                        if (q == SPB - 1) {
                            // look ahead while the tensor pipe still has the earlier MMAs to run
                            if (last) {
                                uint32_t g2 = g, gph2 = gph;
                                ring_next<GROUPS>(g2, gph2);
                                pre_tempty = mbar_test_wait(a.tempty_bar + 8 * g2, gph2);
                            }
                            if (jb == nb - 1) {
                                uint32_t s2 = s, ph2 = ph;
                                ring_next<STAGES>(s2, ph2);
                                pre_full = mbar_test_wait(a.full_bar + 8 * s2, ph2);
                            }
                        }
                        const uint64_t ko = (uint64_t)(2 * (jb * SPB + q));      // 32 bytes per step, in 16-byte units
                        // biased path: always accumulate on top of the bias; else the first step of a block overwrites
                        const uint32_t acc = MAGIC ? 1u : (uint32_t)!(first && q == 0);
                        if (PLANES == 1) {
                            tc_mma_i8(d, a_hi + ko, b_hi + ko, idesc, acc);
                        } else {
                            if (acc == 0u) {
                                tc_mma_i8(d + N_TILE, a_lo + ko, b_hi + ko, idesc2, 0u);
                                tc_mma_i8(d, a_hi + ko, b_hi + ko, idesc, 0u);
                                tc_mma_i8(d + N_TILE, a_hi + ko, b_lo + ko, idesc, 1u);
                            } else {
                                tc_mma_i8(d, a_hi + ko, b_hi + ko, idesc2, 1u);
                                tc_mma_i8(d + N_TILE, a_lo + ko, b_hi + ko, idesc2, 1u);
                            }
                        }
                    }
                    if (last) {
                        tc_commit(a.tfull_bar + 8 * g);
                        ring_next<GROUPS>(g, gph);
                        ++blk;
                        sib = 0;
                    } else {
                        ++sib;
                    }
                }
            }
            left -= nb;
            tc_commit(a.empty_bar + 8 * s);        // the stage is free once these MMAs have read it
            ring_next<STAGES>(s, ph);
        }
    }
    tc_commit(a.done_bar);
    mbar_wait(a.done_bar, 0, a.abort_flag, p.status, 203, false);
}

// ------------------------------------------------------------------------------ kernel

template <int N_TILE, int PLANES, bool MAGIC, bool DUMP, bool TSTORE>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapA1,
               const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
               const __grid_constant__ CUtensorMap mapEA, const __grid_constant__ CUtensorMap mapEB,
               const __grid_constant__ CUtensorMap mapC, const Problem p) {
    using C = Cfg<N_TILE, PLANES, TSTORE>;
    constexpr int STAGES = C::STAGES, GROUPS = C::GROUPS, PARTS = C::PARTS, TSLOTS = C::TABLE_SLOTS;
    constexpr int COLS_PER_WARP = N_TILE / COL_GROUPS;  // warps that share a lane quarter split the columns

    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t mant_base = base;                                        // STAGES x MANT_STAGE, 1024-aligned
    const uint32_t exp_base = mant_base + STAGES * C::MANT_STAGE;           // STAGES x EXP_STAGE
    const uint32_t out_off = (STAGES * (C::MANT_STAGE + C::EXP_STAGE) + 1023u) & ~1023u;   // output boxes (TSTORE), 1024-aligned
    const uint32_t table_off = out_off + C::OUT_BYTES;
    uint32_t* tables = reinterpret_cast<uint32_t*>(base_ptr + table_off);   // [slot][N_TILE column scales | 128 row scales]
    const uint32_t bar_off = table_off + C::TABLE_BYTES;
    const uint32_t bars = base + bar_off;
    const uint32_t full_bar = bars;                          // stage landed (mantissa tiles and exponent slices)
    const uint32_t empty_bar = bars + 8 * STAGES;            // stage consumed (MMA commit + table warp)
    const uint32_t tfull_bar = bars + 16 * STAGES;           // block sums complete (MMA commit) and scale table written
    const uint32_t tempty_bar = tfull_bar + 8 * GROUPS;      // group read (and re-armed) by every rescale warp
    const uint32_t done_bar = tempty_bar + 8 * GROUPS;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + bar_off + 16 * STAGES + 16 * GROUPS + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 2);                 // MMA commit + table warp
        }
        for (int g = 0; g < GROUPS; ++g) {
            mbar_init(tfull_bar + 8 * g, 2);                 // MMA commit + table warp
            mbar_init(tempty_bar + 8 * g, RESCALE_WARPS);
        }
        mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const Shape sh = make_shape(p.bp);
    const int total_work = p.tiles_m * p.tiles_n * p.splits;

    if (warp < CONTROL_WARPS) {
        // the control warpgroup hands most of its registers to the rescale warps
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_CONTROL));
        if (warp == PRODUCER_WARP) {
            // -------------------------------------------------------------- TMA producer
            if (lane == 0) {
                uint32_t s = 0, ph = 0, it = 0;
                bool ok = true;
                for (int wi = blockIdx.x; ok && wi < total_work; wi += gridDim.x) {
                    const Work w = get_work(p, wi);
                    const int n0 = w.nt * N_TILE;
                    const int nst = stages_of(sh, w.nblk);
                    int kb = w.kb0, sib = 0;              // first block touched by the stage; stage inside a long block
                    int kbyte = w.kb0 * p.bp;
                    for (int si = 0; si < nst; ++si, kbyte += STAGE_K, ++it) {
                        if (!mbar_wait(empty_bar + 8 * s, ph ^ 1, abort_flag, p.status, 101)) { ok = false; break; }
                        const uint32_t fb = full_bar + 8 * s;
                        mbar_expect_tx(fb, C::TX_BYTES);
                        const uint32_t ms = mant_base + s * C::MANT_STAGE;
                        // A panels are re-used by every column tile of a group of 16 tile rows: ask L2 to keep
                        // them while the B panels stream past (marking B evict-first doubled the DRAM reads:
                        // the 16 CTAs that share a B panel do not read it at the same instant).
                        tma_load_2d_hint(ms, &mapA0, kbyte, w.m0, fb, L2_EVICT_LAST);
                        tma_load_2d(ms + PLANES * C::A_BYTES, &mapB0, kbyte, n0, fb);
                        if (PLANES == 2) {
                            tma_load_2d_hint(ms + C::A_BYTES, &mapA1, kbyte, w.m0, fb, L2_EVICT_LAST);
                            tma_load_2d(ms + 2 * C::A_BYTES + C::B_BYTES, &mapB1, kbyte, n0, fb);
                        }
                        const uint32_t es = exp_base + s * C::EXP_STAGE;
                        tma_load_2d(es, &mapEA, w.m0, kb, fb);
                        tma_load_2d(es + C::EXP_A, &mapEB, n0, kb, fb);
                        if (sh.lng) { if (++sib == sh.spk) { sib = 0; ++kb; } } else { kb += sh.bps; }
                        ring_next<STAGES>(s, ph);
                    }
                }
                // Drain: every issued copy must have landed before the CTA may exit. In a normal run
                // the consumers already waited for all of them, so these return at once.
                const uint32_t back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                for (uint32_t k = 0; k < back; ++k) {
                    if (s == 0) { s = STAGES - 1; ph ^= 1u; } else { --s; }
                    mbar_wait(full_bar + 8 * s, ph, abort_flag, p.status, 102, false);
                }
            }
        } else if (warp == MMA_WARP) {
            // -------------------------------------------------------------- MMA issuer
            if (lane == 0) {
                const MmaArgs ma{full_bar, empty_bar, tfull_bar, tempty_bar, done_bar, mant_base, tmem_base, total_work, abort_flag};
                if (sh.lng) mma_issue_loop<N_TILE, PLANES, MAGIC, true, 4, TSTORE>(p, sh, ma);
                else if (sh.spb == 2) mma_issue_loop<N_TILE, PLANES, MAGIC, false, 2, TSTORE>(p, sh, ma);
                else mma_issue_loop<N_TILE, PLANES, MAGIC, false, 1, TSTORE>(p, sh, ma);
            }
        } else if (warp == TABLE_WARP) {
            // -------------------------------------------------------------- scale-table builder
            // The table of block b goes to slot b % (2 GROUPS) and its arrival counts on tfull[b % GROUPS].
            // It is written once the previous phase of that barrier (block b - GROUPS) is complete: the
            // MMAs of that block were issued only after every rescale warp had finished block
            // b - 2 GROUPS, the last reader of the slot, and the barrier is back in the phase that the
            // arrival for b belongs to.
            uint32_t s = 0, ph = 0, g = 0, gph = 0, slot = 0, it = 0, blk = 0;
            bool ok = true, out_of_range = false;
            for (int wi = blockIdx.x; ok && wi < total_work; wi += gridDim.x) {
                const Work w = get_work(p, wi);
                const int nst = stages_of(sh, w.nblk);
                int left = w.nblk, sib = 0;
                for (int si = 0; ok && si < nst; ++si, ++it) {
                    if (!mbar_wait_warp(full_bar + 8 * s, ph, abort_flag, p.status, 401)) { ok = false; break; }
                    const unsigned char* eA = base_ptr + (exp_base - base) + s * C::EXP_STAGE;
                    const unsigned char* eB = eA + C::EXP_A;
                    const int nb = sh.lng ? (sib == 0 ? 1 : 0) : min(sh.bps, left);   // blocks that start in this stage
                    for (int jb = 0; jb < nb; ++jb) {
                        // this lane's N_TILE / 32 column exponents and 4 row exponents of the block
                        constexpr int CPL = N_TILE / 32;      // 8, 4 or 2 column bytes per lane
                        uint32_t cw[2] = {0u, 0u};
                        if (CPL == 8) { const uint2 t = *reinterpret_cast<const uint2*>(eB + jb * N_TILE + 8 * lane); cw[0] = t.x; cw[1] = t.y; }
                        else if (CPL == 4) cw[0] = *reinterpret_cast<const uint32_t*>(eB + jb * N_TILE + 4 * lane);
                        else cw[0] = *reinterpret_cast<const uint16_t*>(eB + jb * N_TILE + 2 * lane);
                        const uint32_t ra = *reinterpret_cast<const uint32_t*>(eA + jb * TILE_M + 4 * lane);
                        // the biased path forms 1.5 * 2^23 * 2^sA: finite up to sA = 103; beyond it the result
                        // would be wrong, which is reported instead
                        // (two planes: 1.5 * 2^31 * 2^sA and 2^29 * 2^sA, finite up to sA = 96)
                        if (MAGIC) out_of_range |= __vmaxs4(ra, PLANES == 1 ? 0x67676767u : 0x60606060u) != (PLANES == 1 ? 0x67676767u : 0x60606060u);
                        uint32_t cs[CPL];
#pragma unroll
                        for (int i = 0; i < CPL; ++i) cs[i] = exp_to_field(cw[i >> 2], i & 3, MAGIC ? 127 : 0);
                        uint4 r0;
                        r0.x = exp_to_field(ra, 0, 127); r0.y = exp_to_field(ra, 1, 127);
                        r0.z = exp_to_field(ra, 2, 127); r0.w = exp_to_field(ra, 3, 127);
                        if (!mbar_wait_warp(tfull_bar + 8 * g, gph ^ 1, abort_flag, p.status, 402)) { ok = false; break; }
                        uint32_t* tb = tables + slot * C::TABLE_SLOT_WORDS;
                        if (CPL == 8) {
                            *reinterpret_cast<uint4*>(tb + 8 * lane) = make_uint4(cs[0], cs[1], cs[2], cs[3]);
                            *reinterpret_cast<uint4*>(tb + 8 * lane + 4) = make_uint4(cs[4 % CPL], cs[5 % CPL], cs[6 % CPL], cs[7 % CPL]);
                        } else if (CPL == 4) {
                            *reinterpret_cast<uint4*>(tb + 4 * lane) = make_uint4(cs[0], cs[1], cs[2 % CPL], cs[3 % CPL]);
                        } else {
                            *reinterpret_cast<uint2*>(tb + 2 * lane) = make_uint2(cs[0], cs[1]);
                        }
                        *reinterpret_cast<uint4*>(tb + N_TILE + 4 * lane) = r0;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tfull_bar + 8 * g);
                        ring_next<GROUPS>(g, gph);
                        if (++slot == (uint32_t)TSLOTS) slot = 0;
                        ++blk;
                    }
                    if (sh.lng) { if (++sib == sh.spk) sib = 0; }
                    left -= nb;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_bar + 8 * s);      // the exponent slices are consumed
                    ring_next<STAGES>(s, ph);
                }
            }
            if (out_of_range) atomicCAS(p.status, 0, STATUS_EXPONENT_RANGE);
        }
    } else {
        // ------------------------------------------------------------------ rescale warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_RESCALE));
        const int rwarp = warp - CONTROL_WARPS;              // 0..7
        const int quarter = warp & 3, half = rwarp >> 2;     // tensor-memory lanes follow warp % 4; half = column group
        const int row = quarter * 32 + lane;                 // row of the tile = tensor-memory lane
        const int col0 = half * COLS_PER_WARP;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + col0;
        uint64_t acc2[COLS_PER_WARP / 2];                    // FP32 accumulators, two columns per entry
        uint32_t bias16[MAGIC ? 16 : 1];
        if (MAGIC) {
            {
                uint32_t bias[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) bias[i] = BIAS_BITS;
                for (int gp = 0; gp < GROUPS * PARTS; ++gp)
#pragma unroll
                    for (int c8 = 0; c8 < COLS_PER_WARP / 8; ++c8) tc_st8(lane_addr + gp * N_TILE + c8 * 8, bias);
                tc_wait_st();
            }
            // Read the bias back as one sixteen-register tuple: a tuple that is born as such is passed
            // to every re-arming store in place, while separately defined registers are copied into a
            // fresh tuple for each store (one extra instruction per register and store).
            tc_ld16(lane_addr, reinterpret_cast<uint32_t(&)[16]>(bias16));
            tc_wait_ld();
        }
        // every accumulator group starts out free
        tc_fence_before();
        __syncwarp();
        if (lane == 0)
            for (int g = 0; g < GROUPS; ++g) mbar_arrive(tempty_bar + 8 * g);

        uint32_t g = 0, gph = 0, slot = 0, blk = 0, out_turn = 0;
        bool ok = true;
        for (int wi = blockIdx.x; ok && wi < total_work; wi += gridDim.x) {
            const Work w = get_work(p, wi);
            const int n0 = w.nt * N_TILE;
            const int64_t gi = w.m0 + row;
#pragma unroll
            for (int c = 0; c < COLS_PER_WARP / 2; ++c) acc2[c] = 0ull;
            for (int kb = w.kb0; kb < w.kb0 + w.nblk; ++kb, ++blk) {
                // one wait per block: the block sums are complete and the scale table is written
                if (!__all_sync(0xffffffffu, mbar_wait_quick(tfull_bar + 8 * g, gph, abort_flag, p.status, 302))) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = lane_addr + g * PARTS * N_TILE;
                const uint32_t* tab = tables + slot * C::TABLE_SLOT_WORDS + col0;
                const uint32_t sa_u = tables[slot * C::TABLE_SLOT_WORDS + N_TILE + row];
                if (MAGIC && PLANES == 2) {
                    // Two planes, mantissa = 16 hi + lo: the three armed parts read as binary32 are 1.5*2^23 + hi.hi,
                    // + (hi.lo + lo.hi), + lo.lo. One FMA each removes the bias and applies the part's weight and the
                    // row scale, all exactly: 256 hi.hi 2^sA, 16 mid 2^sA, lo.lo 2^sA. The two lower parts add up
                    // exactly (below 2^23 units); adding the upper part is the one rounding of float(P), which a power
                    // of two does not move; then acc += that * 2^sB. No integer-to-float conversion, no integer
                    // arithmetic per element.
                    const float sa_f = __uint_as_float(sa_u);
                    const float k1 = 16.0f * sa_f, k2 = 256.0f * sa_f;
                    const float c0 = -12582912.0f * sa_f, c1 = -12582912.0f * k1, c2 = -12582912.0f * k2;
                    const uint64_t k0_2 = pack2(__float_as_uint(sa_f), __float_as_uint(sa_f)), c0_2 = pack2(__float_as_uint(c0), __float_as_uint(c0));
                    const uint64_t k1_2 = pack2(__float_as_uint(k1), __float_as_uint(k1)), c1_2 = pack2(__float_as_uint(c1), __float_as_uint(c1));
                    const uint64_t k2_2 = pack2(__float_as_uint(k2), __float_as_uint(k2)), c2_2 = pack2(__float_as_uint(c2), __float_as_uint(c2));
                    constexpr int CH = 16;
                    constexpr int NCHK = COLS_PER_WARP / CH;
                    uint32_t v[2][3][CH];
#pragma unroll
                    for (int part = 0; part < 3; ++part) tc_ld16(taddr + part * N_TILE, v[0][part]);
#pragma unroll
                    for (int ch = 0; ch < NCHK; ++ch) {
                        tc_wait_ld();
                        if (ch + 1 < NCHK) {
#pragma unroll
                            for (int part = 0; part < 3; ++part) tc_ld16(taddr + part * N_TILE + (ch + 1) * CH, v[(ch + 1) & 1][part]);
                        }
                        const uint32_t(&xh)[CH] = v[ch & 1][0];
                        const uint32_t(&xm)[CH] = v[ch & 1][1];
                        const uint32_t(&xl)[CH] = v[ch & 1][2];
                        if (DUMP && p.P != nullptr && gi < p.M) {
#pragma unroll
                            for (int c = 0; c < CH; ++c) {
                                const int64_t gj = n0 + col0 + ch * CH + c;
                                if (gj < p.N)
                                    p.P[(gi * p.N + gj) * p.nkb + kb] =
                                        (int32_t)(((xh[c] - BIAS_BITS) << 8) + ((xm[c] - BIAS_BITS) << 4) + (xl[c] - BIAS_BITS));
                            }
                        }
#pragma unroll
                        for (int q = 0; q < CH; q += 2) {
                            const uint2 sb = *reinterpret_cast<const uint2*>(tab + ch * CH + q);
                            const uint64_t h01 = ffma2(pack2(xh[q], xh[q + 1]), k2_2, c2_2);
                            const uint64_t m01 = ffma2(pack2(xm[q], xm[q + 1]), k1_2, c1_2);
                            const uint64_t l01 = ffma2(pack2(xl[q], xl[q + 1]), k0_2, c0_2);
                            const uint64_t p01 = fadd2(h01, fadd2(m01, l01));
                            acc2[(ch * CH + q) / 2] = ffma2(p01, pack2(sb.x, sb.y), acc2[(ch * CH + q) / 2]);
                        }
#pragma unroll
                        for (int part = 0; part < 3; ++part)
                            tc_st16(taddr + part * N_TILE + ch * CH, reinterpret_cast<const uint32_t(&)[16]>(bias16));   // re-arm
                    }
                    tc_wait_st();
                } else if (MAGIC) {
                    // the accumulator was armed with 0x4B400000, so a block sum read as binary32 is
                    // v = 1.5*2^23 + P exactly;  t = (v - 1.5*2^23) * 2^sA = P * 2^sA;  acc += t * 2^sB
                    const float sa_f = __uint_as_float(sa_u);
                    const float ca_f = -12582912.0f * sa_f;
                    const uint64_t sa2 = pack2(__float_as_uint(sa_f), __float_as_uint(sa_f));
                    const uint64_t ca2 = pack2(__float_as_uint(ca_f), __float_as_uint(ca_f));
                    constexpr int CH = 16;
                    constexpr int NCHK = COLS_PER_WARP / CH;
                    uint32_t v[2][CH];
                    tc_ld16(taddr, v[0]);
#pragma unroll
                    for (int ch = 0; ch < NCHK; ++ch) {
                        tc_wait_ld();
                        if (ch + 1 < NCHK) tc_ld16(taddr + (ch + 1) * CH, v[(ch + 1) & 1]);
                        const uint32_t(&x)[CH] = v[ch & 1];
                        if (DUMP && p.P != nullptr && gi < p.M) {
#pragma unroll
                            for (int c = 0; c < CH; ++c) {
                                const int64_t gj = n0 + col0 + ch * CH + c;
                                if (gj < p.N) p.P[(gi * p.N + gj) * p.nkb + kb] = (int32_t)(x[c] - BIAS_BITS);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < CH; q += 4) {
                            const uint4 sb = *reinterpret_cast<const uint4*>(tab + ch * CH + q);
                            const uint64_t t01 = ffma2(pack2(x[q], x[q + 1]), sa2, ca2);
                            const uint64_t t23 = ffma2(pack2(x[q + 2], x[q + 3]), sa2, ca2);
                            acc2[(ch * CH + q) / 2] = ffma2(t01, pack2(sb.x, sb.y), acc2[(ch * CH + q) / 2]);
                            acc2[(ch * CH + q) / 2 + 1] = ffma2(t23, pack2(sb.z, sb.w), acc2[(ch * CH + q) / 2 + 1]);
                        }
                        tc_st16(taddr + ch * CH, reinterpret_cast<const uint32_t(&)[16]>(bias16));   // re-arm
                    }
                    tc_wait_st();
                } else {
                    const int sa = (int)sa_u;
#pragma unroll
                    for (int ch = 0; ch < COLS_PER_WARP / 16; ++ch) {
                        uint32_t v[16];
                        tc_ld16(taddr + ch * 16, v);
                        if (PLANES == 2) {
                            // mantissa = 16 hi + lo:  P = 256 hi.hi + 16 (hi.lo + lo.hi) + lo.lo
                            uint32_t mid[16], ll[16];
                            tc_ld16(taddr + N_TILE + ch * 16, mid);
                            tc_ld16(taddr + 2 * N_TILE + ch * 16, ll);
                            tc_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c) v[c] = (v[c] << 8) + (mid[c] << 4) + ll[c];
                        } else {
                            tc_wait_ld();
                        }
                        if (DUMP && p.P != nullptr && gi < p.M) {
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const int64_t gj = n0 + col0 + ch * 16 + c;
                                if (gj < p.N) p.P[(gi * p.N + gj) * p.nkb + kb] = (int32_t)v[c];
                            }
                        }
#pragma unroll
                        for (int c4 = 0; c4 < 16; c4 += 4) {
                            const uint4 sb = *reinterpret_cast<const uint4*>(tab + ch * 16 + c4);
                            float a0, a1, a2, a3;
                            unpack2(acc2[(ch * 16 + c4) / 2], a0, a1);
                            unpack2(acc2[(ch * 16 + c4) / 2 + 1], a2, a3);
                            a0 = fmaf((float)(int)v[c4 + 0], __int_as_float(sa + (int)sb.x), a0);
                            a1 = fmaf((float)(int)v[c4 + 1], __int_as_float(sa + (int)sb.y), a1);
                            a2 = fmaf((float)(int)v[c4 + 2], __int_as_float(sa + (int)sb.z), a2);
                            a3 = fmaf((float)(int)v[c4 + 3], __int_as_float(sa + (int)sb.w), a3);
                            acc2[(ch * 16 + c4) / 2] = pack2(__float_as_uint(a0), __float_as_uint(a1));
                            acc2[(ch * 16 + c4) / 2 + 1] = pack2(__float_as_uint(a2), __float_as_uint(a3));
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(tempty_bar + 8 * g);
                }
                ring_next<GROUPS>(g, gph);
                if (++slot == (uint32_t)TSLOTS) slot = 0;
            }
            if (!ok) break;
            // ---- store the tile (or this split's partial tile)
            float* dst = p.splits > 1 ? p.partial + (int64_t)w.split * p.M * p.ldp : p.C;
            const int64_t ldd = p.splits > 1 ? p.ldp : p.ldc;
            if (TSTORE) {
                // Each lane writes its row's 32 columns into a 128B-swizzled box (16-byte piece j of row r at
                // piece j ^ (r & 7): conflict-free), one lane hands the box to the copy engine, and the warp goes
                // on; a box is reused once the copy engine has read the one sent two boxes earlier. The copy
                // clips what lies beyond M or N.
#pragma unroll
                for (int cb = 0; cb < COLS_PER_WARP / 32; ++cb) {
                    const uint32_t buf = base + out_off + (uint32_t)((rwarp * 2 + (out_turn & 1)) * C::OUT_BUF);
                    if (out_turn >= 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t at = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v2.b64 [%0], {%1, %2};" ::"r"(at), "l"(acc2[cb * 16 + 2 * j]), "l"(acc2[cb * 16 + 2 * j + 1]) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                     ::"l"(reinterpret_cast<uint64_t>(&mapC)), "r"(buf), "r"(n0 + col0 + 32 * cb), "r"(w.m0 + quarter * 32) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    ++out_turn;
                }
            } else if (dst != nullptr && gi < p.M) {
                float* rowp = dst + gi * ldd + n0 + col0;
                // full 32-byte sectors per lane where the row pitch allows it (each lane owns a row)
                const bool wide = (ldd & 7) == 0 && (reinterpret_cast<uintptr_t>(dst) & 31) == 0;
                // 16-byte stores need a pitch of whole quads; any other pitch (an output ten columns wide) goes element by element
                const bool quad = (ldd & 3) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0;
#pragma unroll
                for (int c = 0; c < COLS_PER_WARP; c += 4) {
                    const int64_t gj = n0 + col0 + c;
                    if (wide && (c & 7) == 0 && gj + 7 < p.N) {
                        st_global_256(rowp + c, acc2[c / 2], acc2[c / 2 + 1], acc2[c / 2 + 2], acc2[c / 2 + 3]);
                    } else if (wide && (c & 7) == 4 && gj + 3 < p.N) {
                        // second half of a sector already written above
                    } else if (quad && gj + 3 < p.N) {
                        *reinterpret_cast<ulonglong2*>(rowp + c) = make_ulonglong2(acc2[c / 2], acc2[c / 2 + 1]);
                    } else {
                        float e4[4];
                        unpack2(acc2[c / 2], e4[0], e4[1]);
                        unpack2(acc2[c / 2 + 1], e4[2], e4[3]);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (gj + e < p.N) rowp[c + e] = e4[e];
                    }
                }
            }
        }
    }

    // ------------------------------------------------------------------ teardown
    if (TSTORE) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");    // this thread's output boxes have been written
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// Sums the split-K partial tiles in ascending split order.
__global__ void splitk_reduce(const float* __restrict__ partial, int splits, int64_t M, int64_t N, int64_t ldp,
                              float* __restrict__ C, int64_t ldc) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * N) return;
    const int64_t r = i / N, c = i % N;
    float acc = partial[r * ldp + c];
    for (int s = 1; s < splits; ++s) acc = __fadd_rn(acc, partial[(int64_t)s * M * ldp + r * ldp + c]);
    C[r * ldc + c] = acc;
}

// ------------------------------------------------------------------------------ host side

// 2-D FP32 tensor [rows][cols] with pitch ld (elements); box = 32 columns x 32 rows, 128B-swizzled.
int make_map_out(CUtensorMap* m, float* ptr, uint64_t cols, uint64_t rows, uint64_t ld) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return HBFP_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HBFP_OK : HBFP_ERR_CUDA;
}

template <int N_TILE, int PLANES, bool MAGIC, bool DUMP, bool TSTORE = false>
int launch_cfg(const Problem& p, const Packed& a, const Packed& b, cudaStream_t st) {
    using C = Cfg<N_TILE, PLANES, TSTORE>;
    CUtensorMap mA0, mA1, mB0, mB1, mEA, mEB, mC;
    int rc;
    rc = make_map(&mA0, a.mant, a.L.kst, a.L.rows, a.L.kst, STAGE_K, TILE_M, true);
    if (rc) return rc;
    rc = make_map(&mB0, b.mant, b.L.kst, b.L.rows, b.L.kst, STAGE_K, N_TILE, true);
    if (rc) return rc;
    mA1 = mA0;
    mB1 = mB0;
    if (PLANES == 2) {
        rc = make_map(&mA1, a.mant + a.L.plane_stride, a.L.kst, a.L.rows, a.L.kst, STAGE_K, TILE_M, true);
        if (rc) return rc;
        rc = make_map(&mB1, b.mant + b.L.plane_stride, b.L.kst, b.L.rows, b.L.kst, STAGE_K, N_TILE, true);
        if (rc) return rc;
    }
    rc = make_map(&mEA, a.exps, a.L.rs, a.L.nkb, a.L.rs, TILE_M, 4, false);
    if (rc) return rc;
    rc = make_map(&mEB, b.exps, b.L.rs, b.L.nkb, b.L.rs, N_TILE, 4, false);
    if (rc) return rc;
    mC = mEB;                                                  // unused unless TSTORE
    if (TSTORE) {
        rc = make_map_out(&mC, p.C, (uint64_t)p.N, (uint64_t)p.M, (uint64_t)p.ldc);
        if (rc) return rc;
    }
    // the attribute belongs to the device: set once per device, not once per process
    static bool attr_set[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return HBFP_ERR_CUDA;
    if (!attr_set[dev]) {
        HBFP_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<N_TILE, PLANES, MAGIC, DUMP, TSTORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        attr_set[dev] = true;
    }
    const int64_t work = (int64_t)p.tiles_m * p.tiles_n * p.splits;
    const int grid = (int)(work < sm_count() ? work : sm_count());
    gemm_tc_kernel<N_TILE, PLANES, MAGIC, DUMP, TSTORE><<<grid, THREADS, C::SMEM, st>>>(mA0, mA1, mB0, mB1, mEA, mEB, mC, p);
    return launch_status();
}

// One warp waits, with the kernels' own bounded wait and a cycle budget chosen by the caller, on a
// barrier that nobody arrives on: the wait runs out, records `code`, raises the abort flag and the
// kernel returns. No TMA, no tensor memory: nothing that could fault or outlive the launch.
__global__ void __launch_bounds__(32, 1) wait_probe_kernel(int32_t* status, long long limit_cycles, int code, int* outcome) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_word = 0;
    }
    __syncwarp();
    const bool done = mbar_wait(smem_u32(&bar), 0, abort_flag, status, code, true, limit_cycles);
    const bool any_done = __any_sync(0xffffffffu, done);
    if (threadIdx.x == 0 && outcome) *outcome = (any_done ? 1 : 0) | (*abort_flag ? 2 : 0);   // expected: 2
}

}  // namespace

int launch_wait_probe(long long limit_cycles, int code, int* outcome, cudaStream_t st) {
    int32_t* status = device_status_word();
    if (!status) return HBFP_ERR_CUDA;
    if (limit_cycles < 0 || limit_cycles > 100000000ll || code <= 0 || code >= 900) return HBFP_ERR_INVALID_ARG;
    wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_cycles, code, outcome);
    return launch_status();
}

TensorPlan plan_gemm_tensor(int64_t M, int64_t N, int64_t K, const Layout& la, const Layout& lb, int mant_bits_a,
                            int mant_bits_b) {
    TensorPlan t{};
    (void)mant_bits_a;
    (void)mant_bits_b;
    if (M <= 0 || N <= 0 || K <= 0) return t;
    if (la.planes != lb.planes || la.bp != lb.bp || la.nkb != lb.nkb) return t;
    const int64_t bp = la.bp;
    if (!(bp == 32 || bp == 64 || bp == 128 || (bp > 128 && bp % 128 == 0))) return t;
    if (bp > (1 << 20) || M > (1ll << 30) || N > (1ll << 30) || la.kst > (1ll << 31) - 256) return t;
    const int64_t tiles_m = (M + TILE_M - 1) / TILE_M;
    const int SMS = 148;                                   // planning constant: the target part
    int n_tile;
    if (la.planes == 2) {
        n_tile = 64;
    } else {
        n_tile = 256;
        while (n_tile > 64 && (tiles_m * ((N + n_tile - 1) / n_tile) < SMS || N <= n_tile / 2)) n_tile /= 2;
    }
    const int64_t tiles = tiles_m * ((N + n_tile - 1) / n_tile);
    // split-K for small outputs with a long contraction: at least two stages per split, split
    // boundaries on stage boundaries.
    const int64_t stages_total = (la.nkb * bp + STAGE_K - 1) / STAGE_K;
    int64_t splits = 1;
    if (tiles * 2 <= SMS) {
        splits = SMS / tiles;
        if (splits > stages_total / 2) splits = stages_total / 2;
        if (splits < 1) splits = 1;
    }
    const int64_t unit = bp >= STAGE_K ? 1 : STAGE_K / bp;   // blocks per stage
    int64_t kbps = (la.nkb + splits - 1) / splits;
    kbps = (kbps + unit - 1) / unit * unit;
    splits = (la.nkb + kbps - 1) / kbps;
    t.supported = 1;
    t.n_tile = n_tile;
    t.splits = (int)splits;
    t.kb_per_split = kbps;
    t.partial_bytes = splits > 1 ? (size_t)splits * (size_t)M * (size_t)round_up(N, 4) * sizeof(float) : 0;
    return t;
}

int launch_gemm_tensor(int64_t M, int64_t N, int64_t K, const Packed& a, const Packed& b, float* Cout, int64_t ldc,
                       int32_t* P, const TensorPlan& plan, void* partial, cudaStream_t st) {
    (void)K;
    if (!plan.supported) return HBFP_ERR_UNSUPPORTED;
    Problem p{};
    p.M = M;
    p.N = N;
    p.nkb = a.L.nkb;
    p.bp = (int)a.L.bp;
    p.tiles_m = (int)((M + TILE_M - 1) / TILE_M);
    p.tiles_n = (int)((N + plan.n_tile - 1) / plan.n_tile);
    p.splits = P ? 1 : plan.splits;
    p.kb_per_split = P ? a.L.nkb : plan.kb_per_split;
    p.C = Cout;
    p.ldc = ldc;
    p.partial = static_cast<float*>(partial);
    p.ldp = round_up(N, 4);
    p.P = P;
    p.status = device_status_word();
    if (!p.status) return HBFP_ERR_CUDA;
    if (p.splits > 1 && !partial) return HBFP_ERR_WORKSPACE;
    int rc;
    // the biased-accumulator path needs every |P| < 2^22
    const int64_t qa = (1ll << (a.mant_bits - 1)) - 1, qb = (1ll << (b.mant_bits - 1)) - 1;
    // (two planes: the largest part, hi.hi, stays below 128 * 128 * b)
    const bool magic = a.L.planes == 1 ? qa * qb * a.L.b < (1ll << 22) : 128ll * 128ll * a.L.b < (1ll << 22);
    // Short contractions are bound by the write of C: the tile then leaves through shared memory and TMA stores,
    // which the copy engine writes as whole lines while the warps go on with the next tile.
    const bool tstore = p.splits == 1 && !P && a.L.nkb * a.L.bp <= 1024 && (reinterpret_cast<uintptr_t>(Cout) & 15) == 0 && (ldc % 4) == 0;
    if (P) {   // the inspection build of the kernel: 64-column tiles, writes the block sums
        p.tiles_n = (int)((N + 63) / 64);
        if (a.L.planes == 2) rc = magic ? launch_cfg<64, 2, true, true>(p, a, b, st) : launch_cfg<64, 2, false, true>(p, a, b, st);
        else rc = magic ? launch_cfg<64, 1, true, true>(p, a, b, st) : launch_cfg<64, 1, false, true>(p, a, b, st);
    } else if (a.L.planes == 2) rc = magic ? launch_cfg<64, 2, true, false>(p, a, b, st) : launch_cfg<64, 2, false, false>(p, a, b, st);
    else if (magic && tstore && plan.n_tile == 256) rc = launch_cfg<256, 1, true, false, true>(p, a, b, st);
    else if (magic && tstore && plan.n_tile == 128) rc = launch_cfg<128, 1, true, false, true>(p, a, b, st);
    else if (plan.n_tile == 256) rc = magic ? launch_cfg<256, 1, true, false>(p, a, b, st) : launch_cfg<256, 1, false, false>(p, a, b, st);
    else if (plan.n_tile == 128) rc = magic ? launch_cfg<128, 1, true, false>(p, a, b, st) : launch_cfg<128, 1, false, false>(p, a, b, st);
    else rc = magic ? launch_cfg<64, 1, true, false>(p, a, b, st) : launch_cfg<64, 1, false, false>(p, a, b, st);
    if (rc) return rc;
    if (p.splits > 1) {
        const int64_t n = M * N;
        splitk_reduce<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(p.partial, p.splits, M, N, p.ldp, Cout, ldc);
        return launch_status();
    }
    return HBFP_OK;
}

}  // namespace hbfp
