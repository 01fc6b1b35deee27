// Paired-SM tensor-core BFP GEMM for sm_100a (8-bit mantissas, blocks of 32, 64 or 128 elements).
//
// Two CTAs of a cluster (one SM each) compute one 256 x 256 output tile: tcgen05.mma
// cta_group::2 with M = 256 reads the A rows of both CTAs and one half of the B rows from each
// CTA's shared memory, and leaves rows 0-127 of the int32 block sums in the first CTA's tensor
// memory and rows 128-255 in the second one's. Per SM this is the same arithmetic and the same
// rescale work as a 128 x 256 tile on one SM, but only half of the B panel crosses from L2 into
// each SM, which is what limits the single-SM kernel on large problems.
//
// Roles per CTA (16 warps): warp 0 TMA producer, warp 1 MMA issuer (only in the cluster's first
// CTA, the leader) and tensor-memory owner, warps 2 and 3 scale-table builders (even / odd
// K-blocks), warps 4-15 rescale (Eq. 2 per block, blocks accumulated in FP32, Sec. 4): three per
// lane quarter of tensor memory, which split the 256 columns 88 + 88 + 80.
//
// Barriers. Mantissa tiles of both CTAs complete on the leader's full[s]; exponent slices on a
// local efull[s]; the leader's MMA thread commits to tfull[g] of both CTAs (one commit per
// K-block and no other); the table builders hand the stages back to the producer (empty[s]); the
// rescale warps of both CTAs arrive on the leader's tempty[g]. A rescale warp does one wait and
// one arrival per K-block: the builder's "scales written" arrival is counted on tfull[g]
// together with the MMA commit, and the builder learns that a table slot is free again from
// the completion of tfull two blocks back (the MMAs of that block were issued only after every
// rescale warp had finished the slot's last reader). Every wait is bounded: when one expires the
// CTA records a code in the device status word, raises its abort flag, drains what it can wait
// for and leaves through the common teardown (cluster barrier, tensor memory freed).
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace hbfp {
namespace {

constexpr int N_TILE = 256;            // columns of the pair tile = accumulator columns per CTA
constexpr int PAIR_M = 2 * TILE_M;     // rows of the pair tile
constexpr int B_HALF = N_TILE / 2;     // B rows staged in each CTA
// Rescale warps: three per sub-partition (88 + 88 + 80 columns). The rescale is bound by latencies, not
// by a pipe, so the third warp pays.
constexpr int RESCALE_WARPS = 12;
constexpr int CONTROL_WARPS = 4;
constexpr int PRODUCER_WARP = 0, MMA_WARP = 1, TABLE_WARP = 2;
constexpr int THREADS = 32 * (CONTROL_WARPS + RESCALE_WARPS);
// setmaxnreg totals must not exceed the launch allocation (512 threads x 128 registers)
constexpr int REGS_RESCALE = 144, REGS_CONTROL = 64, REGS_LAUNCH = 128;
static_assert(128 * REGS_CONTROL + 32 * RESCALE_WARPS * REGS_RESCALE <= THREADS * REGS_LAUNCH - 512, "register split");

// Offset step (see rescale_loop): 32 products 255 * 255 per accumulator word. The scale of a block
// is split 2^(sA + c) * 2^(sB + 149 - c); c = SHIFT suits sA in [-63, 41] and sB in [-63, 64], and the
// table warp moves it per block when the exponents ask for it.
constexpr int OFFSET = 32 * 255 * 255;
constexpr int SHIFT = 86;
constexpr int GROUPS = TMEM_COLS / N_TILE;                  // 2 accumulator groups
constexpr int A_BYTES = TILE_M * STAGE_K, B_BYTES = B_HALF * STAGE_K;
constexpr int MANT_STAGE = A_BYTES + B_BYTES;               // 32 KB per CTA and stage
constexpr int EXP_A = 4 * TILE_M, EXP_B = 4 * N_TILE;       // up to four blocks start in a stage
constexpr int EXP_STAGE = EXP_A + EXP_B;
constexpr int TSLOTS = 4;
constexpr int TABLE_SLOT_WORDS = N_TILE + TILE_M;
constexpr int TABLE_BYTES = 4 * TSLOTS * TABLE_SLOT_WORDS;
constexpr int STAGES = 5;      // measured: 5 stages 2.6 % fewer cycles than 6 (n = 16384), 4 as many as 6, 3 far more
constexpr int ONES_BYTES = TILE_M * STAGE_K;   // 128 rows of 0xFF bytes: both operands of the offset step
constexpr int SMEM = 1024 + STAGES * (MANT_STAGE + EXP_STAGE) + TABLE_BYTES + ONES_BYTES + 1024;
static_assert(SMEM <= 232448, "shared memory");

// Length of the last launch in SM cycles, per CTA (hbfp_last_gemm_cycles): cycles ÷ event time is the clock the
// SMs really ran at, which under the power cap is well below the one the driver reports.
constexpr int MAX_CTAS = 2 * 148 * 2;
__device__ unsigned long long g_cta_cycles[MAX_CTAS];

struct Problem {
    int64_t M, N;
    int64_t nkb;
    int bp;
    int tiles_m, tiles_n;   // pair tiles
    int splits;
    int64_t kb_per_split;
    float* C;
    int64_t ldc;
    float* partial;
    int64_t ldp;
    int32_t* status;
};

struct Work {
    int m0, n0, split;
    int kb0, nblk;          // first K-block and number of K-blocks of this item
};

// Same traversal as the single-SM kernel: groups of tile rows (2048 matrix rows) sweep across N
// so that their B panels are shared in L2. 32-bit arithmetic only; returned by value so that the
// fields stay in registers.
__device__ __forceinline__ Work get_work(const Problem& p, int w) {
    Work out;
    const int tiles = p.tiles_m * p.tiles_n;
    const int split = w / tiles;
    const int t = w - split * tiles;
    const int G = 8;
    const int per_group = G * p.tiles_n;
    const int group = t / per_group;
    const int first_m = group * G;
    const int gsize = min(G, p.tiles_m - first_m);
    const int within = t - group * per_group;
    const int nt = within / gsize;
    out.m0 = (first_m + (within - nt * gsize)) * PAIR_M;
    out.n0 = nt * N_TILE;
    out.split = split;
    out.kb0 = split * (int)p.kb_per_split;
    out.nblk = min((int)p.nkb, out.kb0 + (int)p.kb_per_split) - out.kb0;
    return out;
}

// ------------------------------------------------------------------------------ cluster PTX

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in the CTA of the given rank.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    // release at CTA scope: what the arrival has to order are this warp's tensor-memory accesses, and
    // tcgen05.wait + tcgen05.fence::before_thread_sync do that; a cluster-scope release costs ~1000 cycles
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}

// Non-blocking look at a barrier phase.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

// try_wait with a short suspend hint: the thread sleeps at most about `ns` nanoseconds and takes no issue slots from
// the rescale warps of its sub-partition meanwhile.
__device__ __forceinline__ bool mbar_try_wait_ns(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}

// Wait on a barrier that threads of the other CTA arrive on. What the arrivals order are tensor-memory
// accesses, fenced with tcgen05.fence on both sides, so the default (CTA-scope) acquire is enough.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(WAIT_HINT_NS) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  int32_t* status, int code) {
    // A thread that try_wait has put to sleep with the long hint below wakes up late (the kernel then settles in a
    // mode 20 % slower), and a thread that spins on test_wait takes issue slots from the rescale warps of its
    // sub-partition: 32 looks, then naps of at most 64 ns, the long sleep only when those run out. Measured in
    // cycles per launch against spinning alone (n = 8192): - 5 % for blocks of 128, - 1 % for 64, - 4 % for 32;
    // one look before the naps is as good for 128 but 8 % worse for 64; the nap's length (32-128 ns) does not matter.
    for (int i = 0; i < 32; ++i)
        if (mbar_test_wait(bar, parity)) return true;
    for (int i = 0; i < 1024; ++i)
        if (mbar_try_wait_ns(bar, parity, 64u)) return true;
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort_flag = 1;
            atomicCAS(status, 0, code);
            return false;
        }
    }
}

// Tile copy issued by one CTA of a pair; the completion bytes may be counted on a barrier of
// either CTA (`bar` is a cluster-window address). A plain copy to one destination.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar, uint64_t hint) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "l"(hint) : "memory");
}
constexpr uint64_t L2_EVICT_NORMAL = 0x1000000000000000ull;

// D[tmem of both CTAs] (+)= A * B, int8 x int8 -> int32, M = 256 (128 rows per CTA), K = 32.
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives (once all earlier MMAs of this thread have completed) on the barrier at this offset in
// every CTA of the mask.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(cta_mask) : "memory");
}
__device__ __forceinline__ constexpr uint32_t idesc_i8_pair() {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N_TILE >> 3) << 17) | ((uint32_t)(PAIR_M >> 4) << 24);
}
// The same shape with both operands taken as unsigned bytes (the offset step).
__device__ __forceinline__ constexpr uint32_t idesc_u8_pair() {
    return (2u << 4) | ((uint32_t)(N_TILE >> 3) << 17) | ((uint32_t)(PAIR_M >> 4) << 24);
}

// 2^(e + sh) as binary32 bits, e = signed byte i of a packed word of four exponents.
__device__ __forceinline__ uint32_t exp_to_scale(uint32_t packed, int i, int sh) {
    const int e = (int)(int8_t)(packed >> (8 * i));
    return (uint32_t)(e + 127 + sh) << 23;
}
// Smallest / largest of the four signed bytes of a word.
__device__ __forceinline__ int byte_min(uint32_t w) {
    w = __vmins4(w, w >> 16);
    w = __vmins4(w, w >> 8);
    return (int)(int8_t)w;
}
__device__ __forceinline__ int byte_max(uint32_t w) {
    w = __vmaxs4(w, w >> 16);
    w = __vmaxs4(w, w >> 8);
    return (int)(int8_t)w;
}

// Advances a ring position (stage, accumulator group or table slot) and its phase bit.
template <int N>
__device__ __forceinline__ void ring_next(uint32_t& i, uint32_t& ph) {
    if (++i == N) { i = 0; ph ^= 1u; }
}

// ------------------------------------------------------------------------------ rescale warps

struct RescaleArgs {
    uint32_t tfull_bar, leader_tempty, tmem_base;
    uint32_t* tables;
    int total_work, cluster, nclusters;
    uint32_t rank;
    volatile int* abort_flag;
};

// The loop of one rescale warp: rows = its lane quarter of this CTA's half tile, columns
// [col0, col0 + NCOLS) of every accumulator group, read in chunks of CHW columns.
//
// Every block's first MMA step multiplies two constant operands (all bytes 255, taken as unsigned)
// and overwrites the group with OFFSET = 32 * 255 * 255; the block's own steps accumulate on top, so
// a word read back is X = OFFSET + P with 0 < X < 2^23 (|P| <= 127 * 127 * 128 < OFFSET): as a
// binary32 pattern that is the subnormal X * 2^-149, exactly linear in P. Two packed FMAs finish Eq. 2:
//   t   = fma(x, 2^(sA + c), -OFFSET * 2^(sA + c - 149)) = P * 2^(sA + c - 149)   (exact)
//   acc = fma(t, 2^(sB + 149 - c), acc)                                        (one rounding)
// with the block's split c chosen by the table warp.
// Nothing has to be written back to tensor memory, and the group is handed back as soon as its last
// chunk is in registers.
template <int NCOLS, int CHW>
__device__ __forceinline__ void rescale_loop(const Problem& p, const RescaleArgs& a, int col0) {
    constexpr int NCHK = NCOLS / CHW;
    static_assert(NCOLS % CHW == 0 && NCOLS % 8 == 0, "column split");
    const int lane = threadIdx.x & 31, quarter = (threadIdx.x >> 5) & 3;   // tensor-memory lanes follow warp % 4
    const int row = quarter * 32 + lane;                 // row of this CTA's half tile = tensor-memory lane
    const uint32_t lane_addr = a.tmem_base + ((uint32_t)(quarter * 32) << 16) + col0;
    uint64_t acc2[NCOLS / 2];                            // FP32 accumulators, two columns per entry
    {
        // One tensor-memory read before the loop (its result is not used). With it the loop below runs
        // 6 % faster (n = 16384: 1 560 -> 1 680 TOP/s, four runs each): a code-generation effect, measured.
        uint32_t z[8];
        tc_ldn(lane_addr, z);
        tc_wait_ld();
    }
    tc_fence_before();
    __syncwarp();
    // every accumulator group starts out free
    if (lane == 0)
        for (int g = 0; g < GROUPS; ++g) mbar_arrive_remote(a.leader_tempty + 8 * g);

    uint32_t g = 0, gph = 0, slot = 0;
    bool ok = true;
    for (int wi = a.cluster; ok && wi < a.total_work; wi += a.nclusters) {
        const Work w = get_work(p, wi);
        const int64_t gi = w.m0 + (int)a.rank * TILE_M + row;
#pragma unroll
        for (int c = 0; c < NCOLS / 2; ++c) acc2[c] = 0ull;
        for (int kb = 0; kb < w.nblk; ++kb) {
            const uint32_t taddr = lane_addr + g * N_TILE;
            uint32_t v[2][CHW];
            // one wait per block: the block sums are complete and this CTA's scale table is written
            // (polled first: a warp that try_wait has put to sleep wakes up late)
            {
                bool hit = false;
                for (int i = 0; i < 2048 && !hit; ++i) hit = mbar_test_wait(a.tfull_bar + 8 * g, gph);
                if (!__all_sync(0xffffffffu, hit) && !mbar_wait_warp(a.tfull_bar + 8 * g, gph, a.abort_flag, p.status, 312)) { ok = false; break; }
            }
            tc_fence_after();
            tc_ldn(taddr, v[0]);
            const uint32_t* tab = a.tables + slot * TABLE_SLOT_WORDS + col0;
            const uint32_t tab_s = smem_u32(tab);
            const float sa_f = __uint_as_float(a.tables[slot * TABLE_SLOT_WORDS + N_TILE + row]);   // 2^(sA + c)
            const float ca_f = -__uint_as_float((uint32_t)OFFSET) * sa_f;               // -OFFSET * 2^(sA + c - 149)
            const uint64_t sa2 = pack2(__float_as_uint(sa_f), __float_as_uint(sa_f));
            const uint64_t ca2 = pack2(__float_as_uint(ca_f), __float_as_uint(ca_f));
#pragma unroll
            for (int ch = 0; ch < NCHK; ++ch) {
                // the column scales of the chunk are requested before the wait for its block sums, so
                // that their shared-memory latency passes during that wait
                // (asked for as 8-byte pairs: the compiler still fetches 16 bytes at a time but is free in where each
                // pair lands, which saves register moves: 1.1 % fewer cycles than a 16-byte vector load)
                uint64_t sbp[CHW / 2];
#pragma unroll
                for (int q = 0; q < CHW; q += 2)
                    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(sbp[q / 2]) : "r"(tab_s + 4u * (uint32_t)(ch * CHW + q)));
                tc_wait_ld();
                if (ch + 1 < NCHK) {
                    tc_ldn(taddr + (ch + 1) * CHW, v[(ch + 1) & 1]);
                } else {
                    // the whole group is in registers: hand it back before the last chunk's arithmetic
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(a.leader_tempty + 8 * g);
                }
                const uint32_t(&x)[CHW] = v[ch & 1];
#pragma unroll
                for (int q = 0; q < CHW; q += 4) {
                    const uint64_t t01 = ffma2(pack2(x[q], x[q + 1]), sa2, ca2);
                    const uint64_t t23 = ffma2(pack2(x[q + 2], x[q + 3]), sa2, ca2);
                    // The table holds each four column factors as (2 3 0 1): the first accumulator pair of a quad then
                    // takes the second register pair of the loaded quad and the second the first. With the straight
                    // order the compiler emits a register move for about every fifth packed FMA more (operand pairs
                    // in the same register bank); measured 2 % of a stand-alone rescale loop.
                    acc2[(ch * CHW + q) / 2] = ffma2(t01, sbp[q / 2 + 1], acc2[(ch * CHW + q) / 2]);
                    acc2[(ch * CHW + q) / 2 + 1] = ffma2(t23, sbp[q / 2], acc2[(ch * CHW + q) / 2 + 1]);
                }
            }
            ring_next<GROUPS>(g, gph);
            slot = (slot + 1) & (TSLOTS - 1);
        }
        if (!ok) break;
        // ---- store this warp's part of the tile (or of this split's partial tile)
        float* dst = p.splits > 1 ? p.partial + (int64_t)w.split * p.M * p.ldp : p.C;
        const int64_t ldd = p.splits > 1 ? p.ldp : p.ldc;
        if (gi < p.M) {
            float* rowp = dst + gi * ldd + w.n0 + col0;
            // full 32-byte sectors per lane where the row pitch allows it (each lane owns a row)
            const bool wide = (ldd & 7) == 0 && (reinterpret_cast<uintptr_t>(dst) & 31) == 0;
#pragma unroll
            for (int c = 0; c < NCOLS; c += 4) {
                const int64_t gj = w.n0 + col0 + c;
                if (wide && (c & 7) == 0 && gj + 7 < p.N) {
                    st_global_256(rowp + c, acc2[c / 2], acc2[c / 2 + 1], acc2[c / 2 + 2], acc2[c / 2 + 3]);
                } else if (wide && (c & 7) == 4 && gj + 3 < p.N) {
                    // second half of a sector already written above
                } else if (gj + 3 < p.N) {
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

// ------------------------------------------------------------------------------ kernel

// LB = log2(K-blocks per 128-byte stage): 0 for blocks of 128 bytes, 1 for 64, 2 for 32.
template <int LB>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                const __grid_constant__ CUtensorMap mapEA, const __grid_constant__ CUtensorMap mapEB,
                const Problem p) {
    constexpr int BPS = 1 << LB;          // K-blocks per stage
    constexpr int SPB = 4 >> LB;          // K=32 MMA steps per block
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t mant_base = base;                                     // STAGES x MANT_STAGE, 1024-aligned
    const uint32_t exp_base = mant_base + STAGES * MANT_STAGE;           // STAGES x EXP_STAGE
    const uint32_t table_off = STAGES * (MANT_STAGE + EXP_STAGE);
    uint32_t* tables = reinterpret_cast<uint32_t*>(base_ptr + table_off);   // [slot][256 column scales | 128 row scales]
    const uint32_t ones_off = table_off + TABLE_BYTES;                      // 1024-aligned: stages and tables are multiples of 1 KB
    const uint32_t bar_off = ones_off + ONES_BYTES;
    const uint32_t bars = base + bar_off;
    const uint32_t full_bar = bars;                          // leader: mantissa tiles of both CTAs landed
    const uint32_t efull_bar = full_bar + 8 * STAGES;        // local: exponent slices landed
    const uint32_t empty_bar = efull_bar + 8 * STAGES;       // local: stage consumed (both table builders)
    const uint32_t tfull_bar = empty_bar + 8 * STAGES;       // local: block sums complete (MMA commit) and scale table written
    const uint32_t tempty_bar = tfull_bar + 8 * GROUPS;      // leader: group read and re-armed by the rescale warps of both CTAs
    const uint32_t done_bar = tempty_bar + 8 * GROUPS;
    constexpr int BAR_BYTES = 24 * STAGES + 16 * GROUPS + 8;
    static_assert(BAR_BYTES + 8 <= 1024, "barrier area");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + bar_off + BAR_BYTES);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long cycles_start = clock64();
    const uint32_t rank = cluster_ctarank();                 // 0 = leader
    const int cluster = (int)cluster_id_x(), nclusters = (int)cluster_count_x();
    const int total_work = p.tiles_m * p.tiles_n * p.splits;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(efull_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 2);               // this CTA's two table builders, once the stage's MMAs are complete
        }
        for (int g = 0; g < GROUPS; ++g) {
            mbar_init(tfull_bar + 8 * g, 2);                 // MMA commit + this CTA's table builder of the group
            mbar_init(tempty_bar + 8 * g, 2 * RESCALE_WARPS);
        }
        mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < ONES_BYTES / 4; i += THREADS) reinterpret_cast<uint32_t*>(base_ptr + ones_off)[i] = 0xFFFFFFFFu;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes, read by the tensor core
    if (warp == MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_barrier();            // both CTAs' barriers and tensor memory exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < CONTROL_WARPS) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_CONTROL));
        if (warp == PRODUCER_WARP) {
            // -------------------------------------------------------------- TMA producer (both CTAs)
            if (lane == 0) {
                const uint32_t leader_full = map_to_rank(full_bar, 0);
                uint32_t s = 0, ph = 0, it = 0;
                bool ok = true;
                for (int wi = cluster; ok && wi < total_work; wi += nclusters) {
                    const Work w = get_work(p, wi);
                    const int my_m = w.m0 + (int)rank * TILE_M;      // this CTA's A rows
                    const int my_n = w.n0 + (int)rank * B_HALF;      // this CTA's half of the B rows
                    const int nst = (w.nblk + BPS - 1) >> LB;
                    int kb = w.kb0, kbyte = w.kb0 * (128 >> LB);
                    for (int si = 0; si < nst; ++si, kb += BPS, kbyte += STAGE_K, ++it) {
                        if (!mbar_wait(empty_bar + 8 * s, ph ^ 1, abort_flag, p.status, 111)) { ok = false; break; }
                        if (rank == 0) mbar_expect_tx(full_bar + 8 * s, 2u * MANT_STAGE);
                        mbar_expect_tx(efull_bar + 8 * s, (uint32_t)EXP_STAGE);
                        const uint32_t ms = mant_base + s * MANT_STAGE;
                        tma_load_2d_pair(ms, &mapA, kbyte, my_m, leader_full + 8 * s, L2_EVICT_LAST);
                        tma_load_2d_pair(ms + A_BYTES, &mapB, kbyte, my_n, leader_full + 8 * s, L2_EVICT_NORMAL);
                        const uint32_t es = exp_base + s * EXP_STAGE;
                        tma_load_2d(es, &mapEA, my_m, kb, efull_bar + 8 * s);
                        tma_load_2d(es + EXP_A, &mapEB, w.n0, kb, efull_bar + 8 * s);
                        ring_next<STAGES>(s, ph);
                    }
                }
                // Drain the copies this CTA can wait for: its exponent slices, and on the leader the
                // mantissa tiles of both CTAs. In a normal run the consumers already waited for all
                // of them, so these return at once.
                const uint32_t back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                for (uint32_t k = 0; k < back; ++k) {
                    if (s == 0) { s = STAGES - 1; ph ^= 1u; } else { --s; }
                    mbar_wait(efull_bar + 8 * s, ph, abort_flag, p.status, 112, false);
                    if (rank == 0) mbar_wait(full_bar + 8 * s, ph, abort_flag, p.status, 113, false);
                }
            }
        } else if (warp == MMA_WARP) {
            // -------------------------------------------------------------- MMA issuer (leader only)
            if (lane == 0 && rank == 0) {
                constexpr uint32_t idesc = idesc_i8_pair();
                const uint64_t ones_desc = smem_desc_sw128(base + ones_off);
                uint32_t s = 0, ph = 0, g = 0, gph = 0, it = 0, blk = 0;
                // The barriers the next MMAs will need are polled (without blocking) just before the last
                // MMA of a block is issued, while earlier MMAs still occupy the tensor pipe; a barrier found
                // complete then is not waited on again, so the pipe is refilled without a bubble.
                bool pre_full = false, pre_tempty = false;
                bool ok = true;
                for (int wi = cluster; ok && wi < total_work; wi += nclusters) {
                    const Work w = get_work(p, wi);
                    const int nst = (w.nblk + BPS - 1) >> LB;
                    int left = w.nblk;
                    for (int si = 0; ok && si < nst; ++si, left -= BPS, ++it) {
                        if (pre_full) pre_full = false;
                        else if (!mbar_wait(full_bar + 8 * s, ph, abort_flag, p.status, 211)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t ms = mant_base + s * MANT_STAGE;
                        const uint64_t a_desc = smem_desc_sw128(ms), b_desc = smem_desc_sw128(ms + A_BYTES);
                        const int nb = left < BPS ? left : BPS;       // blocks of this stage
#pragma unroll
                        for (int jb = 0; jb < BPS; ++jb) {
                            if (jb < nb) {
                                // the group was read by the rescale warps of both CTAs
                                if (pre_tempty) pre_tempty = false;
                                else if (!mbar_wait_cluster(tempty_bar + 8 * g, gph, abort_flag, p.status, 212)) { ok = false; break; }
                                tc_fence_after();
                                const uint32_t d = tmem_base + g * N_TILE;
                                // offset step: overwrites the group with 32 * 255 * 255 in every word
                                tc_mma_i8_pair(d, ones_desc, ones_desc, idesc_u8_pair(), 0u);
#pragma unroll
                                for (int q = 0; q < SPB; ++q) {
                                    if (q == SPB - 1) {
                                        // look ahead while the tensor pipe still has the earlier MMAs to run
                                        uint32_t g2 = g, gph2 = gph;
                                        ring_next<GROUPS>(g2, gph2);
                                        pre_tempty = mbar_test_wait(tempty_bar + 8 * g2, gph2);
                                        if (jb == nb - 1) {
                                            uint32_t s2 = s, ph2 = ph;
                                            ring_next<STAGES>(s2, ph2);
                                            pre_full = mbar_test_wait(full_bar + 8 * s2, ph2);
                                        }
                                    }
                                    const uint64_t ko = (uint64_t)(2 * (jb * SPB + q));     // 32 bytes per step, in 16-byte units
                                    tc_mma_i8_pair(d, a_desc + ko, b_desc + ko, idesc, 1u);   // on top of the offset
                                }
                                tc_commit_pair(tfull_bar + 8 * g, 3);
                                ring_next<GROUPS>(g, gph);
                                ++blk;
                            }
                        }
                        ring_next<STAGES>(s, ph);
                    }
                }
                tc_commit_pair(done_bar, 1);
                mbar_wait(done_bar, 0, abort_flag, p.status, 213, false);
            }
        } else {
            // -------------------------------------------------------------- scale-table builders (warps 2 and 3)
            // Warp 2 builds the tables of the even blocks (accumulator group 0), warp 3 those of the odd blocks
            // (group 1): a single builder made the rescale warps of its sub-partition the last to hand every
            // group back. The table of block b goes to slot b % 4 and its arrival counts on tfull[b % 2]. It is
            // written once the phase of block b - 2 on that barrier is complete: the MMAs of b - 2 were issued
            // only after every rescale warp had finished b - 4, the last reader of the slot, and the barrier is
            // back in the phase that the arrival for b belongs to.
            //
            // Stage hand-back. A commit costs the MMA thread several hundred cycles, so it issues one per block
            // (tfull) and none per stage: each builder arrives once per stage on empty[s] (count 2). A builder
            // with blocks in the stage does so when it sees the tfull phase of its last block there complete,
            // which it waits for anyway at its next block (MMAs complete in order); a builder without a block
            // in the stage arrives at once. Both wait for the stage's exponent slices first: their arrival shows
            // that the producer has consumed the previous phase of empty[s], so an arrival can never fall into it.
            const uint32_t me = (uint32_t)(warp - TABLE_WARP);
            uint32_t s = 0, ph = 0, g = 0, own_ph = 0, slot = me;
            int pend = -1;                 // stage to hand back at this builder's next block
            bool ok = true, out_of_range = false;
            for (int wi = cluster; ok && wi < total_work; wi += nclusters) {
                const Work w = get_work(p, wi);
                const int nst = (w.nblk + BPS - 1) >> LB;
                int left = w.nblk;
                for (int si = 0; ok && si < nst; ++si, left -= BPS) {
                    if (!mbar_wait_warp(efull_bar + 8 * s, ph, abort_flag, p.status, 411)) { ok = false; break; }
                    const unsigned char* eA = base_ptr + (exp_base - base) + s * EXP_STAGE;
                    const unsigned char* eB = eA + EXP_A;
                    bool own_any = false;
#pragma unroll
                    for (int jb = 0; jb < BPS; ++jb) {
                        if (jb < left) {
                            if (g == me) {
                                own_any = true;
                                // this lane's 8 column exponents and 4 row exponents of block jb of the stage
                                const uint2 cb = *reinterpret_cast<const uint2*>(eB + jb * N_TILE + 8 * lane);
                                const uint32_t ra = *reinterpret_cast<const uint32_t*>(eA + jb * TILE_M + 4 * lane);
                                // The split of the scales (rescale_loop): c = SHIFT wherever the block's exponents allow
                                // it, otherwise moved into the window in which every factor and every P * 2^(sA + c - 149)
                                // is a normal binary32 number. The window is empty only when the row exponents of the
                                // block span more than 104 or the true products leave binary32: reported, not computed.
                                const int a_lo = __reduce_min_sync(0xffffffffu, byte_min(ra)), a_hi = __reduce_max_sync(0xffffffffu, byte_max(ra));
                                const int b_lo = __reduce_min_sync(0xffffffffu, byte_min(__vmins4(cb.x, cb.y)));
                                const int b_hi = __reduce_max_sync(0xffffffffu, byte_max(__vmaxs4(cb.x, cb.y)));
                                const int c_lo = max(23 - a_lo, 22 + b_hi), c_hi = min(127 - a_hi, 275 + b_lo);
                                out_of_range |= c_lo > c_hi;
                                const int c = min(max(SHIFT, c_lo), c_hi);
                                uint4 c0, c1, r0;
                                // the two pairs of every four column factors are stored crossed (columns 2 3 0 1): see rescale_loop
                                c0.z = exp_to_scale(cb.x, 0, 149 - c); c0.w = exp_to_scale(cb.x, 1, 149 - c); c0.x = exp_to_scale(cb.x, 2, 149 - c); c0.y = exp_to_scale(cb.x, 3, 149 - c);
                                c1.z = exp_to_scale(cb.y, 0, 149 - c); c1.w = exp_to_scale(cb.y, 1, 149 - c); c1.x = exp_to_scale(cb.y, 2, 149 - c); c1.y = exp_to_scale(cb.y, 3, 149 - c);
                                r0.x = exp_to_scale(ra, 0, c); r0.y = exp_to_scale(ra, 1, c); r0.z = exp_to_scale(ra, 2, c); r0.w = exp_to_scale(ra, 3, c);
                                if (!mbar_wait_warp(tfull_bar + 8 * me, own_ph ^ 1, abort_flag, p.status, 412)) { ok = false; break; }
                                if (pend >= 0 && lane == 0) mbar_arrive(empty_bar + 8 * pend);   // this builder's previous block is complete
                                pend = (jb + 2 >= BPS || jb + 2 >= left) ? (int)s : -1;          // its last block of this stage?
                                uint32_t* tb = tables + slot * TABLE_SLOT_WORDS;
                                *reinterpret_cast<uint4*>(tb + 8 * lane) = c0;
                                *reinterpret_cast<uint4*>(tb + 8 * lane + 4) = c1;
                                *reinterpret_cast<uint4*>(tb + N_TILE + 4 * lane) = r0;
                                __syncwarp();
                                if (lane == 0) mbar_arrive(tfull_bar + 8 * me);
                                own_ph ^= 1u;
                                slot = (slot + 2) & (TSLOTS - 1);
                            }
                            g ^= 1u;
                        }
                    }
                    if (!ok) break;
                    if (!own_any && lane == 0) mbar_arrive(empty_bar + 8 * s);     // nothing of this builder's in the stage
                    ring_next<STAGES>(s, ph);
                }
            }
            if (out_of_range) atomicCAS(p.status, 0, STATUS_EXPONENT_RANGE);
        }
    } else {
        // ------------------------------------------------------------------ rescale warps (both CTAs)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_RESCALE));
        const RescaleArgs ra{tfull_bar, map_to_rank(tempty_bar, 0), tmem_base, tables, total_work, cluster, nclusters, rank, abort_flag};
        const int rwarp = warp - CONTROL_WARPS, part = rwarp >> 2;     // warps that share a lane quarter split the columns
        if (part == 2) rescale_loop<80, 8>(p, ra, 176);
        else rescale_loop<88, 8>(p, ra, part * 88);
    }

    // ------------------------------------------------------------------ teardown
    // Neither CTA may leave while the other can still signal its barriers or read its shared memory.
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && blockIdx.x < MAX_CTAS) g_cta_cycles[blockIdx.x] = (unsigned long long)(clock64() - cycles_start);
    cluster_barrier();
    if (warp == MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// Largest number of co-resident clusters on the current device (0: not known yet, -1: the query failed).
int max_clusters() {
    static int n[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return -1;
    if (!n[dev]) {
        // the attribute belongs to the device: set once per device, before the occupancy query that needs it
        if (cudaFuncSetAttribute(gemm_tc2_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gemm_tc2_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gemm_tc2_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess) {
            cudaGetLastError();
            n[dev] = -1;
            return -1;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 148, 1, 1);
        cfg.blockDim = dim3(THREADS, 1, 1);
        cfg.dynamicSmemBytes = SMEM;
        int c = 0;
        if (cudaOccupancyMaxActiveClusters(&c, gemm_tc2_kernel<0>, &cfg) != cudaSuccess || c < 1) {
            cudaGetLastError();
            c = -1;
        }
        n[dev] = c;
    }
    return n[dev];
}

int g_last_ctas[MAX_DEVICES] = {};     // CTAs of the last launch, per device

}  // namespace

int pair_gemm_cycles(uint64_t* cycles) {
    unsigned long long host[MAX_CTAS];
    const int dev = current_device();
    const int n = dev >= 0 ? g_last_ctas[dev] : 0;
    *cycles = 0;
    if (n <= 0) return HBFP_OK;
    HBFP_CUDA_OK(cudaDeviceSynchronize());
    HBFP_CUDA_OK(cudaMemcpyFromSymbol(host, g_cta_cycles, sizeof(unsigned long long) * n));
    unsigned long long m = 0;
    for (int i = 0; i < n; ++i) m = host[i] > m ? host[i] : m;
    *cycles = m;
    return HBFP_OK;
}

bool pair_gemm_eligible(int64_t M, int64_t N, const Packed& a, const Packed& b, const TensorPlan& plan) {
    if (a.L.planes != 1 || b.L.planes != 1) return false;
    if (a.L.bp > 128 || plan.n_tile != 256) return false;
    const int64_t qa = (1ll << (a.mant_bits - 1)) - 1, qb = (1ll << (b.mant_bits - 1)) - 1;
    if (qa * qb * a.L.b >= OFFSET) return false;             // the offset keeps OFFSET + P positive
    if (plan.splits != 1) return false;
    // enough pair tiles to occupy every SM pair
    const int64_t tiles = ((M + PAIR_M - 1) / PAIR_M) * ((N + N_TILE - 1) / N_TILE);
    return tiles >= 74 && max_clusters() >= 1;
}

int launch_gemm_tensor_pair(int64_t M, int64_t N, const Packed& a, const Packed& b, float* Cout, int64_t ldc,
                            const TensorPlan& plan, void* partial, cudaStream_t st) {
    Problem p{};
    p.M = M;
    p.N = N;
    p.nkb = a.L.nkb;
    p.bp = (int)a.L.bp;
    p.tiles_m = (int)((M + PAIR_M - 1) / PAIR_M);
    p.tiles_n = (int)((N + N_TILE - 1) / N_TILE);
    p.splits = plan.splits;
    p.kb_per_split = plan.kb_per_split;
    p.C = Cout;
    p.ldc = ldc;
    p.partial = static_cast<float*>(partial);
    p.ldp = round_up(N, 4);
    p.status = device_status_word();
    if (!p.status) return HBFP_ERR_CUDA;
    if (p.splits > 1 && !partial) return HBFP_ERR_WORKSPACE;
    CUtensorMap mA, mB, mEA, mEB;
    int rc;
    rc = make_map(&mA, a.mant, a.L.kst, a.L.rows, a.L.kst, STAGE_K, TILE_M, true);
    if (rc) return rc;
    rc = make_map(&mB, b.mant, b.L.kst, b.L.rows, b.L.kst, STAGE_K, B_HALF, true);
    if (rc) return rc;
    rc = make_map(&mEA, a.exps, a.L.rs, a.L.nkb, a.L.rs, TILE_M, 4, false);
    if (rc) return rc;
    rc = make_map(&mEB, b.exps, b.L.rs, b.L.nkb, b.L.rs, N_TILE, 4, false);
    if (rc) return rc;
    const int clusters_max = max_clusters();
    if (clusters_max < 1) return HBFP_ERR_UNSUPPORTED;
    const int64_t work = (int64_t)p.tiles_m * p.tiles_n * p.splits;
    const int clusters = (int)(work < clusters_max ? work : clusters_max);
    static_assert(2 * 148 <= MAX_CTAS, "cycle stamps");
    if (2 * clusters > MAX_CTAS) return HBFP_ERR_UNSUPPORTED;
    {
        const int dev = current_device();
        if (dev >= 0) g_last_ctas[dev] = 2 * clusters;     // the stamps that pair_gemm_cycles may read
    }
    if (p.bp == 128) gemm_tc2_kernel<0><<<2 * clusters, THREADS, SMEM, st>>>(mA, mB, mEA, mEB, p);
    else if (p.bp == 64) gemm_tc2_kernel<1><<<2 * clusters, THREADS, SMEM, st>>>(mA, mB, mEA, mEB, p);
    else gemm_tc2_kernel<2><<<2 * clusters, THREADS, SMEM, st>>>(mA, mB, mEA, mEB, p);
    return launch_status();
}

}  // namespace hbfp
