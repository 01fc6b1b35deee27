// HBFP oracle: a plain, slow, obviously-correct CPU statement of block-floating-point
// quantisation and of the BFP matrix product.
//
// THIS IS TEST INFRASTRUCTURE. Only the test-suite, the smoke check and the CPU-baseline
// leg of the benchmark may build, load or call it. It shares no source, header, table or
// helper with the CUDA library and is never a fallback for it.
//
// Every function follows one passage of the paper (Drumond et al., "Training DNNs with
// Hybrid Block Floating Point"):
//   * format            : Eq. 1 (value = mantissa * 2^exponent, one exponent per block)
//   * exponent choice   : Sec. 4.1 ("the exponent of the largest tensor value") and Sec. 5.3
//                         (the FP-to-BFP unit detects the maximum exponent, normalises mantissas)
//   * rounding          : Sec. 5.3 (stochastic rounding at mantissa truncation); nearest-even
//                         is the second mode of this build
//   * dot product       : Eq. 2 (integer dot product of mantissas, scaled by 2^(ea+eb))
//   * tiled product     : Sec. 4 after Eq. 2 and Sec. 4.2 "Tiling" (tile products in fixed
//                         point, tiles accumulated in floating point)
//   * wide weight storage: Sec. 4.2 (16-bit long-lived mantissas, the passes read the top bits)
// Arithmetic is double / int64 throughout; nothing is blocked, fused or reordered.
//
// Pins (tests/test_oracle_*.py): exact-rational brute force of exponent + nearest rounding,
// a float64 numpy restatement, idempotence, exact pass-through, power-of-two equivariance,
// sign symmetry, half-ULP / one-ULP error bounds, exhaustive stochastic-rounding mean,
// published Philox4x32-10 known answers, Eq. 2 against a float64 matmul of de-quantised
// operands, exact-rational sums on tiny shapes and closed forms; wide storage: the half-ULP
// bracket in exact rationals, the absence of a systematic offset, agreement with direct quantisation on narrow-representable
// weights, idempotence of the zero update, a binary32 numpy restatement of the update and
// exact integer steps. No function here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// Mirrors the fields of the library's format descriptor; declared separately on purpose.
struct oracle_format {
    int32_t mant_bits;   // m: sign + (m-1) magnitude bits
    int32_t block;       // b: 1-D block length along the contraction axis; 0 = whole axis
    int32_t tile;        // t: 0 = 1-D blocks, t > 0 = t x t tiles of the stored matrix
    int32_t rounding;    // 0 = round to nearest, ties to even; 1 = stochastic (16 random bits)
    int32_t exp_mode;    // 0 = floor(log2 amax)+1 ; 1 = literal ceil(log2 amax)
    uint32_t stream_id;  // third counter word of the random stream
    uint64_t seed;       // Philox key
    // Position of the passed view inside the caller's logical tensor (for the random
    // counter only): element (i,j) of the view has linear index (i+row_off)*idx_cols+(j+col_off).
    int64_t idx_row_off, idx_col_off, idx_cols;
};

int oracle_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
// SC'11): ten rounds; each round multiplies counter words 0 and 2 by two fixed odd
// constants, xors the high halves with the other two words and the key, and the key is
// advanced by two Weyl constants between rounds.
// ---------------------------------------------------------------------------------------
void oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    const uint64_t MUL_A = 0xD2511F53ull, MUL_B = 0xCD9E8D57ull;
    const uint32_t WEYL_A = 0x9E3779B9u, WEYL_B = 0xBB67AE85u;
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t pa = MUL_A * (uint64_t)c0;
        uint64_t pb = MUL_B * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(pb >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)pb;
        uint32_t n2 = (uint32_t)(pa >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)pa;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += WEYL_A; k1 += WEYL_B;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The 16-bit draw of element L: one Philox call serves the 8 elements that share L >> 3;
// word (L & 7) >> 1, low half for even L, high half for odd L.
uint32_t oracle_sr_draw(uint64_t seed, uint32_t stream_id, uint64_t L) {
    uint64_t g = L >> 3;
    uint32_t ctr[4] = {(uint32_t)g, (uint32_t)(g >> 32), stream_id, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    oracle_philox4x32_10(ctr, key, w);
    uint32_t word = w[(L & 7) >> 1];
    return (word >> (16 * (L & 1))) & 0xFFFFu;
}

// ---------------------------------------------------------------------------------------
// Shared exponent of a block from its largest magnitude (Sec. 4.1 / Sec. 5.3).
// Returns the exponent s of the mantissa LSB: a mantissa q stands for q * 2^s (Eq. 1).
// ---------------------------------------------------------------------------------------
int oracle_block_exponent(double amax, int mant_bits, int exp_mode) {
    const int floor_s = -63;
    if (!(amax > 0.0)) return floor_s;              // all-zero block
    int ex;
    double frac = std::frexp(amax, &ex);            // amax = frac * 2^ex, frac in [0.5, 1)
    int e = ex;                                     // floor(log2 amax) + 1
    if (exp_mode == 1 && frac == 0.5) e = ex - 1;   // literal ceil(log2 amax) at exact powers of two
    int s = e - (mant_bits - 1);
    return s < floor_s ? floor_s : s;
}

static inline int64_t clamp_q(int64_t q, int mant_bits) {
    int64_t qmax = ((int64_t)1 << (mant_bits - 1)) - 1;
    if (q > qmax) return qmax;
    if (q < -qmax) return -qmax;
    return q;
}

// Round to nearest, ties to even: q = clamp(rne(x * 2^-s)).
int32_t oracle_round_rne(float x, int s, int mant_bits) {
    double y = std::ldexp((double)x, -s);           // exact: a power-of-two scaling in double
    double r = std::nearbyint(y);                   // default rounding mode = ties to even
    if (!(r == r)) return 0;
    if (r > 1e18) r = 1e18;
    if (r < -1e18) r = -1e18;
    return (int32_t)clamp_q((int64_t)r, mant_bits);
}

// Stochastic rounding with 16 random bits r in [0, 65536):
//   Y = floor( binary32( x * 2^(16-s) ) ),  q = clamp( floor((Y + r) / 65536) ).
int32_t oracle_round_sr(float x, int s, int mant_bits, uint32_t r) {
    double yd = std::ldexp((double)x, 16 - s);      // exact in double
    float yf = (float)yd;                           // the binary32 product (rounds only if subnormal)
    if (!(yf == yf)) return 0;
    double fl = std::floor((double)yf);
    if (fl > 1e18) fl = 1e18;
    if (fl < -1e18) fl = -1e18;
    int64_t Y = (int64_t)fl;
    int64_t t = Y + (int64_t)r;
    int64_t q = t >= 0 ? t / 65536 : -((-t + 65535) / 65536);   // floor division
    return (int32_t)clamp_q(q, mant_bits);
}

// ---------------------------------------------------------------------------------------
// Quantise a logical [d0][d1] binary32 matrix (row stride ld) with blocks along
// contract_axis. Output is canonical: q[rows][k] (int16) and s[rows][nkb] (int8) with
// k = extent of the contraction axis, rows = the other extent, nkb = ceil(k / b).
// With tile t > 0 one exponent serves each t x t tile of the stored matrix (Sec. 4.2
// "Tiling"), and s[r][kb] repeats the exponent of the tile that element (r, kb*t) lies in,
// so W and its transpose see the same mantissas and exponents.
// Returns 0, or a negative number for a bad argument.
// ---------------------------------------------------------------------------------------
int oracle_quantize(const float* x, int64_t d0, int64_t d1, int64_t ld, int contract_axis,
                    const oracle_format* f, int16_t* q, int8_t* s) {
    if (!x || !f || !q || !s || d0 < 0 || d1 < 0 || ld < d1) return -1;
    if (contract_axis != 0 && contract_axis != 1) return -1;
    const int m = f->mant_bits;
    if (m < 2 || m > 16) return -2;
    if (f->tile < 0 || f->block < 0) return -2;
    if (f->tile > 0 && f->block != f->tile) return -2;
    const int64_t k = contract_axis == 1 ? d1 : d0;
    const int64_t rows = contract_axis == 1 ? d0 : d1;
    const int64_t b = f->block == 0 ? (k > 0 ? k : 1) : f->block;
    const int64_t nkb = (k + b - 1) / b;
    const int64_t idx_cols = f->idx_cols > 0 ? f->idx_cols : d1;

    auto src = [&](int64_t r, int64_t kk) -> float {
        return contract_axis == 1 ? x[r * ld + kk] : x[kk * ld + r];
    };
    auto lin = [&](int64_t r, int64_t kk) -> uint64_t {
        int64_t i = contract_axis == 1 ? r : kk, j = contract_axis == 1 ? kk : r;
        return (uint64_t)((i + f->idx_row_off) * idx_cols + (j + f->idx_col_off));
    };

    // Pass 1: exponent of every block (or tile).
    if (f->tile == 0) {
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t kb = 0; kb < nkb; ++kb) {
                double amax = 0.0;
                int64_t k1 = (kb + 1) * b < k ? (kb + 1) * b : k;
                for (int64_t kk = kb * b; kk < k1; ++kk) {
                    double a = std::fabs((double)src(r, kk));
                    if (a > amax) amax = a;
                }
                s[r * nkb + kb] = (int8_t)oracle_block_exponent(amax, m, f->exp_mode);
            }
    } else {
        const int64_t t = f->tile;
        const int64_t nrt = (rows + t - 1) / t;
#pragma omp parallel for schedule(static)
        for (int64_t rt = 0; rt < nrt; ++rt)
            for (int64_t kb = 0; kb < nkb; ++kb) {
                double amax = 0.0;
                int64_t r1 = (rt + 1) * t < rows ? (rt + 1) * t : rows;
                int64_t k1 = (kb + 1) * t < k ? (kb + 1) * t : k;
                for (int64_t r = rt * t; r < r1; ++r)
                    for (int64_t kk = kb * t; kk < k1; ++kk) {
                        double a = std::fabs((double)src(r, kk));
                        if (a > amax) amax = a;
                    }
                int8_t se = (int8_t)oracle_block_exponent(amax, m, f->exp_mode);
                for (int64_t r = rt * t; r < r1; ++r) s[r * nkb + kb] = se;
            }
    }

    // Pass 2: mantissas.
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t kk = 0; kk < k; ++kk) {
            int se = s[r * nkb + kk / b];
            float v = src(r, kk);
            int32_t qq;
            if (f->rounding == 0) {
                qq = oracle_round_rne(v, se, m);
            } else {
                uint32_t rnd = oracle_sr_draw(f->seed, f->stream_id, lin(r, kk));
                qq = oracle_round_sr(v, se, m, rnd);
            }
            q[r * k + kk] = (int16_t)qq;
        }
    return 0;
}

// ---------------------------------------------------------------------------------------
// oracle_quantize for a matrix whose elements are copies of the elements of another tensor (the im2col
// matrix of a convolution, Sec. 5.1): exactly the same two passes, but under stochastic rounding element
// (i, j) takes the draw of index[i * d1 + j] - its position in the tensor it was copied from - so that every
// copy of an activation uses that activation's draw; a negative index marks a structural zero (padding),
// which needs no draw. With index[i * d1 + j] = i * d1 + j this is oracle_quantize.
// ---------------------------------------------------------------------------------------
int oracle_quantize_indexed(const float* x, int64_t d0, int64_t d1, int64_t ld, int contract_axis,
                            const oracle_format* f, const int64_t* index, int16_t* q, int8_t* s) {
    if (!index) return -1;
    oracle_format g = *f;
    g.rounding = 0;                                   // pass 1 (exponents) does not depend on the rounding mode
    int rc = oracle_quantize(x, d0, d1, ld, contract_axis, &g, q, s);
    if (rc || f->rounding == 0) return rc;
    const int m = f->mant_bits;
    const int64_t k = contract_axis == 1 ? d1 : d0, rows = contract_axis == 1 ? d0 : d1;
    const int64_t b = f->block == 0 ? (k > 0 ? k : 1) : f->block, nkb = (k + b - 1) / b;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t kk = 0; kk < k; ++kk) {
            const int64_t i = contract_axis == 1 ? r : kk, j = contract_axis == 1 ? kk : r;
            const int64_t L = index[i * d1 + j];
            const uint32_t rnd = L < 0 ? 0u : oracle_sr_draw(f->seed, f->stream_id, (uint64_t)L);
            q[r * k + kk] = (int16_t)oracle_round_sr(x[i * ld + j], s[r * nkb + kk / b], m, rnd);
        }
    return 0;
}

// ---------------------------------------------------------------------------------------
// Weights of a convolution layer (Sec. 5.1, last sentence: for convolutional layers the two outer,
// feature-map dimensions of the weights are tiled). The weights are w[tap][ci][co], tap = (filter row,
// filter column), stored as the matrix [taps * c_in][c_out] that the convolution GEMM multiplies by.
// Reading taken: a tile is t input maps x t output maps and spans every filter tap, so all
// kh * kw * t * t weights of a tile share one exponent (the filter dimensions are not tiled):
//   E[u][v] = exponent of max |w[tap][ci][co]| over all taps, ci in [u t, (u+1) t), co in [v t, (v+1) t)
// Every weight is then rounded on its tile's grid exactly as in oracle_quantize. Output in the
// canonical layout of that function for the same contraction axis: axis 0 (forward: contraction over
// (tap, ci)) q [c_out][taps * c_in], s [c_out][taps * c_in / t]; axis 1 (backward-data: contraction over
// co) q [taps * c_in][c_out], s [taps * c_in][ceil(c_out / t)]. Needs f->tile == f->block == t > 0 and
// c_in % t == 0 (a K-block never straddles two taps). Returns 0, -1 bad arguments, -2 bad format.
// ---------------------------------------------------------------------------------------
int oracle_quantize_conv_weights(const float* w, int64_t taps, int64_t c_in, int64_t c_out, int64_t ld,
                                 int contract_axis, const oracle_format* f, int16_t* q, int8_t* s) {
    if (!w || !f || !q || !s || taps <= 0 || c_in <= 0 || c_out <= 0 || ld < c_out) return -1;
    if (contract_axis != 0 && contract_axis != 1) return -1;
    const int m = f->mant_bits;
    if (m < 2 || m > 16) return -2;
    const int64_t t = f->tile;
    if (t <= 0 || f->block != t || c_in % t != 0) return -2;
    const int64_t nu = c_in / t, nv = (c_out + t - 1) / t;
    const int64_t d0 = taps * c_in, d1 = c_out;
    const int64_t idx_cols = f->idx_cols > 0 ? f->idx_cols : d1;
    // Pass 1: one exponent per (input-map tile, output-map tile), over all taps.
    std::vector<int> E((size_t)(nu * nv));
    for (int64_t u = 0; u < nu; ++u)
        for (int64_t v = 0; v < nv; ++v) {
            double amax = 0.0;
            const int64_t co1 = (v + 1) * t < c_out ? (v + 1) * t : c_out;
            for (int64_t tap = 0; tap < taps; ++tap)
                for (int64_t ci = u * t; ci < (u + 1) * t; ++ci)
                    for (int64_t co = v * t; co < co1; ++co) {
                        double a = std::fabs((double)w[(tap * c_in + ci) * ld + co]);
                        if (a > amax) amax = a;
                    }
            E[(size_t)(u * nv + v)] = oracle_block_exponent(amax, m, f->exp_mode);
        }
    // Pass 2: mantissas and the canonical exponent array.
    const int64_t nkb0 = d0 / t;
    for (int64_t i = 0; i < d0; ++i)
        for (int64_t j = 0; j < d1; ++j) {
            const int64_t ci = i % c_in;
            const int se = E[(size_t)((ci / t) * nv + j / t)];
            const float v = w[i * ld + j];
            int32_t qq;
            if (f->rounding == 0) {
                qq = oracle_round_rne(v, se, m);
            } else {
                uint32_t rnd = oracle_sr_draw(f->seed, f->stream_id, (uint64_t)((i + f->idx_row_off) * idx_cols + (j + f->idx_col_off)));
                qq = oracle_round_sr(v, se, m, rnd);
            }
            if (contract_axis == 0) {
                q[j * d0 + i] = (int16_t)qq;
                s[j * nkb0 + i / t] = (int8_t)se;
            } else {
                q[i * d1 + j] = (int16_t)qq;
                s[i * nv + j / t] = (int8_t)se;
            }
        }
    return 0;
}

// ---------------------------------------------------------------------------------------
// BFP matrix product of two canonically quantised operands (Eq. 2 applied per block, blocks
// accumulated in floating point):
//   P[i][j][kb] = sum_{k in block kb} qA[i][k] * qB[j][k]                (integers, exact)
//   T           = binary32(P) * 2^(sA[i][kb] + sB[j][kb])
//   c_ref[i][j] = binary32( sum_kb T in double ),  a_mag[i][j] = sum_kb |T|
//   c_seq[i][j] = binary32 accumulation of T in ascending kb, one rounding per step
// qA is [M][K], qB is [N][K] (both contraction-major), sA [M][nkb], sB [N][nkb].
// Any of c_ref, a_mag, c_seq, P may be null. exact_p != 0 keeps P unrounded in c_ref/a_mag
// (isolates the one rounding of binary32(P) for wide mantissas).
// Returns 0; -3 if some P does not fit int32; -1 on bad arguments.
// ---------------------------------------------------------------------------------------
int oracle_gemm(int64_t M, int64_t N, int64_t K, int64_t block,
                const int16_t* qA, const int8_t* sA, const int16_t* qB, const int8_t* sB,
                float* c_ref, double* a_mag, float* c_seq, int32_t* P, int exact_p) {
    if (M < 0 || N < 0 || K < 0 || block < 0 || !qA || !sA || !qB || !sB) return -1;
    const int64_t b = block == 0 ? (K > 0 ? K : 1) : block;
    const int64_t nkb = (K + b - 1) / b;
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            double sum = 0.0, mag = 0.0;
            float seq = 0.0f;
            for (int64_t kb = 0; kb < nkb; ++kb) {
                int64_t k1 = (kb + 1) * b < K ? (kb + 1) * b : K;
                int64_t p = 0;
                for (int64_t kk = kb * b; kk < k1; ++kk)
                    p += (int64_t)qA[i * K + kk] * (int64_t)qB[j * K + kk];
                if (p > INT32_MAX || p < INT32_MIN) overflow = 1;
                if (P) P[(i * N + j) * nkb + kb] = (int32_t)p;
                int e = (int)sA[i * nkb + kb] + (int)sB[j * nkb + kb];
                float pf = (float)p;                          // round to nearest even
                double t = std::ldexp(exact_p ? (double)p : (double)pf, e);
                sum += t;
                mag += std::fabs(t);
                float tf = std::ldexp(pf, e);                 // exact while 2^e*|pf| is a normal binary32
                volatile float next = seq + tf;               // one binary32 rounding
                seq = next;
            }
            if (c_ref) c_ref[i * N + j] = (float)sum;
            if (a_mag) a_mag[i * N + j] = mag;
            if (c_seq) c_seq[i * N + j] = seq;
        }
    return overflow ? -3 : 0;
}

// ---------------------------------------------------------------------------------------
// The whole dot-product path on binary32 operands: quantise op(A) and op(B) along the
// contraction axis ("convert tensors to BFP before every dot product", Sec. 4.1), then the
// BFP product. A is [M][K] (transA = 0) or [K][M] (transA = 1); B is [K][N] (transB = 0) or
// [N][K] (transB = 1). forward = (0,0), backward-data = (0,1), backward-weight = (1,0).
// ---------------------------------------------------------------------------------------
int oracle_hbfp_gemm(int transA, int transB, int64_t M, int64_t N, int64_t K,
                     const float* A, int64_t lda, const float* B, int64_t ldb,
                     const oracle_format* fA, const oracle_format* fB,
                     float* c_ref, double* a_mag, float* c_seq) {
    if (!fA || !fB) return -1;
    int64_t bA = fA->block == 0 ? (K > 0 ? K : 1) : fA->block;
    int64_t bB = fB->block == 0 ? (K > 0 ? K : 1) : fB->block;
    if (bA != bB) return -2;                       // blocks of the two operands must coincide
    int64_t nkb = (K + bA - 1) / bA;
    std::vector<int16_t> qA((size_t)(M * K)), qB((size_t)(N * K));
    std::vector<int8_t> sA((size_t)(M * nkb)), sB((size_t)(N * nkb));
    int rc;
    // op(A) is M x K: stored [M][K] -> contraction is axis 1; stored [K][M] -> axis 0.
    rc = transA ? oracle_quantize(A, K, M, lda, 0, fA, qA.data(), sA.data())
                : oracle_quantize(A, M, K, lda, 1, fA, qA.data(), sA.data());
    if (rc) return rc;
    // op(B) is K x N: stored [K][N] -> contraction is axis 0; stored [N][K] -> axis 1.
    rc = transB ? oracle_quantize(B, N, K, ldb, 1, fB, qB.data(), sB.data())
                : oracle_quantize(B, K, N, ldb, 0, fB, qB.data(), sB.data());
    if (rc) return rc;
    return oracle_gemm(M, N, K, bA, qA.data(), sA.data(), qB.data(), sB.data(),
                       c_ref, a_mag, c_seq, nullptr, 0);
}

// ---------------------------------------------------------------------------------------
// Wide weight storage (Sec. 4.2): the long-lived copy of a weight matrix keeps 16-bit
// mantissas (one exponent per t x t tile); forward and backward passes read only the m most
// significant bits of each stored word. Plain truncation of the two's-complement mantissa would
// make every narrow weight half a narrow ULP too small on average, a bias that adds up coherently
// over a dot product with same-signed activations; the stored word is therefore the mantissa plus
// half a narrow ULP, so that its top m bits are the mantissa rounded to nearest (ties upward),
// which is also what the paper's simulation feeds the passes (the weights rounded to the narrow
// format, Sec. 5.1). In canonical arrays:
//   narrow mantissa = clamp( floor((q16 + 2^(15-m)) / 2^(16-m)), +-(2^(m-1) - 1) )
//   narrow exponent = s16 + (16 - m)            (the weight of the narrow LSB)
// so the narrow value lies within half a narrow ULP of the wide one (one ULP where it saturates).
// n_q mantissas, n_s exponents. Returns 0; -2 for m outside [2, 16].
// ---------------------------------------------------------------------------------------
int oracle_wide_narrow(const int16_t* q16, const int8_t* s16, int64_t n_q, int64_t n_s, int m,
                       int16_t* qm, int8_t* sm) {
    if (!q16 || !s16 || !qm || !sm || n_q < 0 || n_s < 0) return -1;
    if (m < 2 || m > 16) return -2;
    const int64_t d = (int64_t)1 << (16 - m);
    const int64_t half = d / 2;                                  // 0 when m = 16
    for (int64_t i = 0; i < n_q; ++i) {
        int64_t v = (int64_t)q16[i] + half;
        int64_t fl = v >= 0 ? v / d : -((-v + d - 1) / d);      // floor division
        qm[i] = (int16_t)clamp_q(fl, m);
    }
    for (int64_t i = 0; i < n_s; ++i) sm[i] = (int8_t)(s16[i] + (16 - m));
    return 0;
}

// ---------------------------------------------------------------------------------------
// Weight update on wide storage (Sec. 4.2 "only weight updates use the wider mantissa";
// Sec. 5.1: the update itself is computed in FP32, then the weights are converted back):
//   w[i][j] = binary32( q16[i][j] * 2^s16 + delta[i][j] )      (q16 * 2^s16 is exact in binary32)
//   (q16, s16) = 16-bit quantisation of w with one exponent per t x t tile of the stored matrix
// q16 is [d0][d1], s16 is canonical [d0][ceil(d1/t)] (each row repeats its tile's exponent),
// delta is [d0][d1] with row stride ldd. f gives tile (= block), rounding, exponent rule and
// random stream; f->mant_bits is ignored (the wide width is 16). Returns what oracle_quantize returns.
// ---------------------------------------------------------------------------------------
int oracle_wide_update(int16_t* q16, int8_t* s16, const float* delta, int64_t ldd, int64_t d0, int64_t d1,
                       const oracle_format* f) {
    if (!q16 || !s16 || !delta || !f || d0 < 0 || d1 < 0 || ldd < d1) return -1;
    if (f->tile <= 0 || f->block != f->tile) return -2;
    const int64_t t = f->tile, nkb = (d1 + t - 1) / t;
    std::vector<float> w((size_t)(d0 * d1));
    for (int64_t i = 0; i < d0; ++i)
        for (int64_t j = 0; j < d1; ++j) {
            volatile float dq = std::ldexp((float)q16[i * d1 + j], (int)s16[i * nkb + j / t]);
            volatile float sum = dq + delta[i * ldd + j];       // one binary32 rounding
            w[(size_t)(i * d1 + j)] = sum;
        }
    oracle_format f16 = *f;
    f16.mant_bits = 16;
    return oracle_quantize(w.data(), d0, d1, d1, 1, &f16, q16, s16);
}

}  // extern "C"
