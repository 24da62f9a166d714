/*
 * CPU oracle for one step of distributed SGD with random block-wise gradient
 * sparsification (RBGS) under error feedback: EF, DEF and DEF-A of
 * "Detached Error Feedback for Distributed SGD with Random Sparsification".
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded statement
 * of what the method computes, written from the paper so that it can be checked
 * against the paper by eye.  It shares no code with the CUDA library and is never
 * on the product path: only the tests, the smoke check and the CPU-baseline leg
 * of the benchmark may call it.
 *
 * Notation follows the paper: K workers are the W rows here, x the model,
 * g_{k,t} the stochastic gradient, e_{k,t} the local compression error,
 * m_{k,t} the momentum buffer, p_{k,t} the error-compensated vector, C the
 * compressor, eta the learning rate, mu the momentum constant, lambda the
 * detach coefficient.  The block length (no symbol in the paper) is k, the
 * block start is s, and delta = k/d.
 *
 * "Column view": every array function works on n columns of a d-dimensional
 * problem.  Column i of the view is coordinate cols[i] of the model
 * (cols == NULL means the identity, coordinate i).  A whole step is n == d with
 * cols == NULL; a view lets a test follow a sample of coordinates of a problem
 * that is too large to run whole.  Every operation of the method is separate
 * per coordinate, so the view changes nothing in the arithmetic.
 *
 * The float functions come in two precisions built from the same text
 * (def_oracle_body.inc): _f32 rounds like the fp32 product (one fused
 * multiply-add per update, workers summed left to right, IEEE division by W),
 * _f64 is the high-precision shadow the fp32 results are compared with.
 *
 * Pins (tests/test_oracle_*.py): hand-worked 8-coordinate example, the
 * telescoping identity of Eq. 8 with and without momentum (Eq. 10), k = d
 * against plain momentum SGD (Eq. 2), C(p) + e' = p (Algorithm 1), additivity
 * (Assumption 3), delta = k/d over all d starts (Assumption 5 and the remark
 * under it), K = 1 / lambda = 1 SGD path, the iterate-averaging closed form of
 * Eq. 11, and the Philox generator against an independent library engine.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

enum { DEF_ORACLE_COMPRESSOR_RBGS = 0, DEF_ORACLE_COMPRESSOR_SCALE = 1 };
enum { DEF_ORACLE_VARIANT_DEF = 0, DEF_ORACLE_VARIANT_DEF_A = 1, DEF_ORACLE_VARIANT_EF = 2 };

/* ------------------------------------------------------------------------
 * Shared random block start (Section 1: every worker holds the same seed and
 * draws one uniformly random start index per iteration, cost O(1)).
 *
 * The paper names no generator.  The reading taken here: Philox4x32-10
 * (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
 * SC'11), a counter-based generator, so the start of step t is a pure function
 * of (seed, t) and needs no state.
 * ---------------------------------------------------------------------- */

/* One Philox4x32 bijection of `rounds` rounds.  A round multiplies counter
 * words 0 and 2 by two fixed odd constants, keeps both halves of each 64-bit
 * product, and mixes the high halves with the other two words and the key;
 * the key is bumped by the Weyl constants between rounds. */
void def_oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], int rounds,
                           uint32_t out[4])
{
    const uint32_t MUL0 = 0xD2511F53u, MUL1 = 0xCD9E8D57u;
    const uint32_t WEYL0 = 0x9E3779B9u, WEYL1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < rounds; ++r) {
        if (r > 0) { k0 += WEYL0; k1 += WEYL1; }
        uint64_t prod0 = (uint64_t)MUL0 * c0;
        uint64_t prod1 = (uint64_t)MUL1 * c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Start index s_t in [0, d): key = seed, counter = (t, domain tag "RBGS", 0);
 * the first two output words form a 64-bit r, and s = floor(r * d / 2^64).
 * The map is uniform up to a bias below d / 2^64. */
int64_t def_oracle_block_start(uint64_t seed, uint64_t step, int64_t d)
{
    uint32_t ctr[4] = { (uint32_t)step, (uint32_t)(step >> 32), 0x52424753u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    def_oracle_philox4x32(ctr, key, 10, out);
    uint64_t r = (uint64_t)out[0] | ((uint64_t)out[1] << 32);
    unsigned __int128 wide = (unsigned __int128)r * (unsigned __int128)(uint64_t)d;
    return (int64_t)(uint64_t)(wide >> 64);
}

/* Is coordinate j one of the k block coordinates {(s + i) mod d : 0 <= i < k}?
 * The paper says only "a block of gradient" from one random start; the block
 * wraps around the end of the flat vector, which is the one reading under which
 * every coordinate is kept with probability exactly k/d, as Assumption 5's
 * remark (delta equal to the compression ratio) and the proofs' E_C C(v) =
 * delta v require. */
int def_oracle_in_block(int64_t j, int64_t s, int64_t k, int64_t d)
{
    int64_t offset = j - s;
    if (offset < 0) offset += d;
    return offset < k;
}

/* 0/1 mask of the block over a column view. */
void def_oracle_block_mask(int64_t d, int64_t k, int64_t s, int64_t n, const int64_t *cols,
                           uint8_t *mask)
{
    for (int64_t i = 0; i < n; ++i) {
        int64_t j = cols ? cols[i] : i;
        mask[i] = (uint8_t)def_oracle_in_block(j, s, k, d);
    }
}

/* Loops over coordinates: serial here; a parallel-for in the all-cores build (see the body). */
#ifdef _OPENMP
#define FOR_EACH_COORDINATE _Pragma("omp parallel for schedule(static)")
#else
#define FOR_EACH_COORDINATE
#endif

#define REAL float
#define FMA fmaf
#define NAME(base) base##_f32
#include "def_oracle_body.inc"
#undef REAL
#undef FMA
#undef NAME

#define REAL double
#define FMA fma
#define NAME(base) base##_f64
#include "def_oracle_body.inc"
#undef REAL
#undef FMA
#undef NAME

/* Threads the coordinate loops run on: 1 in the plain build. */
int def_oracle_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
