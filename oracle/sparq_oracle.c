/*
 * CPU oracle for the SPARQ hot path (arXiv 2105.11010) -- TEST INFRASTRUCTURE.
 *
 * A plain, slow, byte-at-a-time restatement of what the paper defines.  It is
 * only ever called by the tests, by the smoke check and by the CPU-baseline
 * leg of the benchmark; the CUDA library shares no code with it and never
 * calls it.  There is no blocking, fusion or reordering here beyond the
 * definitions: rows are independent, and the only concession to run time is
 * an OpenMP loop over independent output rows.
 *
 * Conventions
 *   n     window width in bits (the paper uses 4, 3 and 2; Section 3.1, 5.1).
 *   mask  placement set: bit s set <=> the window may sit at bits [s+n-1 : s],
 *         i.e. be followed by a shift-left of s (Section 3.1: 5opt = shifts
 *         {0,1,2,3,4}, 3opt = {0,2,4}, 2opt = {0,4}).
 *   rnd   0 = trim the bits below the window, 1 = round on the residual LSBs
 *         (Section 3.1, last paragraph).  The paper does not say which way a
 *         tie goes: ties go UP here (add half, then trim).  PARITY UNPINNED
 *         for the tie direction alone; everything else is pinned by the tests.
 *   mode  0 = none (plain 8b-8b), 1 = bSPARQ on every activation,
 *         2 = vSPARQ on adjacent pairs with bSPARQ when both are non-zero (Eq. 2).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- Section 3.1: bSPARQ ------------------------------------------------ */

/* Index of the most significant set bit of a non-zero byte (Section 3.1: the window
 * is found by looking for the leading one). */
static int leading_one(unsigned x)
{
    int p = 7;
    while (p > 0 && !((x >> p) & 1u)) --p;
    return p;
}

/* The placement actually used for x: the lowest allowed shift whose n-bit window
 * still covers the leading one (Section 3.1 examples: 27 -> [4:1] under 5opt,
 * [5:2] under 3opt, [7:4] under 2opt).  Returns -1 if the set has no such shift. */
int oracle_window_shift(unsigned x, int n, unsigned mask)
{
    if (x == 0) return 0;
    int p = leading_one(x);
    for (int s = 0; s <= 8 - n; ++s) {
        if (!((mask >> s) & 1u)) continue;
        if (s + n - 1 >= p) return s;
    }
    return -1;
}

/* Is v exactly "an n-bit window shifted left by an allowed amount"? */
static int representable(unsigned v, int n, unsigned mask)
{
    for (int s = 0; s <= 8 - n; ++s) {
        if (!((mask >> s) & 1u)) continue;
        if ((v >> s) < (1u << n) && (v & ((1u << s) - 1u)) == 0) return 1;
    }
    return 0;
}

/* bSPARQ of one 8-bit activation (Section 3.1).  n = 8 is the identity. */
unsigned oracle_bsparq(unsigned x, int n, unsigned mask, int rnd)
{
    x &= 0xFFu;
    if (x == 0 || n >= 8) return x;
    int s = oracle_window_shift(x, n, mask);
    if (s < 0) return 0xFFFFFFFFu; /* invalid placement set */
    if (!rnd) return (x >> s) << s;                /* trim */
    unsigned half = s ? (1u << (s - 1)) : 0u;
    unsigned r = (x + half) >> s;                  /* round on the residual LSBs, ties up */
    if (r < (1u << n)) return r << s;
    /* The window overflowed to 2^n: the value is the single bit 2^(s+n).  It is
     * kept when a higher placement can hold it; at the top of the 8-bit range it
     * cannot, and the window saturates. */
    unsigned v = 1u << (s + n);
    if (v <= 255u && representable(v, n, mask)) return v;
    return ((1u << n) - 1u) << s;
}

/* The window bits themselves (before the shift-left), for the paper's examples. */
unsigned oracle_bsparq_window(unsigned x, int n, unsigned mask, int rnd, int *shift_out)
{
    unsigned q = oracle_bsparq(x, n, mask, rnd);
    int s = 0;
    /* the placement of the RESULT: lowest allowed shift that represents q */
    for (s = 0; s <= 8 - n; ++s) {
        if (!((mask >> s) & 1u)) continue;
        if ((q >> s) < (1u << n) && (q & ((1u << s) - 1u)) == 0) break;
    }
    if (!rnd) s = oracle_window_shift(x, n, mask); /* trim never moves the window */
    if (shift_out) *shift_out = s;
    return q >> s;
}

/* ---- Section 3.2: vSPARQ ------------------------------------------------ */

/* A lone non-zero activation of a pair owns the whole 2n-bit budget (Section 1,
 * contributions; Section 5.1 gives the pair's total window as 6 bits for n = 3 and 4 bits
 * for n = 2).
 * With 2n >= 8 that is the exact 8-bit value.  Otherwise it is a 2n-bit window made
 * of the two adjacent n-bit halves of Eq. 4, which may sit at any shift 0..8-2n. */
static unsigned lone_budget(unsigned x, int n, int rnd)
{
    int wide = 2 * n;
    if (wide >= 8) return x & 0xFFu;
    unsigned full = (1u << (8 - wide + 1)) - 1u; /* shifts 0 .. 8-2n, all allowed */
    return oracle_bsparq(x, wide, full, rnd);
}

/* Eq. 2: the pair (a, b) of adjacent activations along the reduction dimension. */
void oracle_vsparq_pair(unsigned a, unsigned b, int n, unsigned mask, int rnd,
                        unsigned *qa, unsigned *qb)
{
    a &= 0xFFu; b &= 0xFFu;
    if (b == 0)      { *qa = lone_budget(a, n, rnd); *qb = 0; }
    else if (a == 0) { *qa = 0; *qb = lone_budget(b, n, rnd); }
    else             { *qa = oracle_bsparq(a, n, mask, rnd); *qb = oracle_bsparq(b, n, mask, rnd); }
}

/* The activation transform T over `rows` rows of `row_len` bytes.  Pairs are
 * (2j, 2j+1) inside a row (Eq. 1) and never cross rows; an odd row length leaves
 * the last element paired with an implicit zero. */
void oracle_transform(const uint8_t *in, uint8_t *out, size_t rows, size_t row_len,
                      int mode, int n, unsigned mask, int rnd)
{
    for (size_t r = 0; r < rows; ++r) {
        const uint8_t *x = in + r * row_len;
        uint8_t *y = out + r * row_len;
        if (mode == 0) {
            for (size_t k = 0; k < row_len; ++k) y[k] = x[k];
        } else if (mode == 1) {
            for (size_t k = 0; k < row_len; ++k) y[k] = (uint8_t)oracle_bsparq(x[k], n, mask, rnd);
        } else {
            for (size_t k = 0; k < row_len; k += 2) {
                unsigned a = x[k], b = (k + 1 < row_len) ? x[k + 1] : 0u, qa, qb;
                oracle_vsparq_pair(a, b, n, mask, rnd, &qa, &qb);
                y[k] = (uint8_t)qa;
                if (k + 1 < row_len) y[k + 1] = (uint8_t)qb;
            }
        }
    }
}

/* ---- Eq. 4 / Section 3.1: the encoded form -------------------------------- */

/* What the multiplier of Eq. 4 receives for one pair (n = 4): two 4-bit inputs, their
 * shift-left amounts (ShiftCtrl, "opt" in Eq. 4; the 3-bit identifier of Section 3.1 for
 * five placements) and which weight each multiplier takes (MuxCtrl, Section 5.1):
 *   mux 0  in1 meets the first weight, in2 the second (both activations non-zero: each
 *          is its bSPARQ window at its own placement);
 *   mux 1  both meet the FIRST weight: the second activation is zero and the first is
 *          passed whole as its two nibbles, shifts 4 and 0 (Eq. 3);
 *   mux 2  both meet the SECOND weight, same with the roles swapped.
 * Without vSPARQ (mode 1) every pair is mux 0.  The placement stored for a window is the
 * one of the RESULT (after rounding may have carried into the next window). */
void oracle_pair_fields(unsigned a, unsigned b, int mode, unsigned mask, int rnd,
                        unsigned *in1, int *opt1, unsigned *in2, int *opt2, int *mux)
{
    a &= 0xFFu; b &= 0xFFu;
    if (mode == 2 && b == 0)      { *in1 = a >> 4; *opt1 = 4; *in2 = a & 15u; *opt2 = 0; *mux = 1; }
    else if (mode == 2 && a == 0) { *in1 = b >> 4; *opt1 = 4; *in2 = b & 15u; *opt2 = 0; *mux = 2; }
    else {
        *in1 = oracle_bsparq_window(a, 4, mask, rnd, opt1);
        *in2 = oracle_bsparq_window(b, 4, mask, rnd, opt2);
        *mux = 0;
    }
}

/* Number of allowed placements below shift s = the identifier stored for shift s. */
static int shift_rank(int s, unsigned mask)
{
    int r = 0;
    for (int t = 0; t < s; ++t) r += (int)((mask >> t) & 1u);
    return r;
}

static int set_size(unsigned mask) { return shift_rank(5, mask); }

/* The pair's metadata as ONE number (Section 5.1 mentions sharing metadata among several
 * activations and leaves it open; this library groups the two ShiftCtrl fields and the
 * MuxCtrl of a pair): with ns allowed placements,
 *   mux 0 -> id(opt1) * ns + id(opt2)      mux 1 -> ns*ns      mux 2 -> ns*ns + 1
 * so a pair has ns*ns + 2 states with vSPARQ and ns*ns without. */
int oracle_pack_states(int mode, unsigned mask)
{
    int ns = set_size(mask);
    return ns * ns + (mode == 2 ? 2 : 0);
}

int oracle_pack_ctrl_bits(int mode, unsigned mask)
{
    int states = oracle_pack_states(mode, mask), bits = 0;
    while ((1 << bits) < states) ++bits;
    return bits;
}

/* Packed stream of `rows` rows of `row_len` activations (row_len a multiple of 16, n = 4).
 * data: one byte per pair, (in1 << 4) | in2, pairs in order: rows * row_len / 2 bytes.
 * ctrl: per unit of 16 activations (8 pairs) the 8 state numbers, pair j at bits
 *       [j*cb, (j+1)*cb) of a little-endian integer of cb = ctrl_bits bytes (8 * cb bits):
 *       rows * row_len / 16 * cb bytes.
 * Returns 0, or -1 for an unsupported row length. */
int oracle_pack(const uint8_t *in, size_t rows, size_t row_len, int mode, unsigned mask, int rnd,
                uint8_t *data, uint8_t *ctrl)
{
    if (row_len % 16) return -1;
    const int ns = set_size(mask), cb = oracle_pack_ctrl_bits(mode, mask);
    for (size_t u = 0; u < rows * row_len / 16; ++u) {
        uint64_t word = 0;
        for (int j = 0; j < 8; ++j) {
            unsigned in1, in2;
            int opt1, opt2, mux;
            oracle_pair_fields(in[16 * u + 2 * j], in[16 * u + 2 * j + 1], mode, mask, rnd,
                               &in1, &opt1, &in2, &opt2, &mux);
            data[8 * u + j] = (uint8_t)((in1 << 4) | in2);
            unsigned state = mux == 0 ? (unsigned)(shift_rank(opt1, mask) * ns + shift_rank(opt2, mask))
                                      : (unsigned)(ns * ns + mux - 1);
            word |= (uint64_t)state << (j * cb);
        }
        for (int k = 0; k < cb; ++k) ctrl[(size_t)cb * u + k] = (uint8_t)(word >> (8 * k));
    }
    return 0;
}

/* The transformed activations T(x) back from the packed stream: Eq. 4 with unit weights,
 * 2^opt1 * in1 and 2^opt2 * in2, routed to the pair's slots by the mux state. */
int oracle_unpack(const uint8_t *data, const uint8_t *ctrl, size_t rows, size_t row_len,
                  int mode, unsigned mask, uint8_t *out)
{
    if (row_len % 16) return -1;
    const int ns = set_size(mask), cb = oracle_pack_ctrl_bits(mode, mask);
    int shift_of[8], r = 0;
    for (int t = 0; t <= 4; ++t) if ((mask >> t) & 1u) shift_of[r++] = t;
    for (size_t u = 0; u < rows * row_len / 16; ++u) {
        uint64_t word = 0;
        for (int k = 0; k < cb; ++k) word |= (uint64_t)ctrl[(size_t)cb * u + k] << (8 * k);
        for (int j = 0; j < 8; ++j) {
            unsigned state = (unsigned)((word >> (j * cb)) & ((1u << cb) - 1u));
            unsigned d = data[8 * u + j], qa, qb;
            if (state < (unsigned)(ns * ns)) {
                qa = (d >> 4) << shift_of[state / ns];
                qb = (d & 15u) << shift_of[state % ns];
            } else if (state == (unsigned)(ns * ns)) { qa = d; qb = 0; }
            else { qa = 0; qb = d; }
            out[16 * u + 2 * j] = (uint8_t)qa;
            out[16 * u + 2 * j + 1] = (uint8_t)qb;
        }
    }
    return 0;
}

/* ---- the encoded form for any window width (Section 5.1: 3- and 2-bit windows) ------------ */

/* Eq. 4's fields for n-bit windows.  Two non-zero activations: their n-bit windows and
 * placements, as above.  A lone non-zero activation (vSPARQ) owns the pair's 2n-bit budget
 * (Section 5.1: 6 bits for n = 3, 4 bits for n = 2): its 2n-bit window w at shift s_l in
 * 0..8-2n is handed to the two multipliers as the two n-bit halves of Eq. 3 / Eq. 4,
 *     in1 = w >> n at shift s_l + n,    in2 = w & (2^n - 1) at shift s_l,
 * both against the lone activation's weight (mux 1: first slot, mux 2: second slot).
 * For n = 4 the window is the whole byte at s_l = 0 and this is oracle_pair_fields. */
void oracle_pair_fields_n(unsigned a, unsigned b, int mode, int n, unsigned mask, int rnd,
                          unsigned *in1, int *opt1, unsigned *in2, int *opt2, int *mux)
{
    a &= 0xFFu; b &= 0xFFu;
    if (mode == 2 && (b == 0 || a == 0)) {
        unsigned x = (b == 0) ? a : b, w = x;
        int sl = 0;
        if (2 * n < 8) {
            unsigned full = (1u << (8 - 2 * n + 1)) - 1u;      /* shifts 0 .. 8-2n */
            w = oracle_bsparq_window(x, 2 * n, full, rnd, &sl);
        }
        *in1 = w >> n; *opt1 = sl + n;
        *in2 = w & ((1u << n) - 1u); *opt2 = sl;
        *mux = (b == 0) ? 1 : 2;
    } else {
        *in1 = oracle_bsparq_window(a, n, mask, rnd, opt1);
        *in2 = oracle_bsparq_window(b, n, mask, rnd, opt2);
        *mux = 0;
    }
}

static int set_size_n(int n, unsigned mask) { return shift_rank(8 - n + 1, mask); }
static int lone_places(int n) { return 8 - 2 * n + 1; }        /* n = 4: 1, n = 3: 3, n = 2: 5 */

/* States of a pair: ns*ns for two windows; with vSPARQ also the lone window's placement in
 * either slot: ns*ns + s_l (first slot), ns*ns + lone_places + s_l (second slot). */
int oracle_pack_states_n(int mode, int n, unsigned mask)
{
    int ns = set_size_n(n, mask);
    return ns * ns + (mode == 2 ? 2 * lone_places(n) : 0);
}

int oracle_pack_ctrl_bits_n(int mode, int n, unsigned mask)
{
    int states = oracle_pack_states_n(mode, n, mask), bits = 0;
    while ((1 << bits) < states) ++bits;
    return bits;
}

/* Packed stream for n-bit windows, per unit of 16 activations (8 pairs):
 * data: pair j's field (in1 << n) | in2 at bits [j*2n, (j+1)*2n) of a little-endian integer
 *       of 2n bytes (n = 4: one byte per pair, as oracle_pack);
 * ctrl: pair j's state at bits [j*cb, (j+1)*cb) of a little-endian integer of cb bytes. */
int oracle_pack_n(const uint8_t *in, size_t rows, size_t row_len, int mode, int n, unsigned mask, int rnd,
                  uint8_t *data, uint8_t *ctrl)
{
    if (row_len % 16) return -1;
    const int ns = set_size_n(n, mask), cb = oracle_pack_ctrl_bits_n(mode, n, mask), nl = lone_places(n);
    for (size_t u = 0; u < rows * row_len / 16; ++u) {
        uint64_t dword = 0, cword = 0;
        for (int j = 0; j < 8; ++j) {
            unsigned in1, in2;
            int opt1, opt2, mux;
            oracle_pair_fields_n(in[16 * u + 2 * j], in[16 * u + 2 * j + 1], mode, n, mask, rnd,
                                 &in1, &opt1, &in2, &opt2, &mux);
            dword |= (uint64_t)((in1 << n) | in2) << (j * 2 * n);
            unsigned state = mux == 0 ? (unsigned)(shift_rank(opt1, mask) * ns + shift_rank(opt2, mask))
                                      : (unsigned)(ns * ns + (mux - 1) * nl + opt2);
            cword |= (uint64_t)state << (j * cb);
        }
        for (int k = 0; k < 2 * n; ++k) data[(size_t)(2 * n) * u + k] = (uint8_t)(dword >> (8 * k));
        for (int k = 0; k < cb; ++k) ctrl[(size_t)cb * u + k] = (uint8_t)(cword >> (8 * k));
    }
    return 0;
}

/* T(x) back from the packed stream: 2^opt1 * in1 and 2^opt2 * in2 (Eq. 4 with unit weights);
 * for a lone value the two halves add up in its slot. */
int oracle_unpack_n(const uint8_t *data, const uint8_t *ctrl, size_t rows, size_t row_len,
                    int mode, int n, unsigned mask, uint8_t *out)
{
    if (row_len % 16) return -1;
    const int ns = set_size_n(n, mask), cb = oracle_pack_ctrl_bits_n(mode, n, mask), nl = lone_places(n);
    int shift_of[8], r = 0;
    for (int t = 0; t <= 8 - n; ++t) if ((mask >> t) & 1u) shift_of[r++] = t;
    for (size_t u = 0; u < rows * row_len / 16; ++u) {
        uint64_t dword = 0, cword = 0;
        for (int k = 0; k < 2 * n; ++k) dword |= (uint64_t)data[(size_t)(2 * n) * u + k] << (8 * k);
        for (int k = 0; k < cb; ++k) cword |= (uint64_t)ctrl[(size_t)cb * u + k] << (8 * k);
        for (int j = 0; j < 8; ++j) {
            unsigned state = (unsigned)((cword >> (j * cb)) & ((1u << cb) - 1u));
            unsigned f = (unsigned)((dword >> (j * 2 * n)) & ((1u << (2 * n)) - 1u));
            unsigned in1 = f >> n, in2 = f & ((1u << n) - 1u), qa, qb;
            if (state < (unsigned)(ns * ns)) {
                qa = in1 << shift_of[state / ns];
                qb = in2 << shift_of[state % ns];
            } else {
                unsigned t = state - (unsigned)(ns * ns), sl = t % (unsigned)nl;
                unsigned v = (in1 << (sl + n)) + (in2 << sl);
                if (t / (unsigned)nl == 0) { qa = v; qb = 0; } else { qa = 0; qb = v; }
            }
            out[16 * u + 2 * j] = (uint8_t)qa;
            out[16 * u + 2 * j + 1] = (uint8_t)qb;
        }
    }
    return 0;
}

/* ---- Eq. 1: the dot product over the transformed activations ------------- */

/* acc[m][j] = sum_k T(A)[m][k] * B[k][j]; A is M x K (row-major, u8), B is the
 * logical K x N matrix (row-major, s8), int32 accumulation.  |acc| <= K*255*128,
 * which cannot overflow 32 bits for K <= 65793. */
void oracle_gemm(const uint8_t *A, const int8_t *B, int32_t *acc,
                 int64_t M, int64_t N, int64_t K,
                 int mode, int n, unsigned mask, int rnd)
{
#pragma omp parallel
    {
        uint8_t *ta = (uint8_t *)__builtin_malloc((size_t)(K > 0 ? K : 1));
#pragma omp for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            oracle_transform(A + m * K, ta, 1, (size_t)K, mode, n, mask, rnd);
            for (int64_t j = 0; j < N; ++j) acc[m * N + j] = 0;
            for (int64_t k = 0; k < K; ++k) {
                int32_t a = ta[k];
                const int8_t *brow = B + k * N;
                for (int64_t j = 0; j < N; ++j) acc[m * N + j] += a * (int32_t)brow[j];
            }
        }
        __builtin_free(ta);
    }
}

/* ---- Section 4 / 5.3: SPARQ on top of a sparse tensor core ------------------- */

/* Weights pruned 2:4 are stored compressed: per output channel j and per group g of four
 * consecutive reduction indices, the two kept values vals[j][2g], vals[j][2g+1] and their
 * coordinates pos[j][2g] < pos[j][2g+1] in 0..3 (Section 4: a sparse tensor core keeps the
 * non-zero weights together with their coordinates).  The coordinates pick two of the
 * group's four activations; vSPARQ then looks at THAT pair (Section 5.3: the activations
 * pass the coordinate multiplexers first and are paired afterwards), so the transform
 * depends on the output channel:
 *     acc[m][j] = sum_g  T2(A[m][4g+p0], A[m][4g+p1]) . (v0, v1)
 * with T2 the pair rule of Eq. 2 (mode 2), bSPARQ on each (mode 1) or the identity (mode 0).
 * K must be a multiple of 4.  Returns 0, or -1 for bad coordinates. */
int oracle_gemm_sparse24(const uint8_t *A, const int8_t *vals, const uint8_t *pos, int32_t *acc,
                         int64_t M, int64_t N, int64_t K, int mode, int n, unsigned mask, int rnd)
{
    if (K % 4) return -1;
    for (int64_t j = 0; j < N; ++j)
        for (int64_t g = 0; g < K / 4; ++g) {
            unsigned p0 = pos[j * (K / 2) + 2 * g], p1 = pos[j * (K / 2) + 2 * g + 1];
            if (p0 >= p1 || p1 > 3) return -1;
        }
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t j = 0; j < N; ++j) {
            int32_t sum = 0;
            for (int64_t g = 0; g < K / 4; ++g) {
                const int64_t c = j * (K / 2) + 2 * g;
                unsigned a = A[m * K + 4 * g + pos[c]], b = A[m * K + 4 * g + pos[c + 1]], qa, qb;
                if (mode == 2) oracle_vsparq_pair(a, b, n, mask, rnd, &qa, &qb);
                else if (mode == 1) { qa = oracle_bsparq(a, n, mask, rnd); qb = oracle_bsparq(b, n, mask, rnd); }
                else { qa = a; qb = b; }
                sum += (int32_t)qa * (int32_t)vals[c] + (int32_t)qb * (int32_t)vals[c + 1];
            }
            acc[m * N + j] = sum;
        }
    }
    return 0;
}

/* Same product accumulated in 64 bits (tiny shapes only): equality with the int32
 * result shows that the 32-bit accumulator never wrapped. */
void oracle_gemm_i64(const uint8_t *A, const int8_t *B, int64_t *acc,
                     int64_t M, int64_t N, int64_t K,
                     int mode, int n, unsigned mask, int rnd)
{
    uint8_t *ta = (uint8_t *)__builtin_malloc((size_t)(K > 0 ? K : 1));
    for (int64_t m = 0; m < M; ++m) {
        oracle_transform(A + m * K, ta, 1, (size_t)K, mode, n, mask, rnd);
        for (int64_t j = 0; j < N; ++j) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k) s += (int64_t)ta[k] * (int64_t)B[k * N + j];
            acc[m * N + j] = s;
        }
    }
    __builtin_free(ta);
}

/* ---- Section 4: convolution as the same dot product --------------------- */

/* Direct convolution.  x is NHWC u8, w is [cout][r][s][c] s8, dilation 1.  The
 * reduction runs over (r, s, c) with c fastest, so vSPARQ pairs are adjacent input
 * channels of one pixel; T is therefore applied once to the whole input tensor with
 * rows = pixels.  Taps that fall outside the image contribute nothing.
 *
 * Only the output pixels listed in `pix` (linear index over n, ho, wo) are computed
 * when pix != NULL; otherwise all of them.  acc is [npix][cout]. */
void oracle_conv2d_nhwc(const uint8_t *x, int nb, int h, int w, int c,
                        const int8_t *wgt, int cout, int r, int s,
                        int stride_h, int stride_w, int pad_h, int pad_w,
                        int mode, int n, unsigned mask, int rnd,
                        const int64_t *pix, int64_t npix, int32_t *acc)
{
    int ho = (h + 2 * pad_h - r) / stride_h + 1;
    int wo = (w + 2 * pad_w - s) / stride_w + 1;
    int64_t total = (int64_t)nb * ho * wo;
    int64_t count = pix ? npix : total;
    size_t in_pixels = (size_t)nb * h * w;
    uint8_t *tx = (uint8_t *)__builtin_malloc(in_pixels * (size_t)c + 1);
    oracle_transform(x, tx, in_pixels, (size_t)c, mode, n, mask, rnd);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        int64_t p = pix ? pix[i] : i;
        int img = (int)(p / ((int64_t)ho * wo));
        int oy = (int)((p / wo) % ho);
        int ox = (int)(p % wo);
        for (int co = 0; co < cout; ++co) {
            int32_t sum = 0;
            for (int fr = 0; fr < r; ++fr) {
                int iy = oy * stride_h - pad_h + fr;
                if (iy < 0 || iy >= h) continue;
                for (int fs = 0; fs < s; ++fs) {
                    int ix = ox * stride_w - pad_w + fs;
                    if (ix < 0 || ix >= w) continue;
                    const uint8_t *xp = tx + (((size_t)img * h + iy) * w + ix) * (size_t)c;
                    const int8_t *wp = wgt + (((size_t)co * r + fr) * s + fs) * (size_t)c;
                    for (int ci = 0; ci < c; ++ci) sum += (int32_t)xp[ci] * (int32_t)wp[ci];
                }
            }
            acc[i * cout + co] = sum;
        }
    }
    __builtin_free(tx);
}

/* ---- Dequantize, bias, ReLU, requantize ---------------------------------- */

/* The paper only fixes the quantization scheme (Section 5: per-layer activation
 * scale, per-kernel weight scale); the arithmetic below is this library's stated
 * fp32 sequence, one IEEE operation per line, no contraction:
 *     t = (float)acc                       int32 -> fp32, round to nearest even
 *     y = fma(t, scale[j], bias[j])        single rounding
 *     y = fma((float)res, res_scale, y)    only with a residual input: the block's u8
 *                                          identity tensor on its own scale, added before
 *                                          the ReLU as in a ResNet bottleneck
 *     y = relu ? max(y, 0) : y             (y > 0 ? y : 0)
 *     z = y * inv_out_scale
 *     u = rint(z)                          nearest even
 *     q = clamp(u, 0, 255) as uint8        NaN -> 0
 * Any of f32_out / u8_out may be NULL; residual may be NULL (no residual step). */
void oracle_epilogue_residual(const int32_t *acc, int64_t M, int64_t N,
                              const float *scale, const float *bias,
                              const uint8_t *residual, float residual_scale,
                              int relu, float inv_out_scale,
                              float *f32_out, uint8_t *u8_out)
{
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t j = 0; j < N; ++j) {
            volatile float t = (float)acc[m * N + j];
            volatile float y = fmaf(t, scale[j], bias ? bias[j] : 0.0f);
            if (residual) {
                volatile float r = (float)residual[m * N + j];
                y = fmaf(r, residual_scale, y);
            }
            if (relu) y = (y > 0.0f) ? y : 0.0f;
            if (f32_out) f32_out[m * N + j] = y;
            if (u8_out) {
                volatile float z = y * inv_out_scale;
                volatile float u = rintf(z);
                uint8_t q;
                if (!(u > 0.0f)) q = 0;             /* negative, zero and NaN */
                else if (u > 255.0f) q = 255;
                else q = (uint8_t)u;
                u8_out[m * N + j] = q;
            }
        }
    }
}

void oracle_epilogue(const int32_t *acc, int64_t M, int64_t N,
                     const float *scale, const float *bias, int relu, float inv_out_scale,
                     float *f32_out, uint8_t *u8_out)
{
    oracle_epilogue_residual(acc, M, N, scale, bias, NULL, 0.0f, relu, inv_out_scale, f32_out, u8_out);
}

/* ---- Section 5: uniform min-max quantization of the network's tensors ------ */

/* Section 5: every layer is quantized uniformly from its min-max statistics -- activations
 * unsigned and symmetric with one scale per layer, weights signed and symmetric with one
 * scale per kernel.  The statistic of both is the largest magnitude; NaNs are skipped.  bf16 inputs are given as their 16-bit patterns and widened
 * exactly (bf16 is the top half of an fp32). */
static float load_elem(const void *x, int is_bf16, size_t i)
{
    if (!is_bf16) return ((const float *)x)[i];
    uint32_t bits = (uint32_t)((const uint16_t *)x)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

float oracle_absmax(const void *x, int is_bf16, size_t n)
{
    float m = 0.0f;
    for (size_t i = 0; i < n; ++i) {
        float a = fabsf(load_elem(x, is_bf16, i));
        if (a > m) m = a;                    /* false for NaN */
    }
    return m;
}

/* Activations, unsigned symmetric per layer: the 8-bit grid spans [0, max], so one step is
 * max / 255.  fp32, one IEEE operation per line:
 *     inv = 255 / max                 (0 when max is 0)
 *     z   = x * inv
 *     q   = clamp(rint(z), 0, 255)    nearest even; negatives and NaN -> 0 */
void oracle_quantize_act(const void *x, int is_bf16, size_t n, float max, uint8_t *out)
{
    volatile float inv = max > 0.0f ? 255.0f / max : 0.0f;
    for (size_t i = 0; i < n; ++i) {
        volatile float z = load_elem(x, is_bf16, i) * inv;
        volatile float u = rintf(z);
        out[i] = !(u > 0.0f) ? 0 : u > 255.0f ? 255 : (uint8_t)u;
    }
}

/* Weights, signed symmetric per kernel (output channel): row j of the cout x k matrix has
 * its own largest magnitude a_j; the grid is [-127, 127] with step a_j / 127:
 *     inv_j = 127 / a_j  (0 when a_j is 0);  q = clamp(rint(w * inv_j), -127, 127)
 * scale_out[j] = a_j / 127 is the factor that maps the integers back. */
void oracle_quantize_weight(const float *w, int64_t cout, int64_t k, int8_t *out, float *scale_out)
{
    for (int64_t j = 0; j < cout; ++j) {
        float a = oracle_absmax(w + j * k, 0, (size_t)k);
        volatile float inv = a > 0.0f ? 127.0f / a : 0.0f;
        for (int64_t i = 0; i < k; ++i) {
            volatile float z = w[j * k + i] * inv;
            volatile float u = rintf(z);
            out[j * k + i] = u > 127.0f ? 127 : u < -127.0f ? -127 : (u == u ? (int8_t)u : 0);
        }
        volatile float sc = a / 127.0f;
        scale_out[j] = sc;
    }
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}
