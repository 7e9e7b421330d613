// Shared host/device pieces of the SPARQ library: error reporting, parameter
// validation, and the packed (4 activations per 32-bit word) form of the
// bSPARQ / vSPARQ transform used by both the standalone kernel and the fused GEMM.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sparq.h"

namespace sparq {

// ---- host side ---------------------------------------------------------------------

int set_error(int code, const char *fmt, ...);
int cuda_error(cudaError_t e, const char *what);

// Host-validated, kernel-ready description of the transform.
struct XformArgs {
    int mode;           // SPARQ_MODE_*
    int n;              // window bits: 2, 3, 4
    int rnd;            // 0 trim, 1 nearest
    int widen_rounds;   // longest run of consecutive disallowed shifts
    uint32_t widen_c;   // per byte: bit d set for every disallowed shift d (0 < d < 8-n)
    uint32_t mask;      // placement mask as given
};

// Checks `p` (Section 3.1 placement sets, Section 5.1 widths) and fills `x`.
int validate_params(const sparq_params *p, XformArgs *x);

// Device status word shared by all kernels of this library on the current device.
// Bit 0: a bounded wait expired.  Allocated on first use, freed by sparq_shutdown().
int get_status_word(unsigned int **dptr);

// ---- device side -------------------------------------------------------------------

#define SPARQ_HD __host__ __device__ __forceinline__

// prmt.b32: byte i of the result is byte (sel nibble i & 7) of {b:a}; nibble bit 3 asks
// for that byte's top bit replicated over all eight bits instead.
SPARQ_HD uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
#ifdef __CUDA_ARCH__
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
#else
    uint64_t src = ((uint64_t)b << 32) | a;
    uint32_t d = 0;
    for (int i = 0; i < 4; ++i) {
        uint32_t nib = (sel >> (4 * i)) & 0xFu;
        uint32_t byte = (uint32_t)(src >> (8 * (nib & 7u))) & 0xFFu;
        if (nib & 8u) byte = (byte & 0x80u) ? 0xFFu : 0u;
        d |= byte << (8 * i);
    }
    return d;
#endif
}

// Kernel-side copy of the placement-set constants of XformArgs.
struct XformDev {
    uint32_t widen_c;
    int rounds;
    int n;
    // Full placement sets only (every shift 0..8-n allowed; see xform_word_fullset): per 16-bit
    // half, twice in a word -- the rounding increment, the mask of the kept bits and the
    // saturation value of the n-bit window (f_*) and of the 2n-bit window of a lone non-zero (l_*).
    uint32_t f_add, f_mask, f_sat;
    uint32_t l_add, l_mask, l_sat;
};

// binary16 bit pattern of an integer 0 < v < 2048 (exact)
inline uint32_t half_bits_of_int(uint32_t v)
{
    int p = 0;
    while ((v >> (p + 1)) != 0) ++p;
    return ((uint32_t)(p + 15) << 10) | ((v << (10 - p)) & 0x3FFu);
}

// Constants of xform_word_fullset for window width n and the rounding flag.
inline void fill_fullset(XformDev *d, int n, int rnd)
{
    auto set = [&](int w, uint32_t *add, uint32_t *mask, uint32_t *sat) {
        if (w >= 8) {                    // the window holds all 8 bits: nothing is dropped
            *add = 0u; *mask = 0xFFFFFFFFu; *sat = half_bits_of_int(255u) * 0x00010001u;
            return;
        }
        const uint32_t m16 = (0xFFFFu << (11 - w)) & 0xFFFFu;      // sign, exponent and the top w-1 fraction bits
        const uint32_t a16 = rnd ? (1u << (10 - w)) : 0u;          // half of the lowest kept bit
        *mask = m16 * 0x00010001u;
        *add = a16 * 0x00010001u;
        *sat = half_bits_of_int(((1u << w) - 1u) << (8 - w)) * 0x00010001u;
    };
    set(n, &d->f_add, &d->f_mask, &d->f_sat);
    set(2 * n, &d->l_add, &d->l_mask, &d->l_sat);
}

// Mask of the bits BELOW the window for each of the four bytes of x (Section 3.1: the
// window's top bit is the leading one, or the window sits at the bottom).  The window
// width is WT when WT != 0, else the run-time value w_rt.  With WIDEN, a window that landed
// on a disallowed placement moves up to the next allowed one: one step `m |= (m << 1) & c`
// moves every byte that sits on a disallowed shift up by one and leaves the others alone,
// so three unconditional steps cover the longest possible run (n - 1 <= 3) and need no
// branch.
template <int WT, bool WIDEN>
SPARQ_HD uint32_t drop_mask(uint32_t x, int w_rt, uint32_t widen_c)
{
    const int w = WT ? WT : w_rt;
    const uint32_t low = 0x01010101u * (0xFFu >> w);
    uint32_t m = (x >> w) & low;                 // bits of x above the lowest window
    m |= (m >> 1) & 0x7F7F7F7Fu;                 // smear the leading one downwards
    if (!WT || 8 - WT > 2) m |= (m >> 2) & 0x3F3F3F3Fu;
    if (!WT || 8 - WT > 4) m |= (m >> 4) & 0x0F0F0F0Fu;
    if (WIDEN) {
        m |= (m << 1) & widen_c;
        m |= (m << 1) & widen_c;
        m |= (m << 1) & widen_c;
    }
    return m;
}

// Trim or round four bytes given their drop masks (w = window width).  Rounding adds
// half a window LSB; a byte that would overflow 8 bits (only possible at the highest
// placement, where the half is 0x80 >> w) keeps its trimmed value, i.e. saturates to
// the all-ones window.
template <bool RND>
SPARQ_HD uint32_t apply_mask(uint32_t x, uint32_t m, int w)
{
    if (!RND) return x & ~m;
    uint32_t half = m ^ ((m >> 1) & 0x7F7F7F7Fu);   // (m + 1) >> 1 per byte
    uint32_t x7 = x & 0x7F7F7F7Fu, x8 = x & 0x80808080u;
    uint32_t lo = x7 + half;                        // no carry leaves a byte
    uint32_t ovf = lo & x8;                         // bit 7: x + half >= 256
    lo -= ovf >> w;
    return (lo ^ x8) & ~m;
}

// T on four packed activations (bytes 0,1 and bytes 2,3 are the pairs of Eq. 2).
// N = 2, 3, 4 fixes the window width at compile time; N = 0 takes it from d.n.
// WIDEN = false is only valid for full placement sets (d.rounds == 0).
template <int MODE, int N, bool RND, bool WIDEN>
SPARQ_HD uint32_t xform_word(uint32_t x, const XformDev &d)
{
    if (MODE == SPARQ_MODE_NONE) return x;
    const int n = N ? N : d.n;
    uint32_t q = apply_mask<RND>(x, drop_mask<N, WIDEN>(x, n, d.widen_c), n);
    if (MODE == SPARQ_MODE_BSPARQ) return q;
    // vSPARQ: a byte whose partner is zero keeps the 2n-bit budget (all 8 bits for n = 4;
    // a 2n-bit window at any shift 0..8-2n otherwise, Section 5.1).
    uint32_t lone = x;
    if (N == 2 || N == 3) {
        lone = apply_mask<RND>(x, drop_mask<(N == 4 ? 0 : 2 * N), false>(x, 2 * n, 0u), 2 * n);
    } else if (N == 0) {
        // run-time width: n = 4 gives a window of 8 bits, whose drop mask is empty
        const int w2 = 2 * n;
        lone = apply_mask<RND>(x, w2 < 8 ? drop_mask<0, false>(x, w2, 0u) : 0u, w2 < 8 ? w2 : 7);
    }
    uint32_t nz = ((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x;   // bit 7 of each byte: byte != 0
    uint32_t partner_nz = prmt(nz, nz, 0xAB89u);           // swap within pairs, replicate bit 7
    return (q & partner_nz) | (lone & ~partner_nz);
}

#ifdef __CUDACC__
// ---- full placement sets: the window through the floating-point unit --------------------------
// With every shift allowed, bSPARQ keeps the n most significant bits starting at the leading
// one (Section 3.1) -- which is what a binary floating-point number with n - 1 fraction bits
// holds.  A byte b is exact in binary16 (11 significant bits); as bit patterns, two bytes per
// 32-bit register:
//     0x6400 | b            = 1024 + b          (one byte permute per pair)
//     (1024 + b) - 1024     = b, normalized: the subtraction finds the leading one
//     (bits + half) & mask  = b rounded to n significant bits, ties up, a carry moving into the
//                             exponent (31 -> 32); without the increment: trimmed
//     min(., top window)    = the saturation at the top of the byte range (248.. -> 240)
//     . + 1024              = the integer back in the low byte of each half
// 13 instructions per four activations for any width and either rounding (17 with the pair
// rule for n = 4, 26 for n < 4 with its second, 2n-bit window), where the packed integer form
// with a run-time width needs about twice as many; for n = 4 the integer form specialized at
// compile time (19 with the pair rule) measured a few per cent faster and is kept.
__device__ __forceinline__ uint32_t h2_sub(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t h2_add(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("add.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t h2_min(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("min.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

template <int MODE>
__device__ __forceinline__ uint32_t xform_word_fullset(uint32_t x, const XformDev &d)
{
    if (MODE == SPARQ_MODE_NONE) return x;
    const uint32_t k1024 = 0x64006400u;
    // bytes 0,1 and bytes 2,3 as halves
    const uint32_t lo = h2_sub(prmt(x, 0x64646464u, 0x4140u), k1024);
    const uint32_t hi = h2_sub(prmt(x, 0x64646464u, 0x4342u), k1024);
    const uint32_t qlo = h2_add(h2_min((lo + d.f_add) & d.f_mask, d.f_sat), k1024);
    const uint32_t qhi = h2_add(h2_min((hi + d.f_add) & d.f_mask, d.f_sat), k1024);
    const uint32_t q = prmt(qlo, qhi, 0x6420u);
    if (MODE == SPARQ_MODE_BSPARQ) return q;
    // vSPARQ: a byte whose partner is zero keeps the 2n-bit window (the whole byte for n = 4)
    uint32_t lone = x;
    if (d.l_mask != 0xFFFFFFFFu) {       // uniform: a kernel argument
        const uint32_t llo = h2_add(h2_min((lo + d.l_add) & d.l_mask, d.l_sat), k1024);
        const uint32_t lhi = h2_add(h2_min((hi + d.l_add) & d.l_mask, d.l_sat), k1024);
        lone = prmt(llo, lhi, 0x6420u);
    }
    const uint32_t nz = ((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x;   // bit 7 of each byte: byte != 0
    const uint32_t partner_nz = prmt(nz, nz, 0xAB89u);           // swap within pairs, replicate bit 7
    return (q & partner_nz) | (lone & ~partner_nz);
}

// The transform of a fused kernel instantiated for (MODE, XN, RND): XN = 4 is n = 4 with all
// five placements (packed-integer form, width fixed at compile time), XN = 8 any other full
// placement set (6opt, 7opt; either rounding, through the constants; RND unused), XN = 0 the
// general packed-integer form with run-time width and the placement widening.
template <int MODE, int XN, bool RND>
__device__ __forceinline__ uint32_t xform_fused(uint32_t x, const XformDev &d)
{
    if (XN == 8) return xform_word_fullset<MODE>(x, d);
    if (XN == 4) return xform_word<MODE, 4, RND, false>(x, d);
    return xform_word<MODE, 0, RND, true>(x, d);
}
#endif

}  // namespace sparq
