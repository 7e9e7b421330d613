// Fused SPARQ GEMM / implicit-GEMM convolution for sm_100a.
//
//   acc[m][j] = sum_k T(A)[m][k] * B[j][k]      (Eq. 1 with Eq. 2 applied on the fly)
//
// One persistent CTA per SM walks output tiles of 128 x BN.  Warp roles:
//   warp 0        TMA producer: A tile (tiled 2-D box for the GEMM, im2col box for the
//                 convolution) and B tile into a ring of shared-memory stages
//   warp 1        allocates tensor memory; one lane issues tcgen05.mma kind::i8
//                 (u8 x s8 -> s32) on each transformed stage
//   warps 2..9    epilogue: tcgen05.ld of a finished accumulator, fp32 scale / bias /
//                 ReLU / requantize, global stores (warp w reads lane quarter w % 4 and
//                 one half of the tile's columns)
//   warps 10..17  transform: rewrite the A stage in place with bSPARQ / vSPARQ
//
// A stage travels  TMA (async proxy) -> transform warps (generic proxy) -> MMA (async
// proxy); the hand-offs are mbarriers, with fence.proxy.async after the in-place rewrite.
// The 128-byte (64-byte) shared-memory swizzle only permutes 16-byte chunks inside a
// row, and a vSPARQ pair never straddles a 16-byte chunk, so the transform treats the
// stage as a flat array of 16-byte vectors.
//
// Every wait is bounded: when a wait gives up it sets bit 0 of the status word, raises a
// CTA-wide abort flag that makes all later waits return at once, and the kernel still
// runs to its normal end (loops have fixed trip counts), drains its own copies and frees
// its tensor memory.
#pragma once

#include <cuda.h>

#include "sparq_common.cuh"

namespace sparq {

constexpr int kBM = 128;                 // rows of an output tile = MMA M
constexpr int kNumEpiWarps = 8;          // two per tensor-memory lane quarter; without a transform
                                         // (mode NONE) the transform warps are epilogue warps too
constexpr int kNumXfWarps = 8;
// The transform warps work as two teams that take stages (or window pieces) alternately: a
// stage's chain of barrier read, shared-memory loads, arithmetic, stores and fence is mostly
// latency, and one team's chain overlaps the other's.
constexpr int kXfTeams = 2;
constexpr int kXfTeamWarps = kNumXfWarps / kXfTeams;
constexpr int kFirstEpiWarp = 2;
constexpr int kFirstXfWarp = kFirstEpiWarp + kNumEpiWarps;
constexpr int kGemmThreads = 32 * (kFirstXfWarp + kNumXfWarps);
// Epilogue warps of a kernel instantiated for `mode`.
__host__ __device__ constexpr int epi_warps(int mode) { return mode == SPARQ_MODE_NONE ? kNumEpiWarps + kNumXfWarps : kNumEpiWarps; }
constexpr int kSmemBudget = 200 * 1024;  // for the stage ring
// Default limit of every device-side wait, in SM clock cycles (about a second).  The limit is a
// kernel argument, so that a diagnostic launch can make a wait run out in microseconds.
constexpr long long kWaitLimitCycles = 2000000000LL;

struct GemmArgs {
    // problem
    int64_t M, N, K;        // GEMM view (K = r*s*c for the convolution)
    int k_blocks;           // number of BK-wide reduction steps
    // convolution geometry (conv = 1) for the im2col producer
    int conv;
    int c_blocks;           // BK-wide channel blocks per filter tap (the last one may reach past C: zero fill)
    int tap_k;              // bytes of a filter row per tap (= C)
    int S;                  // filter width (taps are ordered r-major, s-minor)
    int Ho, Wo;
    int stride_h, stride_w, pad_h, pad_w;
    // transform
    XformDev xf;
    // epilogue
    const float *scale;
    const float *bias;
    int relu;
    float inv_out_scale;
    int32_t *acc_out;
    float *f32_out;
    uint8_t *u8_out;
    unsigned int *status;
    long long wait_limit;   // cycles after which a device-side wait gives up
    // producer-side transform of u8_out (mode NONE = off)
    int next_mode, next_rnd;
    XformDev next_xf;
    // residual input of the epilogue (nullptr = none)
    const uint8_t *residual;
    float residual_scale;
};

// ---- PTX wrappers ---------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Non-blocking look at a phase: 1 if it has completed.  Unlike try_wait this never suspends
// the thread, and nothing waits for its result until the value is used.
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}

// Three looks at once (bit i: barrier i): all reads are in flight together before any answer
// is consumed.
__device__ __forceinline__ uint32_t mbar_test3(uint32_t bar0, uint32_t parity0, uint32_t bar1, uint32_t parity1,
                                               uint32_t bar2, uint32_t parity2)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p, q, r;\n\t.reg .u32 a, b, c;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 q, [%3], %4;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 r, [%5], %6;\n\t"
        "selp.u32 a, 1, 0, p;\n\t"
        "selp.u32 b, 2, 0, q;\n\t"
        "selp.u32 c, 4, 0, r;\n\t"
        "or.b32 a, a, b;\n\t"
        "or.b32 %0, a, c;\n\t}"
        : "=r"(ok) : "r"(bar0), "r"(parity0), "r"(bar1), "r"(parity1), "r"(bar2), "r"(parity2) : "memory");
    return ok;
}

// Bounded wait.  Returns false (after flagging) if the phase did not complete in time or
// if another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          unsigned int *status, long long limit_cycles, bool ignore_abort = false)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (!ignore_abort && *abort_flag) return false;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 0x3Fu) == 0) {
            if (!ignore_abort && *abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                *abort_flag = 1u;
                atomicOr(status, 1u);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

// im2col box: `pixels-per-column` output pixels starting at base pixel (w, h, n), channels
// c .. c+box, filter tap offset (woff, hoff); out-of-image taps are filled with zeros.
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                                   int c, int w, int h, int n, uint16_t woff, uint16_t hoff)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        :: "r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(woff), "h"(hoff) : "memory");
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" :: "l"(map) : "memory");
}

// Programmatic dependent launch: the kernel may start while the previous kernel on the
// stream is still draining.  dep_launch() lets the next kernel start its own prologue;
// dep_wait() blocks until every earlier kernel has completed and its writes are visible,
// and is executed by every thread before it touches global memory.
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], 128 x N x 32, u8 x s8 -> s32.
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// The same two instructions for a warp that runs its loop converged: every lane executes
// the surrounding code (so that descriptor arithmetic on warp-uniform values can stay in
// the uniform datapath) and only the lane with `elected` != 0 issues.
__device__ __forceinline__ void tc_mma_i8_if(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate, uint32_t elected)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(elected) : "memory");
}

__device__ __forceinline__ void tc_commit_if(uint32_t bar, uint32_t elected)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        :: "r"(bar), "r"(elected) : "memory");
}

// One lane of a converged warp (the same lane every time it is asked within a launch is not
// guaranteed; callers ask once and keep the answer).
__device__ __forceinline__ uint32_t elect_one()
{
    uint32_t e;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
    return e;
}

// Shared-memory matrix descriptor of a K-major tile whose rows are ROW_BYTES long
// (128 or 64) and swizzled with the matching TMA mode; 8-row groups are contiguous.
template <int ROW_BYTES>
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr)
{
    constexpr uint64_t layout = (ROW_BYTES == 128) ? 2ull : 4ull;   // 128B / 64B swizzle
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);            // start address
    d |= (uint64_t)1 << 16;                              // leading-dimension offset (unused when swizzled)
    d |= (uint64_t)((8 * ROW_BYTES) >> 4) << 32;         // stride between 8-row groups
    d |= (uint64_t)1 << 46;                              // descriptor version of this architecture
    d |= layout << 61;
    return d;
}

// kind::i8 instruction descriptor: s32 accumulator, unsigned A, signed B, both K-major.
__device__ __forceinline__ constexpr uint32_t make_idesc_i8(int n)
{
    return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Barrier among the epilogue warps only (hardware barrier 1).
template <int WARPS>
__device__ __forceinline__ void epi_bar_sync()
{
    asm volatile("bar.sync 1, %0;" :: "n"(WARPS * 32) : "memory");
}

// 32 contiguous bytes with one 256-bit store (dst 32-byte aligned).
__device__ __forceinline__ void st_global_v8(void *dst, const uint32_t (&w)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

__device__ __forceinline__ void tmem_ld_32x32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}

__device__ __forceinline__ void tmem_ld_32x16_issue(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

// ---- epilogue arithmetic ----------------------------------------------------------------

// int32 accumulator -> fp32 value, one IEEE operation per step.  SMALL: the caller
// guarantees |acc| < 2^22, where (float)acc is exact and equals
// bits(acc + bits(1.5 * 2^23)) - 1.5 * 2^23.
template <bool SMALL>
__device__ __forceinline__ float dequant(int32_t acc, float scale, float bias, int relu)
{
    float t = SMALL ? __fadd_rn(__int_as_float(acc + 0x4B400000), -12582912.0f) : __int2float_rn(acc);
    float y = __fmaf_rn(t, scale, bias);
    if (relu) y = fmaxf(y, 0.0f);        // NaN -> 0, like (y > 0 ? y : 0)
    return y;
}

// Four fp32 values on the output grid -> four bytes clamp(rint(z), 0, 255) in one word, z0 in
// the low byte: a round-to-nearest-even conversion to int32 each (NaN gives 0, the infinities
// the int32 limits), then two instructions that saturate two integers to bytes and pack them
// beside the bytes already there.  Clamping and rounding with fp32 instructions (max, min, add
// of 1.5 * 2^23) and permuting the bytes together took eleven issue slots where this takes six.
__device__ __forceinline__ uint32_t requant_pack4(float z0, float z1, float z2, float z3)
{
    uint32_t hi, w;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(__float2int_rn(z3)), "r"(__float2int_rn(z2)), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(__float2int_rn(z1)), "r"(__float2int_rn(z0)), "r"(hi));
    return w;
}

// The next layer's transform on requantized bytes (producer-side SPARQ): four adjacent output
// channels per word, pairs (2j, 2j+1) inside it.  Kept out of line: the epilogue loops are hot
// and every variant inlined at every use made the kernels several times larger than the
// instruction caches, which the warp roles share.
static __device__ __noinline__ void next_xform_words(uint32_t *w, int count, int mode, int rnd, XformDev xf)
{
    const bool full = xf.rounds == 0 && xf.n != 4;   // 6opt / 7opt: the half-precision form
    for (int q = 0; q < count; ++q) {
        uint32_t x = w[q];
        if (mode == SPARQ_MODE_VSPARQ) {
            if (full) x = xform_word_fullset<SPARQ_MODE_VSPARQ>(x, xf);
            else if (xf.rounds == 0) x = rnd ? xform_word<SPARQ_MODE_VSPARQ, 4, true, false>(x, xf) : xform_word<SPARQ_MODE_VSPARQ, 4, false, false>(x, xf);
            else x = rnd ? xform_word<SPARQ_MODE_VSPARQ, 0, true, true>(x, xf) : xform_word<SPARQ_MODE_VSPARQ, 0, false, true>(x, xf);
        } else {
            if (full) x = xform_word_fullset<SPARQ_MODE_BSPARQ>(x, xf);
            else if (xf.rounds == 0) x = rnd ? xform_word<SPARQ_MODE_BSPARQ, 4, true, false>(x, xf) : xform_word<SPARQ_MODE_BSPARQ, 4, false, false>(x, xf);
            else x = rnd ? xform_word<SPARQ_MODE_BSPARQ, 0, true, true>(x, xf) : xform_word<SPARQ_MODE_BSPARQ, 0, false, true>(x, xf);
        }
        w[q] = x;
    }
}

// Per-thread view of the epilogue's outputs and constants.
struct EpiView {
    int64_t N;
    int32_t *acc_out;
    float *f32_out;
    uint8_t *u8_out;
    float inv_out_scale;
    bool need_f;      // a dequantized output is requested
    bool relu_op;     // the ReLU select has to be executed (see below)
    bool small_acc;   // |acc| < 2^22 guaranteed
    bool vec_ok;      // rows allow 16/32-byte vector stores
    bool u8_wide;     // 256-bit stores allowed on u8_out
    bool lean;        // only requantized bytes are wanted and whole 32-byte groups can be stored: see epi_chunk_u8
    int next_mode;    // SPARQ mode applied to the requantized bytes (producer-side transform)
    int next_rnd;
    XformDev next_xf;
    const uint8_t *residual;   // u8 identity tensor added before the ReLU, or nullptr
    float residual_scale;
};

template <class Args>
__device__ __forceinline__ EpiView make_epi_view(const Args &g)
{
    EpiView e;
    e.N = g.N;
    e.acc_out = g.acc_out;
    e.f32_out = g.f32_out;
    e.u8_out = g.u8_out;
    e.inv_out_scale = g.inv_out_scale;
    e.need_f = (g.f32_out != nullptr) || (g.u8_out != nullptr);
    // relu(y) * inv clamped to [0, 255] equals y * inv clamped when inv > 0, so the ReLU
    // select is only needed when the fp32 value itself is an output
    e.relu_op = g.relu && (g.f32_out != nullptr || !(g.inv_out_scale > 0.0f));
    // |acc| <= K * 255 * 128; below 2^22 the int -> float conversion is exact and can be
    // done with an integer add and a float subtract instead of the conversion unit
    e.small_acc = g.K * (255 * 128) < (1 << 22);
    e.vec_ok = (g.N % 32) == 0;
    e.u8_wide = (reinterpret_cast<uintptr_t>(g.u8_out) & 31u) == 0;
    e.lean = e.u8_out && !g.acc_out && !g.f32_out && !g.residual && g.next_mode == SPARQ_MODE_NONE && !e.relu_op &&
             e.vec_ok && e.u8_wide;
    e.next_mode = g.next_mode;
    e.next_rnd = g.next_rnd;
    e.next_xf = g.next_xf;
    e.residual = g.residual;
    e.residual_scale = g.residual_scale;
    return e;
}

// One thread's NV (32 or 16) consecutive accumulators of output row `row` (columns col0 ..
// col0+NV-1, tile-local column ct): optional raw store, dequantize, optional fp32 store,
// requantize and store.  v is overwritten.
// REG: scale and bias of the NV columns come from the caller's registers rs / rb instead of
// shared memory (shared-memory reads queue behind the tensor core's operand fetches).
template <int NV = 32, bool REG = false>
__device__ __forceinline__ void epi_chunk(const EpiView &e, uint32_t (&v)[NV], int64_t row, int64_t col0, int ct,
                                          const float *s_scale, const float *s_bias,
                                          const float *rs = nullptr, const float *rb = nullptr)
{
    static_assert(NV == 32 || NV == 16, "chunk width");
    constexpr int NQ = NV / 4;      // groups of four columns = words of packed bytes
    const int64_t off = row * e.N + col0;
    const bool full = e.vec_ok && (col0 + NV <= e.N);
    if (e.acc_out) {
        if (full) {
            int4 *dst = reinterpret_cast<int4 *>(e.acc_out + off);
#pragma unroll
            for (int q = 0; q < NQ; ++q)
                dst[q] = make_int4((int)v[4 * q], (int)v[4 * q + 1], (int)v[4 * q + 2], (int)v[4 * q + 3]);
        } else {
            for (int i = 0; i < NV && col0 + i < e.N; ++i) e.acc_out[off + i] = (int32_t)v[i];
        }
    }
    if (!e.need_f) return;
    // with a residual input the ReLU comes after the sum
    const int relu_first = e.residual ? 0 : (int)e.relu_op;
    // v[i] becomes the fp32 value's bits in place
    // scale and bias of 16 columns at a time: the eight 16-byte shared-memory reads are issued
    // together, so that their latencies (long while the tensor core is fetching operands)
    // overlap instead of adding up
#pragma unroll
    for (int h = 0; h < NV / 16; ++h) {
        float hs[16], hb[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (REG) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    hs[4 * q + j] = rs[16 * h + 4 * q + j];
                    hb[4 * q + j] = rb[16 * h + 4 * q + j];
                }
            } else {
                const float4 sc = *reinterpret_cast<const float4 *>(&s_scale[ct + 16 * h + 4 * q]);
                const float4 bi = *reinterpret_cast<const float4 *>(&s_bias[ct + 16 * h + 4 * q]);
                hs[4 * q] = sc.x; hs[4 * q + 1] = sc.y; hs[4 * q + 2] = sc.z; hs[4 * q + 3] = sc.w;
                hb[4 * q] = bi.x; hb[4 * q + 1] = bi.y; hb[4 * q + 2] = bi.z; hb[4 * q + 3] = bi.w;
            }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int c = 16 * h + i;
            v[c] = __float_as_uint(e.small_acc ? dequant<true>((int32_t)v[c], hs[i], hb[i], relu_first)
                                               : dequant<false>((int32_t)v[c], hs[i], hb[i], relu_first));
        }
    }
    if (e.residual) {
        uint32_t r[NQ];
        if (full) {
#pragma unroll
            for (int h = 0; h < NV / 16; ++h) {
                const uint4 rr = __ldg(reinterpret_cast<const uint4 *>(e.residual + off) + h);
                r[4 * h] = rr.x; r[4 * h + 1] = rr.y; r[4 * h + 2] = rr.z; r[4 * h + 3] = rr.w;
            }
        } else {
#pragma unroll
            for (int q = 0; q < NQ; ++q) r[q] = 0u;
            for (int i = 0; i < NV && col0 + i < e.N; ++i)
                r[i >> 2] |= (uint32_t)__ldg(e.residual + off + i) << (8 * (i & 3));
        }
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const float rv = __uint2float_rn((r[i >> 2] >> (8 * (i & 3))) & 0xFFu);
            float y = __fmaf_rn(rv, e.residual_scale, __uint_as_float(v[i]));
            if (e.relu_op) y = fmaxf(y, 0.0f);
            v[i] = __float_as_uint(y);
        }
    }
    if (e.f32_out) {
        if (full) {
            uint4 *dst = reinterpret_cast<uint4 *>(e.f32_out + off);
#pragma unroll
            for (int q = 0; q < NQ; ++q) dst[q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else {
            for (int i = 0; i < NV && col0 + i < e.N; ++i) e.f32_out[off + i] = __uint_as_float(v[i]);
        }
    }
    if (e.u8_out) {
        uint32_t w[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q)
            w[q] = requant_pack4(__fmul_rn(__uint_as_float(v[4 * q]), e.inv_out_scale),
                                 __fmul_rn(__uint_as_float(v[4 * q + 1]), e.inv_out_scale),
                                 __fmul_rn(__uint_as_float(v[4 * q + 2]), e.inv_out_scale),
                                 __fmul_rn(__uint_as_float(v[4 * q + 3]), e.inv_out_scale));
        if (e.next_mode != SPARQ_MODE_NONE) next_xform_words(w, NQ, e.next_mode, e.next_rnd, e.next_xf);
        if (full) {
            if constexpr (NV == 32) {
                if (e.u8_wide) {
                    st_global_v8(e.u8_out + off, w);
                } else {
                    uint4 *dst = reinterpret_cast<uint4 *>(e.u8_out + off);
                    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                }
            } else {
                *reinterpret_cast<uint4 *>(e.u8_out + off) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        } else {
            for (int i = 0; i < NV && col0 + i < e.N; ++i)
                e.u8_out[off + i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
        }
    }
}

// Two fp32 values in one 64-bit register and the packed arithmetic of sm_100: each instruction
// performs the IEEE round-to-nearest operation on both halves, so a pair of columns costs one
// issue slot where the scalar form costs two.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t r, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// The form every layer of a network uses -- requantized bytes only, no residual, full 32-column
// groups -- as straight-line code with nothing decided per element and the fp32 steps done two
// columns at a time: per accumulator an exact int -> float step, one fma, one multiply and the
// conversion back to an integer, then two saturating packs per four columns.  Same IEEE
// sequence per element as epi_chunk.
template <bool SMALL>
__device__ __forceinline__ void epi_chunk_u8(const EpiView &e, uint32_t (&v)[32], int64_t row, int64_t col0, int ct,
                                             const float *s_scale, const float *s_bias)
{
    const uint64_t inv2 = f2_pack(e.inv_out_scale, e.inv_out_scale);
    const uint64_t neg_magic2 = f2_pack(-12582912.0f, -12582912.0f);
    uint32_t w[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float4 sc = *reinterpret_cast<const float4 *>(&s_scale[ct + 4 * q]);
        const float4 bi = *reinterpret_cast<const float4 *>(&s_bias[ct + 4 * q]);
        float z[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int32_t a0 = (int32_t)v[4 * q + 2 * h], a1 = (int32_t)v[4 * q + 2 * h + 1];
            // (float)acc: exact through the add-based form when |acc| < 2^22
            const uint64_t t = SMALL ? f2_add(f2_pack(__int_as_float(a0 + 0x4B400000), __int_as_float(a1 + 0x4B400000)), neg_magic2)
                                     : f2_pack(__int2float_rn(a0), __int2float_rn(a1));
            const uint64_t y = f2_fma(t, h ? f2_pack(sc.z, sc.w) : f2_pack(sc.x, sc.y), h ? f2_pack(bi.z, bi.w) : f2_pack(bi.x, bi.y));
            f2_unpack(f2_mul(y, inv2), z[2 * h], z[2 * h + 1]);
        }
        w[q] = requant_pack4(z[0], z[1], z[2], z[3]);
    }
    st_global_v8(e.u8_out + row * e.N + col0, w);
}

// A warp's share of one accumulator: CW (16, 32, 64 or 128) columns starting at
// tensor-memory address taddr0 (tile-local column cbase), for this thread's output row.
// After the last load has landed in registers the warp hands the accumulator back by
// arriving on acc_empty_bar.
template <int CW>
__device__ __forceinline__ void epi_warp_columns(const EpiView &e, uint32_t taddr0, int cbase, int64_t row, bool row_ok,
                                                 int64_t n0, const float *s_scale, const float *s_bias,
                                                 uint32_t acc_empty_bar, int lane)
{
    if constexpr (CW == 16) {
        uint32_t v[16];
        tmem_ld_32x16_issue(taddr0, v);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty_bar);
        const int64_t col0 = n0 + cbase;
        if (row_ok && col0 < e.N) epi_chunk<16, false>(e, v, row, col0, cbase, s_scale, s_bias);
    } else {
        constexpr int CHUNKS = CW / 32;
#pragma unroll 1
        for (int ch = 0; ch < CHUNKS; ++ch) {
            uint32_t v[32];
            tmem_ld_32x32_issue(taddr0 + (uint32_t)(ch * 32), v);
            tmem_ld_wait();
            if (ch + 1 == CHUNKS) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty_bar);
            }
            const int ct = cbase + ch * 32;              // column inside the tile
            const int64_t col0 = n0 + ct;
            if (!row_ok || col0 >= e.N) continue;
            if (e.lean && col0 + 32 <= e.N) {
                if (e.small_acc) epi_chunk_u8<true>(e, v, row, col0, ct, s_scale, s_bias);
                else epi_chunk_u8<false>(e, v, row, col0, ct, s_scale, s_bias);
            } else {
                epi_chunk<32, false>(e, v, row, col0, ct, s_scale, s_bias);
            }
        }
    }
}

// Stages the scale and bias of columns n0 .. n0+bn-1 in shared memory (epilogue warps only).
template <int WARPS, class Args>
__device__ __forceinline__ void epi_stage_scale_bias(const Args &g, int64_t n0, int bn, int et,
                                                     float *s_scale, float *s_bias)
{
    epi_bar_sync<WARPS>();                      // previous readers are done
    for (int c = et; c < bn; c += WARPS * 32) {
        const int64_t col = n0 + c;
        const bool ok = col < g.N;
        s_scale[c] = ok ? __ldg(g.scale + col) : 0.0f;
        s_bias[c] = (ok && g.bias) ? __ldg(g.bias + col) : 0.0f;
    }
    epi_bar_sync<WARPS>();
}

// ---- the kernel ---------------------------------------------------------------------------

template <int BN, int BK>
struct TileCfg {
    static constexpr int kABytes = kBM * BK;
    static constexpr int kBBytes = BN * BK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStagesRaw = kSmemBudget / kStageBytes;
    static constexpr int kStages = kStagesRaw > 8 ? 8 : kStagesRaw;
    static constexpr int kTmemCols = (2 * BN < 32) ? 32 : 2 * BN;   // two accumulators
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024; // + alignment slack
};

template <int BN, int BK, int MODE, int XN, bool RND>
__global__ void __launch_bounds__(kGemmThreads, 1)
sparq_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const GemmArgs g)
{
    using Cfg = TileCfg<BN, BK>;
    constexpr int S = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[S], bar_xf[S], bar_empty[S];
    __shared__ __align__(8) uint64_t bar_acc_full[2], bar_acc_empty[2], bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_word;
    __shared__ __align__(16) float s_scale[BN], s_bias[BN];

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile uint32_t *abort_flag = &abort_word;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    auto a_stage = [&](int s) { return smem_base + (uint32_t)s * Cfg::kStageBytes; };
    auto b_stage = [&](int s) { return smem_base + (uint32_t)s * Cfg::kStageBytes + Cfg::kABytes; };

    // A tile's epilogue is mostly latency (barrier read, tensor-memory loads, stores).  On 64-wide
    // tiles, and on 128-wide tiles with a transform (eight epilogue warps), with one column tile and
    // only requantized bytes wanted, the epilogue warps split into two teams, one per accumulator
    // stage, each warp taking twice the columns of its lane quarter: two tiles' epilogues overlap.
    constexpr bool kTeamsPay = BN == 64 || (BN == 128 && MODE != SPARQ_MODE_NONE);
    const bool epi_teams = kTeamsPay && g.N <= BN && make_epi_view(g).lean;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_xf[s]), kXfTeamWarps);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bar_acc_full[a]), 1);
            mbar_init(smem_u32(&bar_acc_empty[a]), epi_teams ? epi_warps(MODE) / 2 : epi_warps(MODE));
        }
        mbar_init(smem_u32(&bar_done), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)Cfg::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    dep_launch();
    dep_wait();

    const int64_t m_tiles = (g.M + kBM - 1) / kBM;
    const int64_t n_tiles = (g.N + BN - 1) / BN;
    // tile indices fit 32 bits (the host refuses larger problems); a 64-bit division per tile
    // and thread costs more instructions than a tile's share of the epilogue arithmetic
    const uint32_t total_tiles = (uint32_t)(m_tiles * n_tiles);
    const uint32_t n_tiles32 = (uint32_t)n_tiles;
    const int kb_count = g.k_blocks;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t it = 0;   // running stage counter across tiles
            for (uint32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
                const uint32_t mt = (n_tiles32 == 1) ? tile : tile / n_tiles32, nt = tile - mt * n_tiles32;
                const int64_t m0 = (int64_t)mt * kBM;
                const int n0 = (int)(nt * BN);
                int base_w = 0, base_h = 0, base_n = 0;
                if (g.conv) {
                    const uint32_t hw = (uint32_t)(g.Ho * g.Wo), m032 = (uint32_t)m0;   // M of a convolution fits 31 bits
                    base_n = (int)(m032 / hw);
                    const int rem = (int)(m032 - (uint32_t)base_n * hw);
                    base_h = (rem / g.Wo) * g.stride_h - g.pad_h;
                    base_w = (rem % g.Wo) * g.stride_w - g.pad_w;
                }
                for (int kb = 0; kb < kb_count; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t use = it / S;
                    if (use > 0) mbar_wait(smem_u32(&bar_empty[s]), (use - 1) & 1, abort_flag, g.status, g.wait_limit);
                    if (*abort_flag) break;   // stop issuing copies once the CTA has given up
                    const uint32_t full = smem_u32(&bar_full[s]);
                    mbar_expect_tx(full, Cfg::kStageBytes);
                    int bx = kb * BK;
                    if (g.conv) {
                        // Channels past C arrive as zeros, so whatever the weight block holds
                        // there (the next tap's first bytes) adds nothing.
                        const int tap = kb / g.c_blocks, cb = kb % g.c_blocks;
                        tma_load_im2col_4d(a_stage(s), &map_a, full, cb * BK, base_w, base_h, base_n,
                                           (uint16_t)(tap % g.S), (uint16_t)(tap / g.S));
                        bx = tap * g.tap_k + cb * BK;
                    } else {
                        tma_load_2d(a_stage(s), &map_a, full, kb * BK, (int)m0);
                    }
                    tma_load_2d(b_stage(s), &map_b, full, bx, n0);
                }
                if (*abort_flag) break;
            }
            // After an abort: wait (bounded) for the copies this thread still has in
            // flight, so that none lands after the CTA has exited.
            if (*abort_flag) {
                const uint32_t first = it > (uint32_t)S ? it - S : 0;
                for (uint32_t j = first; j < it; ++j)
                    mbar_wait(smem_u32(&bar_full[j % S]), (j / S) & 1, abort_flag, g.status, g.wait_limit, true);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // The whole warp runs this loop converged and one elected lane issues, so that the
        // descriptor arithmetic (warp-uniform values only) can stay in the uniform datapath.
        {
            const uint32_t elected = elect_one();
            constexpr uint32_t idesc = make_idesc_i8(BN);
            // descriptors of stage 0; a stage adds its byte offset / 16 to the start-address field
            const uint64_t adesc0 = make_smem_desc<BK>(smem_base);
            const uint64_t bdesc0 = make_smem_desc<BK>(smem_base + Cfg::kABytes);
            uint32_t local_tile = 0;
            int s = 0;             // stage
            uint32_t ph = 0;       // its phase parity
            for (uint32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++local_tile) {
                const int acc = local_tile & 1;
                const uint32_t acc_use = local_tile >> 1;
                if (acc_use > 0) mbar_wait(smem_u32(&bar_acc_empty[acc]), (acc_use - 1) & 1, abort_flag, g.status, g.wait_limit);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < kb_count; ++kb) {
                    if (MODE == SPARQ_MODE_NONE) mbar_wait(smem_u32(&bar_full[s]), ph, abort_flag, g.status, g.wait_limit);
                    else mbar_wait(smem_u32(&bar_xf[s]), ph, abort_flag, g.status, g.wait_limit);
                    tc_fence_after();
                    const uint64_t st_off = (uint64_t)((uint32_t)s * (uint32_t)(Cfg::kStageBytes >> 4));
                    const uint64_t adesc = adesc0 + st_off, bdesc = bdesc0 + st_off;
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)
                        tc_mma_i8_if(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                                     (kb > 0 || k > 0) ? 1u : 0u, elected);
                    tc_commit_if(smem_u32(&bar_empty[s]), elected);       // stage reusable once these MMAs retire
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
                tc_commit_if(smem_u32(&bar_acc_full[acc]), elected);      // accumulator complete
            }
            // all tensor-core work of this CTA has retired before tensor memory is freed
            tc_commit_if(smem_u32(&bar_done), elected);
            mbar_wait(smem_u32(&bar_done), 0, abort_flag, g.status, g.wait_limit, true);
        }
        __syncwarp();
    } else if (warp < kFirstEpiWarp + epi_warps(MODE)) {
        // ================= epilogue =================
        constexpr int kEpi = epi_warps(MODE);
        constexpr int kColsPerWarp = BN / (kEpi / 4);        // the tile's columns are split over the warps of a quarter
        const int quarter = warp & 3;                        // tensor-memory lanes this warp may read
        const int part = (warp - kFirstEpiWarp) >> 2;        // which share of the tile's columns
        const int et = threadIdx.x - kFirstEpiWarp * 32;     // 0 .. kEpi * 32 - 1
        const EpiView ev = make_epi_view(g);
        uint32_t local_tile = 0;
        int64_t staged_nt = -1;
        if (epi_teams) {
            constexpr int kTeamWarps = kEpi / 2;
            constexpr int kTeamCols = BN / (kTeamWarps / 4);          // columns per warp
            epi_stage_scale_bias<kEpi>(g, 0, BN, et, s_scale, s_bias);
            const uint32_t team = (uint32_t)(warp - kFirstEpiWarp) / kTeamWarps;   // team t takes the tiles of parity t
            const int tcbase = (((warp - kFirstEpiWarp) % kTeamWarps) >> 2) * kTeamCols;
            for (uint32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++local_tile) {
                if ((local_tile & 1u) != team) continue;
                const int64_t row = (int64_t)tile * kBM + quarter * 32 + lane;    // one column tile: row tile = tile
                const bool row_ok = row < g.M;
                const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + team * BN + (uint32_t)tcbase;
                mbar_wait(smem_u32(&bar_acc_full[team]), (local_tile >> 1) & 1u, abort_flag, g.status, g.wait_limit);
                tc_fence_after();
#pragma unroll 1
                for (int ch = 0; ch < kTeamCols / 32; ++ch) {
                    uint32_t v[32];
                    tmem_ld_32x32_issue(taddr0 + (uint32_t)(ch * 32), v);
                    tmem_ld_wait();
                    if (ch + 1 == kTeamCols / 32) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[team]));
                    }
                    const int ct = tcbase + ch * 32;
                    if (!row_ok || ct >= (int)g.N) continue;          // N is a multiple of 32 here
                    if (ev.small_acc) epi_chunk_u8<true>(ev, v, row, ct, ct, s_scale, s_bias);
                    else epi_chunk_u8<false>(ev, v, row, ct, ct, s_scale, s_bias);
                }
            }
        } else
        for (uint32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++local_tile) {
            const uint32_t mt32 = (n_tiles32 == 1) ? tile : tile / n_tiles32;
            const int64_t mt = mt32, nt = tile - mt32 * n_tiles32;
            const int acc = local_tile & 1;
            const uint32_t acc_use = local_tile >> 1;
            if (ev.need_f && nt != staged_nt) {              // new column tile: new scale / bias
                staged_nt = nt;
                epi_stage_scale_bias<kEpi>(g, nt * BN, BN, et, s_scale, s_bias);
            }
            mbar_wait(smem_u32(&bar_acc_full[acc]), acc_use & 1, abort_flag, g.status, g.wait_limit);
            tc_fence_after();
            const int64_t row = mt * kBM + quarter * 32 + lane;
            const bool row_ok = row < g.M;
            const int cbase = part * kColsPerWarp;
            const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + cbase);
            epi_warp_columns<kColsPerWarp>(ev, taddr0, cbase, row, row_ok, nt * BN, s_scale, s_bias,
                                      smem_u32(&bar_acc_empty[acc]), lane);
        }
        if (warp == kFirstEpiWarp && lane == 0) {
        }
    } else if (MODE != SPARQ_MODE_NONE) {
        // ================= transform =================
        const int team = (warp - kFirstXfWarp) / kXfTeamWarps;
        const int xt = threadIdx.x - (kFirstXfWarp + team * kXfTeamWarps) * 32;   // 0 .. 127 inside the team
        constexpr int kXfThreads = kXfTeamWarps * 32;
        constexpr int kVecs = Cfg::kABytes / 16;
        constexpr int kPerThread = kVecs / kXfThreads;
        constexpr int kBatch = kPerThread < 4 ? kPerThread : 4;     // vectors in flight per thread
        static_assert(kVecs % kXfThreads == 0 && kPerThread % kBatch == 0, "A stage must split evenly over a team");
        const XformDev xf = g.xf;
        uint32_t it = 0;
        for (uint32_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
            for (int kb = 0; kb < kb_count; ++kb, ++it) {
                if ((int)(it & 1u) != team) continue;      // the other team's stage
                const int s = it % S;
                mbar_wait(smem_u32(&bar_full[s]), (it / S) & 1, abort_flag, g.status, g.wait_limit);
                const uint32_t base = a_stage(s) + (uint32_t)xt * 16u;
#pragma unroll
                for (int j0 = 0; j0 < kPerThread; j0 += kBatch) {
                    uint4 v[kBatch];
#pragma unroll
                    for (int j = 0; j < kBatch; ++j)
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w)
                                     : "r"(base + (uint32_t)((j0 + j) * kXfThreads * 16)));
#pragma unroll
                    for (int j = 0; j < kBatch; ++j) {
                        v[j].x = xform_fused<MODE, XN, RND>(v[j].x, xf);
                        v[j].y = xform_fused<MODE, XN, RND>(v[j].y, xf);
                        v[j].z = xform_fused<MODE, XN, RND>(v[j].z, xf);
                        v[j].w = xform_fused<MODE, XN, RND>(v[j].w, xf);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                                     :: "r"(base + (uint32_t)((j0 + j) * kXfThreads * 16)),
                                        "r"(v[j].x), "r"(v[j].y), "r"(v[j].z), "r"(v[j].w) : "memory");
                    }
                }
                fence_proxy_async_smem();       // generic-proxy writes visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_xf[s]));
            }
        }
        if (warp == kFirstXfWarp && lane == 0) {
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     :: "r"(tmem_base), "r"((uint32_t)Cfg::kTmemCols) : "memory");
    }
}

// Launch with programmatic stream serialization allowed (see dep_wait / dep_launch).
template <int THREADS = kGemmThreads, class Kernel, class... KernelArgs>
cudaError_t launch_pdl(Kernel kfn, int grid, int smem_bytes, cudaStream_t st, const KernelArgs &...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kfn, args...);
}

// Host launcher for one tile shape; picks the transform variant.  Defined once per
// (BN, BK) in its own translation unit.
template <int BN, int BK>
cudaError_t launch_gemm_shape(const CUtensorMap &ma, const CUtensorMap &mb, const GemmArgs &g,
                              int mode, int n, int rnd, int grid, cudaStream_t st);

#define SPARQ_LAUNCH_VARIANT(MODE_, XN_, RND_)                                                         \
    do {                                                                                               \
        auto kfn = sparq_gemm_kernel<BN, BK, MODE_, XN_, RND_>;                                        \
        static bool attr_set[64] = {};   /* per device ordinal */                                     \
        int dev_ = 0;                                                                                  \
        cudaError_t e_ = cudaGetDevice(&dev_);                                                         \
        if (e_ != cudaSuccess) return e_;                                                              \
        if (dev_ < 0 || dev_ >= 64 || !attr_set[dev_]) {                                               \
            e_ = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize,                \
                                      TileCfg<BN, BK>::kSmemBytes);                                    \
            if (e_ != cudaSuccess) return e_;                                                          \
            if (dev_ >= 0 && dev_ < 64) attr_set[dev_] = true;                                         \
        }                                                                                              \
        return launch_pdl(kfn, grid, TileCfg<BN, BK>::kSmemBytes, st, ma, mb, g);                      \
    } while (0)

#define SPARQ_DEFINE_GEMM_SHAPE(BN_, BK_)                                                              \
    template <>                                                                                        \
    cudaError_t launch_gemm_shape<BN_, BK_>(const CUtensorMap &ma, const CUtensorMap &mb,              \
                                            const GemmArgs &g, int mode, int n, int rnd, int grid,     \
                                            cudaStream_t st)                                           \
    {                                                                                                  \
        constexpr int BN = BN_, BK = BK_;                                                              \
        if (mode == SPARQ_MODE_NONE) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_NONE, 4, false);                  \
        if (mode == SPARQ_MODE_BSPARQ) {                                                               \
            if (n == 8) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_BSPARQ, 8, true);                              \
            if (n == 4) { if (rnd) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_BSPARQ, 4, true);                   \
                          else SPARQ_LAUNCH_VARIANT(SPARQ_MODE_BSPARQ, 4, false); }                    \
            if (rnd) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_BSPARQ, 0, true);                                 \
            else SPARQ_LAUNCH_VARIANT(SPARQ_MODE_BSPARQ, 0, false);                                    \
        }                                                                                              \
        if (n == 8) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_VSPARQ, 8, true);                                  \
        if (n == 4) { if (rnd) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_VSPARQ, 4, true);                       \
                      else SPARQ_LAUNCH_VARIANT(SPARQ_MODE_VSPARQ, 4, false); }                        \
        if (rnd) SPARQ_LAUNCH_VARIANT(SPARQ_MODE_VSPARQ, 0, true);                                     \
        else SPARQ_LAUNCH_VARIANT(SPARQ_MODE_VSPARQ, 0, false);                                        \
    }

}  // namespace sparq
