// Packed SPARQ stream for 3- and 2-bit windows (Section 5.1).  Same planes as the 4-bit form
// in sparq_pack.cu, with narrower fields:
//
//   data plane   per unit of 16 activations, pair j's field (in1 << n) | in2 at bits
//                [j*2n, (j+1)*2n) of a little-endian integer of 2n bytes
//   ctrl plane   per unit, pair j's state at bits [j*cb, (j+1)*cb) of a little-endian integer
//                of cb bytes
//   state        two windows: id(shift1) * ns + id(shift2); a lone value (vSPARQ) owns the
//                pair's 2n-bit window at shift s_l in 0..8-2n and travels as its two n-bit
//                halves: ns*ns + s_l in the first slot, ns*ns + (9 - 2n) + s_l in the second
//
// One thread owns one unit: the packed transform first, then per value its placement from a
// 256-entry shared-memory table (the bit scans that would compute it run in a slow pipe), and
// per state its meaning from a 64-entry one on the way back.  A block's share of each plane is
// put together in shared memory and moved as whole words.  These widths are the paper's
// secondary configurations; the kernels are bound by their per-pair arithmetic and table
// reads, not by memory.
#include "sparq_common.cuh"

namespace sparq {

struct NarrowArgs {
    int n, ns, nl, cb;
    uint32_t mask;          // placement set
    uint32_t shift_of;      // shift of placement id i in nibble i
    XformDev xf;
};

namespace {

constexpr int kThreads = 256;

// Lowest allowed shift s with (q >> s) < 2^w: the placement that holds the window value q.
__device__ __forceinline__ int placement_of(uint32_t q, int w, uint32_t mask)
{
    const int p = 31 - __clz(q | 1u);                 // leading one (0 for q = 0)
    const int s0 = p - w + 1 > 0 ? p - w + 1 : 0;
    return s0 + __ffs((int)(mask >> s0)) - 1;          // valid sets contain the top placement, so a bit is set
}

// byte i (a compile-time index after unrolling) of a 16-byte vector
__device__ __forceinline__ uint32_t byte_of(const uint4 &v, int i)
{
    const uint32_t w = i < 4 ? v.x : i < 8 ? v.y : i < 12 ? v.z : v.w;
    return (w >> (8 * (i & 3))) & 0xFFu;
}

// `bytes` bytes between shared and global memory by the whole block, as 32-bit words plus a
// byte tail (both addresses 4-byte aligned: a block starts at a multiple of 256 units).
__device__ __forceinline__ void copy_out(uint8_t *dst, const uint8_t *src, uint32_t bytes)
{
    for (uint32_t o = threadIdx.x * 4u; o + 4u <= bytes; o += kThreads * 4u)
        *reinterpret_cast<uint32_t *>(dst + o) = *reinterpret_cast<const uint32_t *>(src + o);
    if (threadIdx.x < (bytes & 3u)) dst[(bytes & ~3u) + threadIdx.x] = src[(bytes & ~3u) + threadIdx.x];
}
__device__ __forceinline__ void copy_in(uint8_t *dst, const uint8_t *src, uint32_t bytes)
{
    for (uint32_t o = threadIdx.x * 4u; o + 4u <= bytes; o += kThreads * 4u)
        *reinterpret_cast<uint32_t *>(dst + o) = __ldcs(reinterpret_cast<const uint32_t *>(src + o));
    if (threadIdx.x < (bytes & 3u)) dst[(bytes & ~3u) + threadIdx.x] = src[(bytes & ~3u) + threadIdx.x];
}

template <int MODE, bool RND, int N>
__global__ void __launch_bounds__(kThreads)
pack_narrow_kernel(const uint4 *__restrict__ in, uint8_t *__restrict__ data, uint8_t *__restrict__ ctrl, size_t units,
                   const NarrowArgs a)
{
    // a block's 256 units occupy 256 * 2n and 256 * cb contiguous bytes of the two planes: they are
    // put together in shared memory and written as whole words
    __shared__ __align__(16) uint8_t s_data[kThreads * 8], s_ctrl[kThreads * 8];
    constexpr int n = N, w2 = 2 * N;
    constexpr uint32_t full = (1u << (8 - w2 + 1)) - 1u;   // lone window: every shift 0 .. 8-2n
    // placement (and its rank in the set) of every window value, looked up per byte: the bit
    // scans that compute them run in a slow pipe
    __shared__ uint8_t s_place[256], s_lone[256];
    {
        const uint32_t v = threadIdx.x;                    // kThreads == 256
        const int s1 = placement_of(v, n, a.mask);
        s_place[v] = (uint8_t)(s1 | (__popc(a.mask & ((1u << s1) - 1u)) << 4));
        s_lone[v] = (uint8_t)placement_of(v, w2, full);
    }
    __syncthreads();
    for (size_t base = (size_t)blockIdx.x * kThreads; base < units; base += (size_t)gridDim.x * kThreads) {
        const size_t u = base + threadIdx.x;
        const bool live = u < units;
        const uint4 x = live ? in[u] : make_uint4(0u, 0u, 0u, 0u);
        uint4 q;
        q.x = xform_word<MODE, 0, RND, true>(x.x, a.xf);
        q.y = xform_word<MODE, 0, RND, true>(x.y, a.xf);
        q.z = xform_word<MODE, 0, RND, true>(x.z, a.xf);
        q.w = xform_word<MODE, 0, RND, true>(x.w, a.xf);
        unsigned long long dword = 0ull, cword = 0ull;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t xa = byte_of(x, 2 * j), xb = byte_of(x, 2 * j + 1);
            const uint32_t qa = byte_of(q, 2 * j), qb = byte_of(q, 2 * j + 1);
            uint32_t field, state;
            if (MODE == SPARQ_MODE_VSPARQ && (xa == 0 || xb == 0)) {
                const uint32_t v = xb == 0 ? qa : qb;
                const uint32_t sl = s_lone[v];
                field = v >> sl;
                state = (uint32_t)(a.ns * a.ns + (xb == 0 ? 0 : a.nl)) + sl;
            } else {
                const uint32_t p1 = s_place[qa], p2 = s_place[qb];
                field = ((qa >> (p1 & 15u)) << n) | (qb >> (p2 & 15u));
                state = (p1 >> 4) * (uint32_t)a.ns + (p2 >> 4);
            }
            dword |= (unsigned long long)field << (j * w2);
            cword |= (unsigned long long)state << (j * a.cb);
        }
        uint8_t *d = s_data + w2 * threadIdx.x;        // 2n bytes: even address
        for (int k = 0; k < w2; k += 2) *reinterpret_cast<uint16_t *>(d + k) = (uint16_t)(dword >> (8 * k));
        uint8_t *c = s_ctrl + a.cb * threadIdx.x;
        for (int k = 0; k < a.cb; ++k) c[k] = (uint8_t)(cword >> (8 * k));
        __syncthreads();
        const size_t left = units - base;
        const uint32_t cnt = (uint32_t)(left < (size_t)kThreads ? left : (size_t)kThreads);
        copy_out(data + (size_t)w2 * base, s_data, cnt * (uint32_t)w2);
        copy_out(ctrl + (size_t)a.cb * base, s_ctrl, cnt * (uint32_t)a.cb);
        __syncthreads();
    }
}

template <int N>
__global__ void __launch_bounds__(kThreads)
unpack_narrow_kernel(const uint8_t *__restrict__ data, const uint8_t *__restrict__ ctrl, uint4 *__restrict__ out,
                     size_t units, const NarrowArgs a)
{
    constexpr int n = N, w2 = 2 * N;
    const uint32_t fmask = (1u << w2) - 1u, nmask = (1u << n) - 1u, cmask = (1u << a.cb) - 1u;
    // what a state means, looked up: bit 7 clear -> the two windows' shifts in the nibbles;
    // bit 7 set -> a lone value, its shift in bits 0-3 and its slot in bit 4
    __shared__ uint8_t s_dec[64];
    if (threadIdx.x < 64) {
        const uint32_t state = threadIdx.x, pairs0 = (uint32_t)(a.ns * a.ns);
        uint32_t d;
        if (state < pairs0) {
            const uint32_t i1 = state / (uint32_t)a.ns, i2 = state - i1 * (uint32_t)a.ns;
            d = ((a.shift_of >> (4 * i1)) & 15u) | (((a.shift_of >> (4 * i2)) & 15u) << 4);
        } else {
            const uint32_t t = state - pairs0, slot = t / (uint32_t)a.nl, sl = t - slot * (uint32_t)a.nl;
            d = 0x80u | ((slot & 1u) << 4) | (sl & 15u);
        }
        s_dec[state] = (uint8_t)d;
    }
    __shared__ __align__(16) uint8_t s_data[kThreads * 8], s_ctrl[kThreads * 8];
    for (size_t base = (size_t)blockIdx.x * kThreads; base < units; base += (size_t)gridDim.x * kThreads) {
        const size_t left = units - base;
        const uint32_t cnt = (uint32_t)(left < (size_t)kThreads ? left : (size_t)kThreads);
        __syncthreads();
        copy_in(s_data, data + (size_t)w2 * base, cnt * (uint32_t)w2);
        copy_in(s_ctrl, ctrl + (size_t)a.cb * base, cnt * (uint32_t)a.cb);
        __syncthreads();
        const size_t u = base + threadIdx.x;
        if (u >= units) continue;
        unsigned long long dword = 0ull, cword = 0ull;
        const uint8_t *d = s_data + w2 * threadIdx.x;
        for (int k = 0; k < w2; k += 2) dword |= (unsigned long long)*reinterpret_cast<const uint16_t *>(d + k) << (8 * k);
        const uint8_t *c = s_ctrl + a.cb * threadIdx.x;
        for (int k = 0; k < a.cb; ++k) cword |= (unsigned long long)c[k] << (8 * k);
        uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t state = (uint32_t)(cword >> (j * a.cb)) & cmask;
            const uint32_t field = (uint32_t)(dword >> (j * w2)) & fmask;
            uint32_t qa, qb;
            const uint32_t d = s_dec[state & 63u];
            if (!(d & 0x80u)) {
                qa = (field >> n) << (d & 15u);
                qb = (field & nmask) << (d >> 4);
            } else {
                const uint32_t v = field << (d & 15u);      // the two halves at shifts s_l + n and s_l
                qa = (d & 0x10u) ? 0u : v;
                qb = (d & 0x10u) ? v : 0u;
            }
            o[j >> 1] |= ((qa & 0xFFu) | ((qb & 0xFFu) << 8)) << (16 * (j & 1));
        }
        out[u] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

int grid_narrow(size_t units, int *blocks)
{
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");
    const size_t want = (units + kThreads - 1) / kThreads, cap = (size_t)sms * 16;
    *blocks = (int)(want < cap ? want : cap);
    return SPARQ_OK;
}

}  // namespace

int narrow_states(const XformArgs &x)
{
    const int ns = __builtin_popcount(x.mask);
    return ns * ns + (x.mode == SPARQ_MODE_VSPARQ ? 2 * (9 - 2 * x.n) : 0);
}

int narrow_ctrl_bits(const XformArgs &x)
{
    int bits = 0;
    while ((1 << bits) < narrow_states(x)) ++bits;
    return bits;
}

static NarrowArgs narrow_args(const XformArgs &x)
{
    NarrowArgs a;
    a.n = x.n;
    a.ns = __builtin_popcount(x.mask);
    a.nl = 9 - 2 * x.n;
    a.cb = narrow_ctrl_bits(x);
    a.mask = x.mask;
    a.shift_of = 0u;
    int r = 0;
    for (int s = 0; s <= 8 - x.n; ++s)
        if ((x.mask >> s) & 1u) a.shift_of |= (uint32_t)s << (4 * r++);
    a.xf = XformDev{x.widen_c, x.widen_rounds, x.n};
    return a;
}

int pack_narrow(const uint8_t *in, uint8_t *data, uint8_t *ctrl, size_t units, const XformArgs &x, cudaStream_t st)
{
    int blocks = 0, rc = grid_narrow(units, &blocks);
    if (rc != SPARQ_OK) return rc;
    const NarrowArgs a = narrow_args(x);
    const uint4 *src = reinterpret_cast<const uint4 *>(in);
#define SPARQ_PACK_NARROW(MODE_, RND_)                                                                          \
    do {                                                                                                        \
        if (x.n == 3) pack_narrow_kernel<MODE_, RND_, 3><<<blocks, kThreads, 0, st>>>(src, data, ctrl, units, a); \
        else pack_narrow_kernel<MODE_, RND_, 2><<<blocks, kThreads, 0, st>>>(src, data, ctrl, units, a);          \
    } while (0)
    if (x.mode == SPARQ_MODE_VSPARQ) {
        if (x.rnd) SPARQ_PACK_NARROW(SPARQ_MODE_VSPARQ, true);
        else SPARQ_PACK_NARROW(SPARQ_MODE_VSPARQ, false);
    } else {
        if (x.rnd) SPARQ_PACK_NARROW(SPARQ_MODE_BSPARQ, true);
        else SPARQ_PACK_NARROW(SPARQ_MODE_BSPARQ, false);
    }
#undef SPARQ_PACK_NARROW
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "pack_narrow_kernel launch");
    return SPARQ_OK;
}

int unpack_narrow(const uint8_t *data, const uint8_t *ctrl, uint8_t *out, size_t units, const XformArgs &x, cudaStream_t st)
{
    int blocks = 0, rc = grid_narrow(units, &blocks);
    if (rc != SPARQ_OK) return rc;
    if (x.n == 3) unpack_narrow_kernel<3><<<blocks, kThreads, 0, st>>>(data, ctrl, reinterpret_cast<uint4 *>(out), units, narrow_args(x));
    else unpack_narrow_kernel<2><<<blocks, kThreads, 0, st>>>(data, ctrl, reinterpret_cast<uint4 *>(out), units, narrow_args(x));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "unpack_narrow_kernel launch");
    return SPARQ_OK;
}

}  // namespace sparq
