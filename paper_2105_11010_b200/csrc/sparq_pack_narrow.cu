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
// One thread owns one unit and computes the fields arithmetically from the packed transform
// (no tables): these widths are the paper's secondary configurations, and the kernels are
// plain streaming kernels.
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

__device__ __forceinline__ uint32_t byte_of(const uint4 &v, int i)
{
    const uint32_t w = i < 4 ? v.x : i < 8 ? v.y : i < 12 ? v.z : v.w;
    return (w >> (8 * (i & 3))) & 0xFFu;
}

template <int MODE, bool RND>
__global__ void __launch_bounds__(kThreads)
pack_narrow_kernel(const uint4 *__restrict__ in, uint8_t *__restrict__ data, uint8_t *__restrict__ ctrl, size_t units,
                   const NarrowArgs a)
{
    const int n = a.n, w2 = 2 * a.n;
    const uint32_t full = (1u << (8 - w2 + 1)) - 1u;   // lone window: every shift 0 .. 8-2n
    for (size_t u = (size_t)blockIdx.x * kThreads + threadIdx.x; u < units; u += (size_t)gridDim.x * kThreads) {
        const uint4 x = in[u];
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
                const int sl = placement_of(v, w2, full);
                field = v >> sl;
                state = (uint32_t)(a.ns * a.ns + (xb == 0 ? 0 : a.nl) + sl);
            } else {
                const int s1 = placement_of(qa, n, a.mask), s2 = placement_of(qb, n, a.mask);
                field = ((qa >> s1) << n) | (qb >> s2);
                state = (uint32_t)(__popc(a.mask & ((1u << s1) - 1u)) * a.ns + __popc(a.mask & ((1u << s2) - 1u)));
            }
            dword |= (unsigned long long)field << (j * w2);
            cword |= (unsigned long long)state << (j * a.cb);
        }
        uint8_t *d = data + (size_t)w2 * u;            // 2n bytes: even address
        for (int k = 0; k < w2; k += 2) *reinterpret_cast<uint16_t *>(d + k) = (uint16_t)(dword >> (8 * k));
        uint8_t *c = ctrl + (size_t)a.cb * u;
        for (int k = 0; k < a.cb; ++k) c[k] = (uint8_t)(cword >> (8 * k));
    }
}

__global__ void __launch_bounds__(kThreads)
unpack_narrow_kernel(const uint8_t *__restrict__ data, const uint8_t *__restrict__ ctrl, uint4 *__restrict__ out,
                     size_t units, const NarrowArgs a)
{
    const int n = a.n, w2 = 2 * a.n;
    const uint32_t fmask = (1u << w2) - 1u, nmask = (1u << n) - 1u, cmask = (1u << a.cb) - 1u;
    const uint32_t pairs = (uint32_t)(a.ns * a.ns);
    for (size_t u = (size_t)blockIdx.x * kThreads + threadIdx.x; u < units; u += (size_t)gridDim.x * kThreads) {
        unsigned long long dword = 0ull, cword = 0ull;
        const uint8_t *d = data + (size_t)w2 * u;
        for (int k = 0; k < w2; k += 2) dword |= (unsigned long long)*reinterpret_cast<const uint16_t *>(d + k) << (8 * k);
        const uint8_t *c = ctrl + (size_t)a.cb * u;
        for (int k = 0; k < a.cb; ++k) cword |= (unsigned long long)c[k] << (8 * k);
        uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t state = (uint32_t)(cword >> (j * a.cb)) & cmask;
            const uint32_t field = (uint32_t)(dword >> (j * w2)) & fmask;
            uint32_t qa, qb;
            if (state < pairs) {
                const uint32_t i1 = state / (uint32_t)a.ns, i2 = state - i1 * (uint32_t)a.ns;
                qa = (field >> n) << ((a.shift_of >> (4 * i1)) & 15u);
                qb = (field & nmask) << ((a.shift_of >> (4 * i2)) & 15u);
            } else {
                const uint32_t t = state - pairs, slot = t / (uint32_t)a.nl, sl = t - slot * (uint32_t)a.nl;
                const uint32_t v = field << sl;             // the two halves at shifts s_l + n and s_l
                qa = slot == 0 ? v : 0u;
                qb = slot == 0 ? 0u : v;
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
    if (x.mode == SPARQ_MODE_VSPARQ) {
        if (x.rnd) pack_narrow_kernel<SPARQ_MODE_VSPARQ, true><<<blocks, kThreads, 0, st>>>(src, data, ctrl, units, a);
        else pack_narrow_kernel<SPARQ_MODE_VSPARQ, false><<<blocks, kThreads, 0, st>>>(src, data, ctrl, units, a);
    } else {
        if (x.rnd) pack_narrow_kernel<SPARQ_MODE_BSPARQ, true><<<blocks, kThreads, 0, st>>>(src, data, ctrl, units, a);
        else pack_narrow_kernel<SPARQ_MODE_BSPARQ, false><<<blocks, kThreads, 0, st>>>(src, data, ctrl, units, a);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "pack_narrow_kernel launch");
    return SPARQ_OK;
}

int unpack_narrow(const uint8_t *data, const uint8_t *ctrl, uint8_t *out, size_t units, const XformArgs &x, cudaStream_t st)
{
    int blocks = 0, rc = grid_narrow(units, &blocks);
    if (rc != SPARQ_OK) return rc;
    unpack_narrow_kernel<<<blocks, kThreads, 0, st>>>(data, ctrl, reinterpret_cast<uint4 *>(out), units, narrow_args(x));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "unpack_narrow_kernel launch");
    return SPARQ_OK;
}

}  // namespace sparq
