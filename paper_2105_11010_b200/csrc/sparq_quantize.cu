// Standalone bSPARQ / vSPARQ transform (Sections 3.1-3.2): uint8 in, uint8 out.
//
// Fast path: the tensor is a flat array of 16-byte vectors.  With an even row length
// every pair (2j, 2j+1) of a row is also an aligned byte pair of the flat array, so rows
// need no special care.  Each thread streams kVec independent 16-byte loads, transforms
// the sixteen 32-bit words in registers and streams them back; the kernel is bound by
// HBM traffic (one byte read, one written per activation).
//
// Generic path: one thread per pair with the scalar form of the same definitions; used
// for odd row lengths and unaligned buffers.
#include "sparq_common.cuh"

namespace sparq {

constexpr int kThreads = 256;
constexpr int kVec = 4;  // 16-byte vectors per thread per iteration

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream(uint4 *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <int MODE, int N, bool RND, bool WIDEN>
__global__ void __launch_bounds__(kThreads)
quantize_vec_kernel(const uint4 *in, uint4 *out, size_t nvec, XformDev d)
{
    const size_t tile = (size_t)kThreads * kVec;
    for (size_t base = (size_t)blockIdx.x * tile; base < nvec; base += (size_t)gridDim.x * tile) {
        uint4 v[kVec];
        size_t idx[kVec];
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            idx[j] = base + (size_t)j * kThreads + threadIdx.x;
            if (idx[j] < nvec) v[j] = ld_stream(in + idx[j]);
        }
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            if (idx[j] < nvec) {
                uint4 o;
                o.x = xform_word<MODE, N, RND, WIDEN>(v[j].x, d);
                o.y = xform_word<MODE, N, RND, WIDEN>(v[j].y, d);
                o.z = xform_word<MODE, N, RND, WIDEN>(v[j].z, d);
                o.w = xform_word<MODE, N, RND, WIDEN>(v[j].w, d);
                st_stream(out + idx[j], o);
            }
        }
    }
}

// ---- scalar definitions (generic path) -----------------------------------------------

// One activation: leading one -> lowest allowed placement that covers it -> trim / round.
__device__ unsigned scalar_window(unsigned x, int w, unsigned mask, int rnd)
{
    if (x == 0) return 0;
    int p = 31 - __clz((int)x);
    int s = p - w + 1;
    if (s < 0) s = 0;
    while (!((mask >> s) & 1u)) ++s;          // the top placement is always allowed
    unsigned q = (x >> s) << s;
    if (rnd && s > 0 && ((x >> (s - 1)) & 1u)) {
        unsigned up = q + (1u << s);
        if (up <= 255u) q = up;               // otherwise stay at the all-ones top window
    }
    return q;
}

__global__ void quantize_pair_kernel(const uint8_t *in, uint8_t *out,
                                     size_t rows, size_t row_len, XformArgs a)
{
    const size_t pairs_per_row = (row_len + 1) / 2;
    const size_t total = rows * pairs_per_row;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i / pairs_per_row, j = i % pairs_per_row;
        size_t k0 = r * row_len + 2 * j;
        bool has_b = (2 * j + 1) < row_len;
        unsigned x0 = in[k0], x1 = has_b ? in[k0 + 1] : 0u;
        unsigned q0, q1;
        if (a.mode == SPARQ_MODE_NONE) {
            q0 = x0; q1 = x1;
        } else if (a.mode == SPARQ_MODE_VSPARQ && (x0 == 0 || x1 == 0)) {
            // the lone non-zero owns 2n bits, at any shift 0 .. 8-2n
            int w2 = 2 * a.n;
            unsigned full = (1u << (8 - w2 + 1)) - 1u;
            q0 = (w2 >= 8) ? x0 : scalar_window(x0, w2, full, a.rnd);
            q1 = (w2 >= 8) ? x1 : scalar_window(x1, w2, full, a.rnd);
        } else {
            q0 = scalar_window(x0, a.n, a.mask, a.rnd);
            q1 = scalar_window(x1, a.n, a.mask, a.rnd);
        }
        out[k0] = (uint8_t)q0;
        if (has_b) out[k0 + 1] = (uint8_t)q1;
    }
}

template <int MODE, int N>
static cudaError_t launch_vec(const uint4 *in, uint4 *out, size_t nvec, const XformArgs &a,
                              int blocks, cudaStream_t st)
{
    XformDev d{a.widen_c, a.widen_rounds, a.n};
    const bool widen = a.widen_rounds > 0;   // restricted placement set
    if (a.rnd && widen) quantize_vec_kernel<MODE, N, true, true><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    else if (a.rnd) quantize_vec_kernel<MODE, N, true, false><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    else if (widen) quantize_vec_kernel<MODE, N, false, true><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    else quantize_vec_kernel<MODE, N, false, false><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    return cudaGetLastError();
}

template <int MODE>
static cudaError_t launch_vec_n(const uint4 *in, uint4 *out, size_t nvec, const XformArgs &a,
                                int blocks, cudaStream_t st)
{
    switch (a.n) {
    case 2: return launch_vec<MODE, 2>(in, out, nvec, a, blocks, st);
    case 3: return launch_vec<MODE, 3>(in, out, nvec, a, blocks, st);
    default: return launch_vec<MODE, 4>(in, out, nvec, a, blocks, st);
    }
}

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_quantize(const uint8_t *in, uint8_t *out, size_t rows, size_t row_len,
                              const sparq_params *p, void *stream)
{
    XformArgs a;
    int rc = validate_params(p, &a);
    if (rc != SPARQ_OK) return rc;
    if (rows == 0 || row_len == 0) return SPARQ_OK;
    if (!in || !out) return set_error(SPARQ_ERR_INVALID_ARG, "in/out pointer is NULL");
    if (rows > ((size_t)1 << 62) / row_len) return set_error(SPARQ_ERR_INVALID_ARG, "rows * row_len overflows");
    const size_t total = rows * row_len;
    if (in != out) {
        const uint8_t *lo = in < (const uint8_t *)out ? in : out;
        const uint8_t *hi = in < (const uint8_t *)out ? out : in;
        if (lo + total > hi) return set_error(SPARQ_ERR_INVALID_ARG, "in and out overlap partially");
    }
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");

    const bool pairs_flat = (a.mode != SPARQ_MODE_VSPARQ) || (row_len % 2 == 0);
    const bool aligned = (((uintptr_t)in | (uintptr_t)out) & 15u) == 0;
    size_t done = 0;
    if (pairs_flat && aligned && total >= 16) {
        const size_t nvec = total / 16;
        const size_t tile = (size_t)kThreads * kVec;
        size_t want = (nvec + tile - 1) / tile;
        size_t cap = (size_t)sms * 64;   // grid-stride beyond this many blocks
        int blocks = (int)(want < cap ? want : cap);
        const uint4 *vi = (const uint4 *)in;
        uint4 *vo = (uint4 *)out;
        if (a.mode == SPARQ_MODE_NONE) e = launch_vec<SPARQ_MODE_NONE, 4>(vi, vo, nvec, a, blocks, st);
        else if (a.mode == SPARQ_MODE_BSPARQ) e = launch_vec_n<SPARQ_MODE_BSPARQ>(vi, vo, nvec, a, blocks, st);
        else e = launch_vec_n<SPARQ_MODE_VSPARQ>(vi, vo, nvec, a, blocks, st);
        if (e != cudaSuccess) return cuda_error(e, "quantize_vec_kernel launch");
        done = nvec * 16;
        if (done == total) return SPARQ_OK;
    }
    // Remainder (or everything, when the fast path does not apply).  With pairs_flat the
    // remaining bytes start at an even offset and form one pseudo-row.
    size_t g_rows = pairs_flat ? 1 : rows;
    size_t g_len = pairs_flat ? total - done : row_len;
    size_t npairs = g_rows * ((g_len + 1) / 2);
    size_t want = (npairs + 255) / 256;
    size_t cap = (size_t)sms * 32;
    int blocks = (int)(want < cap ? want : cap);
    if (blocks < 1) blocks = 1;
    quantize_pair_kernel<<<blocks, 256, 0, st>>>(in + done, out + done, g_rows, g_len, a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "quantize_pair_kernel launch");
    return SPARQ_OK;
}
