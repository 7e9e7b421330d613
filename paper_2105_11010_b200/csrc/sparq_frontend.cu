// Uniform min-max quantization of a layer's tensors (Section 5 of the paper): the step
// that produces the u8 activations and s8 weights the SPARQ kernels consume.
//   activations  unsigned symmetric per layer:  q = clamp(rint(x * (255 / max)), 0, 255)
//   weights      signed symmetric per kernel:   q = clamp(rint(w * (127 / max_j)), -127, 127)
// with max the largest magnitude (gathered over calibration batches by sparq_absmax, which
// folds each batch into a running maximum on the device).  All three kernels are
// streaming kernels bound by HBM traffic; fp32, one IEEE operation per step.
#include "sparq_common.cuh"

namespace sparq {

namespace {

constexpr int kThreads = 256;
constexpr int kVec = 4;   // 16-byte vectors in flight per thread

__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// bf16 is the top half of an fp32: widening is a shift
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// largest magnitude of the 4 (fp32) or 8 (bf16) elements of a vector; fmaxf skips NaNs
template <bool BF16>
__device__ __forceinline__ float vec_absmax(uint4 v, float m)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (BF16) {
            m = fmaxf(m, fabsf(bf16_lo(w[i])));
            m = fmaxf(m, fabsf(bf16_hi(w[i])));
        } else {
            m = fmaxf(m, fabsf(__uint_as_float(w[i])));
        }
    }
    return m;
}

template <bool BF16>
__device__ __forceinline__ float elem(const void *x, size_t i)
{
    if (BF16) return __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(x)[i] << 16);
    return reinterpret_cast<const float *>(x)[i];
}

// Block-wide maximum of non-negative floats (their bit patterns order like unsigned ints).
__device__ __forceinline__ uint32_t block_max_bits(float m, uint32_t *s_red)
{
    uint32_t b = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(m));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s_red[warp] = b;
    __syncthreads();
    b = (threadIdx.x < blockDim.x / 32) ? s_red[threadIdx.x] : 0u;
    if (warp == 0) b = __reduce_max_sync(0xFFFFFFFFu, b);
    return b;   // valid in warp 0
}

// max_inout = max(max_inout, max |x|): one atomic per block on the running maximum
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
absmax_kernel(const void *__restrict__ x, size_t n, float *max_inout)
{
    __shared__ uint32_t s_red[kThreads / 32];
    constexpr int kPer = BF16 ? 8 : 4;
    const size_t nvec = n / kPer;
    const uint4 *xv = reinterpret_cast<const uint4 *>(x);
    float m = 0.0f;
    const size_t tile = (size_t)kThreads * kVec;
    for (size_t base = (size_t)blockIdx.x * tile; base < nvec; base += (size_t)gridDim.x * tile) {
        uint4 v[kVec];
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            const size_t i = base + (size_t)j * kThreads + threadIdx.x;
            v[j] = i < nvec ? ld_stream16(xv + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kVec; ++j) m = vec_absmax<BF16>(v[j], m);
    }
    if (blockIdx.x == 0)   // the elements after the last whole vector
        for (size_t i = nvec * kPer + threadIdx.x; i < n; i += kThreads) m = fmaxf(m, fabsf(elem<BF16>(x, i)));
    const uint32_t b = block_max_bits(m, s_red);
    if (threadIdx.x == 0 && b) atomicMax(reinterpret_cast<unsigned int *>(max_inout), b);
}

// clamp(rint(z), 0, 255) as the low byte of a float: clamping first commutes with the
// rounding (integer bounds; NaN clamps to 0), and adding 1.5 * 2^23 rounds to nearest even
__device__ __forceinline__ uint32_t quant_u8_bits(float x, float inv)
{
    float z = __fmul_rn(x, inv);
    z = fminf(fmaxf(z, 0.0f), 255.0f);
    return __float_as_uint(__fadd_rn(z, 12582912.0f));
}

__device__ __forceinline__ uint32_t bytes4(uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    return prmt(prmt(a, b, 0x0040u), prmt(c, d, 0x0040u), 0x5410u);
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads)
quantize_act_kernel(const void *__restrict__ x, size_t n, const float *__restrict__ max_dev, uint8_t *__restrict__ out)
{
    constexpr int kPer = BF16 ? 8 : 4;
    const float mx = __ldg(max_dev);
    const float inv = mx > 0.0f ? __fdiv_rn(255.0f, mx) : 0.0f;
    const size_t nvec = n / kPer;
    const uint4 *xv = reinterpret_cast<const uint4 *>(x);
    const size_t tile = (size_t)kThreads * kVec;
    for (size_t base = (size_t)blockIdx.x * tile; base < nvec; base += (size_t)gridDim.x * tile) {
        uint4 v[kVec];
        size_t idx[kVec];
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            idx[j] = base + (size_t)j * kThreads + threadIdx.x;
            if (idx[j] < nvec) v[j] = ld_stream16(xv + idx[j]);
        }
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            if (idx[j] >= nvec) continue;
            if (BF16) {
                const uint32_t lo = bytes4(quant_u8_bits(bf16_lo(v[j].x), inv), quant_u8_bits(bf16_hi(v[j].x), inv),
                                           quant_u8_bits(bf16_lo(v[j].y), inv), quant_u8_bits(bf16_hi(v[j].y), inv));
                const uint32_t hi = bytes4(quant_u8_bits(bf16_lo(v[j].z), inv), quant_u8_bits(bf16_hi(v[j].z), inv),
                                           quant_u8_bits(bf16_lo(v[j].w), inv), quant_u8_bits(bf16_hi(v[j].w), inv));
                __stcs(reinterpret_cast<uint2 *>(out) + idx[j], make_uint2(lo, hi));
            } else {
                const uint32_t q = bytes4(quant_u8_bits(__uint_as_float(v[j].x), inv), quant_u8_bits(__uint_as_float(v[j].y), inv),
                                          quant_u8_bits(__uint_as_float(v[j].z), inv), quant_u8_bits(__uint_as_float(v[j].w), inv));
                __stcs(reinterpret_cast<uint32_t *>(out) + idx[j], q);
            }
        }
    }
    if (blockIdx.x == 0)
        for (size_t i = nvec * kPer + threadIdx.x; i < n; i += kThreads)
            out[i] = (uint8_t)quant_u8_bits(elem<BF16>(x, i), inv);
}

// One block per kernel (output channel): its largest magnitude, then its int8 row.
__global__ void __launch_bounds__(kThreads)
quantize_weight_kernel(const float *__restrict__ w, int64_t k, int8_t *__restrict__ out, float *__restrict__ scale_out)
{
    __shared__ uint32_t s_red[kThreads / 32];
    __shared__ float s_max;
    const float *row = w + (int64_t)blockIdx.x * k;
    int8_t *orow = out + (int64_t)blockIdx.x * k;
    float m = 0.0f;
    for (int64_t i = threadIdx.x; i < k; i += kThreads) m = fmaxf(m, fabsf(row[i]));
    const uint32_t b = block_max_bits(m, s_red);
    if (threadIdx.x == 0) s_max = __uint_as_float(b);
    __syncthreads();
    const float a = s_max;
    const float inv = a > 0.0f ? __fdiv_rn(127.0f, a) : 0.0f;
    for (int64_t i = threadIdx.x; i < k; i += kThreads) {
        float z = __fmul_rn(row[i], inv);
        z = fminf(fmaxf(z, -127.0f), 127.0f);                 // NaN -> -127 -> fixed below
        int q = __float2int_rn(z);
        if (row[i] != row[i]) q = 0;
        orow[i] = (int8_t)q;
    }
    if (threadIdx.x == 0) scale_out[blockIdx.x] = __fdiv_rn(a, 127.0f);
}

int stream_grid(size_t nvec, int *blocks)
{
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");
    const size_t tile = (size_t)kThreads * kVec;
    size_t want = (nvec + tile - 1) / tile;
    if (want < 1) want = 1;
    const size_t cap = (size_t)sms * 32;
    *blocks = (int)(want < cap ? want : cap);
    return SPARQ_OK;
}

int check_dtype(int dtype)
{
    if (dtype != SPARQ_DTYPE_F32 && dtype != SPARQ_DTYPE_BF16)
        return set_error(SPARQ_ERR_INVALID_ARG, "dtype %d is neither SPARQ_DTYPE_F32 nor SPARQ_DTYPE_BF16", dtype);
    return SPARQ_OK;
}

}  // namespace

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_absmax(const void *x, int dtype, size_t n, float *max_inout, void *stream)
{
    int rc = check_dtype(dtype);
    if (rc != SPARQ_OK) return rc;
    if (!max_inout) return set_error(SPARQ_ERR_INVALID_ARG, "max_inout is NULL");
    if (n == 0) return SPARQ_OK;
    if (!x) return set_error(SPARQ_ERR_INVALID_ARG, "x is NULL");
    if (((uintptr_t)x & 15u) || ((uintptr_t)max_inout & 3u))
        return set_error(SPARQ_ERR_UNSUPPORTED, "x must be 16-byte aligned and max_inout 4-byte aligned");
    const bool bf16 = dtype == SPARQ_DTYPE_BF16;
    int blocks = 0;
    if ((rc = stream_grid(n / (bf16 ? 8 : 4), &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (bf16) absmax_kernel<true><<<blocks, kThreads, 0, st>>>(x, n, max_inout);
    else absmax_kernel<false><<<blocks, kThreads, 0, st>>>(x, n, max_inout);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "absmax_kernel launch");
    return SPARQ_OK;
}

extern "C" int sparq_quantize_act_u8(const void *x, int dtype, size_t n, const float *max_dev, uint8_t *out,
                                     void *stream)
{
    int rc = check_dtype(dtype);
    if (rc != SPARQ_OK) return rc;
    if (!max_dev) return set_error(SPARQ_ERR_INVALID_ARG, "max_dev is NULL");
    if (n == 0) return SPARQ_OK;
    if (!x || !out) return set_error(SPARQ_ERR_INVALID_ARG, "x/out pointer is NULL");
    if ((((uintptr_t)x | (uintptr_t)out) & 15u) || ((uintptr_t)max_dev & 3u))
        return set_error(SPARQ_ERR_UNSUPPORTED, "x and out must be 16-byte aligned and max_dev 4-byte aligned");
    const bool bf16 = dtype == SPARQ_DTYPE_BF16;
    int blocks = 0;
    if ((rc = stream_grid(n / (bf16 ? 8 : 4), &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (bf16) quantize_act_kernel<true><<<blocks, kThreads, 0, st>>>(x, n, max_dev, out);
    else quantize_act_kernel<false><<<blocks, kThreads, 0, st>>>(x, n, max_dev, out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "quantize_act_kernel launch");
    return SPARQ_OK;
}

extern "C" int sparq_quantize_weight_s8(const float *w, int64_t cout, int64_t k, int8_t *out, float *scale_out,
                                        void *stream)
{
    if (cout < 0 || k < 0) return set_error(SPARQ_ERR_INVALID_ARG, "negative dimension");
    if (cout == 0 || k == 0) return SPARQ_OK;
    if (!w || !out || !scale_out) return set_error(SPARQ_ERR_INVALID_ARG, "w/out/scale_out pointer is NULL");
    if (cout > 2147483647LL) return set_error(SPARQ_ERR_UNSUPPORTED, "more than 2^31-1 kernels");
    if (((uintptr_t)w | (uintptr_t)scale_out) & 3u)
        return set_error(SPARQ_ERR_UNSUPPORTED, "w and scale_out must be 4-byte aligned");
    quantize_weight_kernel<<<(unsigned)cout, kThreads, 0, (cudaStream_t)stream>>>(w, k, out, scale_out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "quantize_weight_kernel launch");
    return SPARQ_OK;
}
