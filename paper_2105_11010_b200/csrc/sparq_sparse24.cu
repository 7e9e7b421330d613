// SPARQ on top of a 2:4 sparse tensor core (Sections 4 and 5.3 of the paper): the weights'
// coordinates pick two of every four activations, and vSPARQ's pair is THAT pair, so the
// transform depends on the output channel and cannot be applied to the activations once.
//
// What it can be applied to once is every pair a coordinate pattern could select: a group
// of four activations has six such pairs, (0,1) (0,2) (0,3) (1,2) (1,3) (2,3).  The
// activation side is therefore expanded to 12 bytes per group -- T2 of each of the six
// pairs, in that order -- and a weight row puts its two values into the two columns of its
// own pattern and zeros into the other ten.  The product of the expanded operands is
// exactly the sparse product with per-channel pairs, and it is a plain dense u8 x s8
// contraction (K' = 3K) that the existing GEMM / convolution kernels run with mode NONE.
// Without the pair rule (modes NONE and BSPARQ) the transform is per element, commutes
// with the selection, and the expansion is just the dense form of the weights (K' = K).
#include "sparq_common.cuh"

namespace sparq {

int check_epilogue_args(const sparq_epilogue *e);

namespace {

constexpr int kThreads = 256;
constexpr unsigned kBadCoordinates = 0x100u;   // status word bit: a group's coordinates were not increasing in 0..3

__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream16(void *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// One group of four activations (bytes of x) -> the six transformed pairs, 12 bytes.
template <int N, bool RND, bool WIDEN>
__device__ __forceinline__ void expand_group(uint32_t x, const XformDev &d, uint32_t &o0, uint32_t &o1, uint32_t &o2)
{
    o0 = xform_word<SPARQ_MODE_VSPARQ, N, RND, WIDEN>(prmt(x, x, 0x2010u), d);   // (0,1) (0,2)
    o1 = xform_word<SPARQ_MODE_VSPARQ, N, RND, WIDEN>(prmt(x, x, 0x2130u), d);   // (0,3) (1,2)
    o2 = xform_word<SPARQ_MODE_VSPARQ, N, RND, WIDEN>(prmt(x, x, 0x3231u), d);   // (1,3) (2,3)
}

// in: vectors of 16 activations (4 groups); out: 48 bytes per vector
template <int N, bool RND, bool WIDEN>
__global__ void __launch_bounds__(kThreads)
expand_act_kernel(const uint4 *__restrict__ in, uint4 *__restrict__ out, size_t nvec, XformDev d)
{
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < nvec; i += (size_t)gridDim.x * kThreads) {
        const uint4 v = ld_stream16(in + i);
        uint32_t g0[3], g1[3], g2[3], g3[3];
        expand_group<N, RND, WIDEN>(v.x, d, g0[0], g0[1], g0[2]);
        expand_group<N, RND, WIDEN>(v.y, d, g1[0], g1[1], g1[2]);
        expand_group<N, RND, WIDEN>(v.z, d, g2[0], g2[1], g2[2]);
        expand_group<N, RND, WIDEN>(v.w, d, g3[0], g3[1], g3[2]);
        st_stream16(out + 3 * i, make_uint4(g0[0], g0[1], g0[2], g1[0]));
        st_stream16(out + 3 * i + 1, make_uint4(g1[1], g1[2], g2[0], g2[1]));
        st_stream16(out + 3 * i + 2, make_uint4(g2[2], g3[0], g3[1], g3[2]));
    }
}

// One thread per (row, group): two values and their coordinates -> 4 (dense) or 12 bytes.
template <bool PAIRS>
__global__ void __launch_bounds__(kThreads)
expand_weight_kernel(const int8_t *__restrict__ vals, const uint8_t *__restrict__ pos, size_t groups,
                     int8_t *__restrict__ out, unsigned int *status)
{
    for (size_t g = (size_t)blockIdx.x * kThreads + threadIdx.x; g < groups; g += (size_t)gridDim.x * kThreads) {
        const uint32_t v0 = (uint8_t)vals[2 * g], v1 = (uint8_t)vals[2 * g + 1];
        const uint32_t p0 = pos[2 * g], p1 = pos[2 * g + 1];
        const bool ok = p0 < p1 && p1 <= 3u;
        if (!ok) atomicOr(status, kBadCoordinates);
        if (PAIRS) {
            // column pair of the pattern: (0,1) (0,2) (0,3) (1,2) (1,3) (2,3) -> 0..5
            const uint32_t c = p0 == 0u ? p1 - 1u : (p0 == 1u ? p1 + 1u : 5u);
            uint32_t w[3] = {0u, 0u, 0u};
            if (ok) w[c >> 1] = (v0 | (v1 << 8)) << (16u * (c & 1u));
            uint32_t *o = reinterpret_cast<uint32_t *>(out + 12 * g);
            o[0] = w[0]; o[1] = w[1]; o[2] = w[2];
        } else {
            uint32_t w = 0u;
            if (ok) w = (v0 << (8u * p0)) | (v1 << (8u * p1));
            reinterpret_cast<uint32_t *>(out)[g] = w;
        }
    }
}

int grid_for(size_t items, int per_sm, int *blocks)
{
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");
    size_t want = (items + kThreads - 1) / kThreads;
    if (want < 1) want = 1;
    const size_t cap = (size_t)sms * per_sm;
    *blocks = (int)(want < cap ? want : cap);
    return SPARQ_OK;
}

template <int N>
cudaError_t launch_expand_act(const uint4 *in, uint4 *out, size_t nvec, const XformArgs &a, int blocks, cudaStream_t st)
{
    const XformDev d{a.widen_c, a.widen_rounds, a.n};
    const bool widen = a.widen_rounds > 0 || N == 0;
    if (a.rnd && widen) expand_act_kernel<N, true, true><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    else if (a.rnd) expand_act_kernel<N, true, false><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    else if (widen) expand_act_kernel<N, false, true><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    else expand_act_kernel<N, false, false><<<blocks, kThreads, 0, st>>>(in, out, nvec, d);
    return cudaGetLastError();
}

}  // namespace

}  // namespace sparq

using namespace sparq;

extern "C" int64_t sparq_sparse24_expanded_k(int64_t K, const sparq_params *p)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if (K < 0 || K % 4) return set_error(SPARQ_ERR_INVALID_ARG, "K (%lld) must be a non-negative multiple of 4", (long long)K);
    return x.mode == SPARQ_MODE_VSPARQ ? 3 * K : K;
}

extern "C" int sparq_sparse24_expand_weights(const int8_t *vals, const uint8_t *pos, int64_t N, int64_t K,
                                             const sparq_params *p, int8_t *w_exp, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if (N < 0 || K < 0 || K % 4) return set_error(SPARQ_ERR_INVALID_ARG, "N >= 0 and K a non-negative multiple of 4 are required");
    if (N == 0 || K == 0) return SPARQ_OK;
    if (!vals || !pos || !w_exp) return set_error(SPARQ_ERR_INVALID_ARG, "vals/pos/w_exp pointer is NULL");
    if ((uintptr_t)w_exp & 3u) return set_error(SPARQ_ERR_UNSUPPORTED, "w_exp must be 4-byte aligned");
    unsigned int *status = nullptr;
    if ((rc = get_status_word(&status)) != SPARQ_OK) return rc;
    const size_t groups = (size_t)N * (size_t)(K / 4);
    int blocks = 0;
    if ((rc = grid_for(groups, 16, &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (x.mode == SPARQ_MODE_VSPARQ) expand_weight_kernel<true><<<blocks, kThreads, 0, st>>>(vals, pos, groups, w_exp, status);
    else expand_weight_kernel<false><<<blocks, kThreads, 0, st>>>(vals, pos, groups, w_exp, status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "expand_weight_kernel launch");
    return SPARQ_OK;
}

extern "C" int sparq_sparse24_expand_activations(const uint8_t *A, size_t rows, size_t K, const sparq_params *p,
                                                 uint8_t *a_exp, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if (rows == 0 || K == 0) return SPARQ_OK;
    if (!A || !a_exp) return set_error(SPARQ_ERR_INVALID_ARG, "A/a_exp pointer is NULL");
    if (K % 16) return set_error(SPARQ_ERR_UNSUPPORTED, "K (%zu) must be a multiple of 16", K);
    if (rows > ((size_t)1 << 60) / K) return set_error(SPARQ_ERR_INVALID_ARG, "rows * K overflows");
    if (x.mode != SPARQ_MODE_VSPARQ)   // per-element transform: the expanded tensor is T(A) itself
        return sparq_quantize(A, a_exp, rows, K, p, stream);
    if (((uintptr_t)A | (uintptr_t)a_exp) & 15u) return set_error(SPARQ_ERR_UNSUPPORTED, "A and a_exp must be 16-byte aligned");
    const size_t nvec = rows * K / 16;
    int blocks = 0;
    if ((rc = grid_for(nvec, 32, &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const uint4 *in = reinterpret_cast<const uint4 *>(A);
    uint4 *out = reinterpret_cast<uint4 *>(a_exp);
    cudaError_t e = (x.n == 4 && x.widen_rounds == 0) ? launch_expand_act<4>(in, out, nvec, x, blocks, st)
                                                       : launch_expand_act<0>(in, out, nvec, x, blocks, st);
    if (e != cudaSuccess) return cuda_error(e, "expand_act_kernel launch");
    return SPARQ_OK;
}

extern "C" int sparq_gemm_s8_sparse24(const uint8_t *A, const int8_t *w_exp, int64_t M, int64_t N, int64_t K,
                                      const sparq_params *p, const sparq_epilogue *e, uint8_t *workspace, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if ((rc = check_epilogue_args(e)) != SPARQ_OK) return rc;
    if (M < 0 || N < 0 || K < 0) return set_error(SPARQ_ERR_INVALID_ARG, "negative dimension");
    if (M == 0 || N == 0) return SPARQ_OK;
    if (x.mode != SPARQ_MODE_VSPARQ)   // dense form of the weights, transform fused as usual
        return sparq_gemm_s8(A, K, w_exp, K, M, N, K, p, e, stream);
    if (!workspace) return set_error(SPARQ_ERR_INVALID_ARG, "workspace is NULL (M * 3K bytes are needed with vSPARQ)");
    if ((rc = sparq_sparse24_expand_activations(A, (size_t)M, (size_t)K, p, workspace, stream)) != SPARQ_OK) return rc;
    const sparq_params none = {SPARQ_MODE_NONE, 4, 0x1Fu, 0};
    return sparq_gemm_s8(workspace, 3 * K, w_exp, 3 * K, M, N, 3 * K, &none, e, stream);
}
