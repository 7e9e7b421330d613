// sparq_gemm_s8_static: the two-kernel form of the fused GEMM for hosts that must not
// allocate device memory.  Its scratch is a fixed array in the library image.
#include <mutex>

#include "sparq_common.cuh"

namespace sparq {

int gemm_with_status(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb, int64_t M, int64_t N, int64_t K,
                     const XformArgs &x, const sparq_epilogue *e, unsigned int *status, cudaStream_t st);
int check_epilogue_args(const sparq_epilogue *e);

namespace {

constexpr size_t kHeaderBytes = 256;   // status word of the bounded waits lives here

// Transformed activations (after the header).  Zero at load; later calls see whatever the
// previous call left, which is harmless: the transform rewrites all M*K bytes that the
// GEMM reads, and the status word is cleared again whenever it is found set.
static __device__ __align__(256) unsigned char g_static_scratch[kHeaderBytes + SPARQ_STATIC_SCRATCH_BYTES];

std::mutex g_mu;
constexpr int kMaxDevices = 64;
unsigned char *g_base[kMaxDevices] = {};

// In host code the array's name is only a handle; the device address comes from the
// runtime, once per device, with that device current.
int scratch_base(unsigned char **base)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_error(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return set_error(SPARQ_ERR_UNSUPPORTED, "device ordinal %d", dev);
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_base[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_error(e, "cudaGetSymbolAddress(static scratch)");
        if (!ptr) return set_error(SPARQ_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_base[dev] = static_cast<unsigned char *>(ptr);
    }
    *base = g_base[dev];
    return SPARQ_OK;
}

}  // namespace

// Device address of the status word inside the static scratch (no allocation).
int static_status_word(unsigned int **dptr)
{
    unsigned char *base = nullptr;
    int rc = scratch_base(&base);
    if (rc != SPARQ_OK) return rc;
    *dptr = reinterpret_cast<unsigned int *>(base);
    return SPARQ_OK;
}

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_gemm_s8_static(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                                    int64_t M, int64_t N, int64_t K,
                                    const sparq_params *p, const sparq_epilogue *e, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    rc = check_epilogue_args(e);
    if (rc != SPARQ_OK) return rc;
    if (M < 0 || N < 0 || K < 0) return set_error(SPARQ_ERR_INVALID_ARG, "negative dimension");
    if (M == 0 || N == 0) return SPARQ_OK;
    if (!A || !B) return set_error(SPARQ_ERR_INVALID_ARG, "A or B is NULL");
    if (K == 0 || K % 16 || K > 65536)
        return set_error(SPARQ_ERR_UNSUPPORTED, "K = %lld must be a multiple of 16 in [16, 65536]", (long long)K);
    if (lda != K) return set_error(SPARQ_ERR_UNSUPPORTED, "sparq_gemm_s8_static needs lda == K (got lda %lld, K %lld)", (long long)lda, (long long)K);
    if (ldb < K || ldb % 16) return set_error(SPARQ_ERR_UNSUPPORTED, "ldb must be a multiple of 16 and at least K");
    if (((uintptr_t)A | (uintptr_t)B) & 15u) return set_error(SPARQ_ERR_UNSUPPORTED, "A and B must be 16-byte aligned");
    if (M > (int64_t)1 << 31 || N > (int64_t)1 << 31) return set_error(SPARQ_ERR_UNSUPPORTED, "M or N too large");
    if ((uint64_t)M * (uint64_t)K > (uint64_t)SPARQ_STATIC_SCRATCH_BYTES)
        return set_error(SPARQ_ERR_UNSUPPORTED,
                         "M * K = %llu bytes of transformed activations exceed the %u-byte static scratch of sparq_gemm_s8_static",
                         (unsigned long long)((uint64_t)M * (uint64_t)K), (unsigned)SPARQ_STATIC_SCRATCH_BYTES);

    unsigned char *base = nullptr;
    rc = scratch_base(&base);
    if (rc != SPARQ_OK) return rc;
    unsigned int *status = reinterpret_cast<unsigned int *>(base);
    uint8_t *ta = base + kHeaderBytes;
    cudaStream_t st = (cudaStream_t)stream;

    // kernel 1: T(A) -> scratch (every byte the GEMM will read is rewritten here)
    rc = sparq_quantize(A, ta, (size_t)M, (size_t)K, p, stream);
    if (rc != SPARQ_OK) return rc;
    // kernel 2: plain u8 x s8 GEMM + epilogue on the transformed activations
    XformArgs none;
    sparq_params pn = {SPARQ_MODE_NONE, 4, 0, 0};
    rc = validate_params(&pn, &none);
    if (rc != SPARQ_OK) return rc;
    rc = gemm_with_status(ta, K, B, ldb, M, N, K, none, e, status, st);
    if (rc != SPARQ_OK) return rc;

    cudaError_t ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) return cuda_error(ce, "cudaStreamSynchronize");
    unsigned int word = 0;
    ce = cudaMemcpy(&word, status, sizeof(word), cudaMemcpyDeviceToHost);
    if (ce != cudaSuccess) return cuda_error(ce, "cudaMemcpy(static status word)");
    if (word) {
        cudaMemset(status, 0, sizeof(word));   // must be zero again before the next call
        return set_error(SPARQ_ERR_TIMEOUT, "a bounded device-side wait expired in sparq_gemm_s8_static (status 0x%x); its outputs are undefined", word);
    }
    return SPARQ_OK;
}
