// Host-side plumbing of the SPARQ library: error text, parameter validation, the
// per-device status word, sparq_check / sparq_shutdown.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "sparq_common.cuh"

namespace sparq {

static thread_local char g_err[512] = "";

int set_error(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int cuda_error(cudaError_t e, const char *what)
{
    return set_error(SPARQ_ERR_CUDA, "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
}

int validate_params(const sparq_params *p, XformArgs *x)
{
    if (!p) return set_error(SPARQ_ERR_INVALID_ARG, "sparq_params is NULL");
    memset(x, 0, sizeof(*x));
    x->mode = p->mode;
    if (p->mode == SPARQ_MODE_NONE) {
        x->n = 4;
        return SPARQ_OK;
    }
    if (p->mode != SPARQ_MODE_BSPARQ && p->mode != SPARQ_MODE_VSPARQ)
        return set_error(SPARQ_ERR_INVALID_ARG, "mode %d is not NONE(0), BSPARQ(1) or VSPARQ(2)", p->mode);
    int n = p->window_bits;
    if (n < 2 || n > 4)
        return set_error(SPARQ_ERR_INVALID_ARG, "window_bits %d is not 2, 3 or 4", n);
    if (p->rounding != SPARQ_ROUND_TRUNCATE && p->rounding != SPARQ_ROUND_NEAREST)
        return set_error(SPARQ_ERR_INVALID_ARG, "rounding %d is not TRUNCATE(0) or NEAREST(1)", p->rounding);
    const int top = 8 - n;
    const uint32_t mask = p->placement_mask;
    if (mask >> (top + 1))
        return set_error(SPARQ_ERR_INVALID_ARG, "placement_mask 0x%x has a shift above %d for %d-bit windows", mask, top, n);
    if (!(mask & 1u) || !((mask >> top) & 1u))
        return set_error(SPARQ_ERR_INVALID_ARG, "placement_mask 0x%x must contain shift 0 and shift %d", mask, top);
    int run = 0, longest = 0;
    uint32_t disallowed = 0;
    for (int d = 1; d < top; ++d) {
        if ((mask >> d) & 1u) {
            run = 0;
        } else {
            disallowed |= 1u << d;
            if (++run > longest) longest = run;
        }
    }
    if (longest >= n)
        return set_error(SPARQ_ERR_INVALID_ARG, "placement_mask 0x%x leaves a gap wider than the %d-bit window", mask, n);
    x->n = n;
    x->rnd = p->rounding;
    x->mask = mask;
    x->widen_rounds = longest;
    x->widen_c = disallowed * 0x01010101u;
    return SPARQ_OK;
}

// ---- per-device status word ------------------------------------------------------------

static std::mutex g_mu;
static constexpr int kMaxDevices = 64;
static unsigned int *g_status[kMaxDevices] = {};

int get_status_word(unsigned int **dptr)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_error(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return set_error(SPARQ_ERR_UNSUPPORTED, "device ordinal %d", dev);
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_status[dev]) {
        unsigned int *p = nullptr;
        e = cudaMalloc(&p, sizeof(unsigned int));
        if (e != cudaSuccess) return cuda_error(e, "cudaMalloc(status word)");
        e = cudaMemset(p, 0, sizeof(unsigned int));
        if (e != cudaSuccess) {
            cudaFree(p);
            return cuda_error(e, "cudaMemset(status word)");
        }
        g_status[dev] = p;
    }
    *dptr = g_status[dev];
    return SPARQ_OK;
}

void release_gemm_state();     // sparq_gemm.cu
void release_host_staging();   // sparq_host.cu

}  // namespace sparq

using namespace sparq;

extern "C" const char *sparq_last_error(void) { return g_err; }

extern "C" int sparq_check(void *stream)
{
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_error(e, "cudaStreamSynchronize");
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_error(e, "cudaGetDevice");
    unsigned int *p = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (dev >= 0 && dev < kMaxDevices) p = g_status[dev];
    }
    if (!p) return SPARQ_OK;  // no kernel that can time out has run on this device
    unsigned int word = 0;
    e = cudaMemcpy(&word, p, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_error(e, "cudaMemcpy(status word)");
    if (word) {
        cudaMemset(p, 0, sizeof(word));
        if (word == 0x100u)
            return set_error(SPARQ_ERR_INVALID_ARG, "2:4 weight coordinates were not strictly increasing in 0..3; those groups were expanded as zeros");
        return set_error(SPARQ_ERR_TIMEOUT, "a bounded device-side wait expired (status 0x%x); outputs of the affected launch are undefined", word);
    }
    return SPARQ_OK;
}

extern "C" int sparq_shutdown(void)
{
    release_gemm_state();
    release_host_staging();
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SPARQ_OK;  // no device: nothing is held
    }
    std::lock_guard<std::mutex> lk(g_mu);
    if (dev >= 0 && dev < kMaxDevices && g_status[dev]) {
        cudaFree(g_status[dev]);
        g_status[dev] = nullptr;
    }
    return SPARQ_OK;
}
