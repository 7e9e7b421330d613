// Host-buffer forms of the entry points: stage the input on the device, run the device
// entry point, copy the outputs back, synchronize.
#include <mutex>

#include "sparq_common.cuh"

namespace sparq {

namespace {

constexpr int kMaxDevices = 64;
constexpr int kSlots = 5;   // 0: input, 1: acc, 2: f32, 3: u8, 4: residual input

struct Staging {
    void *ptr[kSlots] = {};
    size_t cap[kSlots] = {};
};

std::mutex g_mu;
Staging g_staging[kMaxDevices];

// Device buffer of at least `bytes` for slot `slot` on the current device.
int staging(int slot, size_t bytes, void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_error(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return set_error(SPARQ_ERR_UNSUPPORTED, "device ordinal %d", dev);
    std::lock_guard<std::mutex> lk(g_mu);
    Staging &s = g_staging[dev];
    if (s.cap[slot] < bytes) {
        if (s.ptr[slot]) cudaFree(s.ptr[slot]);
        s.ptr[slot] = nullptr;
        s.cap[slot] = 0;
        size_t want = (bytes + 255) & ~(size_t)255;
        e = cudaMalloc(&s.ptr[slot], want);
        if (e != cudaSuccess) return cuda_error(e, "cudaMalloc(staging buffer)");
        s.cap[slot] = want;
    }
    *out = s.ptr[slot];
    return SPARQ_OK;
}

int copy(void *dst, const void *src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st)
{
    cudaError_t e = cudaMemcpyAsync(dst, src, bytes, kind, st);
    if (e != cudaSuccess) return cuda_error(e, "cudaMemcpyAsync");
    return SPARQ_OK;
}

// Replaces the HOST output pointers of `e` by device staging buffers; remembers the pairs.
struct OutPlan {
    void *host[3] = {};
    void *dev[3] = {};
    size_t bytes[3] = {};
};

int plan_outputs(const sparq_epilogue *e, size_t elems, sparq_epilogue *dev_e, OutPlan *plan)
{
    *dev_e = *e;
    void *hosts[3] = {e->acc_out, e->f32_out, e->u8_out};
    size_t width[3] = {4, 4, 1};
    for (int i = 0; i < 3; ++i) {
        if (!hosts[i]) continue;
        void *d = nullptr;
        int rc = staging(1 + i, elems * width[i], &d);
        if (rc != SPARQ_OK) return rc;
        plan->host[i] = hosts[i];
        plan->dev[i] = d;
        plan->bytes[i] = elems * width[i];
    }
    dev_e->acc_out = (int32_t *)plan->dev[0];
    dev_e->f32_out = (float *)plan->dev[1];
    dev_e->u8_out = (uint8_t *)plan->dev[2];
    return SPARQ_OK;
}

// Stages the HOST residual tensor of `e` (if any) on the device and points dev_e at the copy.
int stage_residual(const sparq_epilogue *e, size_t elems, sparq_epilogue *dev_e, cudaStream_t st)
{
    if (!e->residual) return SPARQ_OK;
    void *d = nullptr;
    int rc = staging(4, elems, &d);
    if (rc != SPARQ_OK) return rc;
    if ((rc = copy(d, e->residual, elems, cudaMemcpyHostToDevice, st)) != SPARQ_OK) return rc;
    dev_e->residual = (const uint8_t *)d;
    return SPARQ_OK;
}

int copy_back_and_sync(const OutPlan &plan, cudaStream_t st)
{
    for (int i = 0; i < 3; ++i) {
        if (!plan.host[i]) continue;
        int rc = copy(plan.host[i], plan.dev[i], plan.bytes[i], cudaMemcpyDeviceToHost, st);
        if (rc != SPARQ_OK) return rc;
    }
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_error(e, "cudaStreamSynchronize");
    return SPARQ_OK;
}

}  // namespace

void release_host_staging()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    if (dev < 0 || dev >= kMaxDevices) return;
    std::lock_guard<std::mutex> lk(g_mu);
    for (int i = 0; i < kSlots; ++i) {
        if (g_staging[dev].ptr[i]) cudaFree(g_staging[dev].ptr[i]);
        g_staging[dev].ptr[i] = nullptr;
        g_staging[dev].cap[i] = 0;
    }
}

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_quantize_host(const uint8_t *in_host, uint8_t *out_host, size_t rows, size_t row_len,
                                   const sparq_params *p, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if (rows == 0 || row_len == 0) return SPARQ_OK;
    if (!in_host || !out_host) return set_error(SPARQ_ERR_INVALID_ARG, "in/out pointer is NULL");
    if (rows > ((size_t)1 << 62) / row_len) return set_error(SPARQ_ERR_INVALID_ARG, "rows * row_len overflows");
    const size_t bytes = rows * row_len;
    cudaStream_t st = (cudaStream_t)stream;
    void *d_in = nullptr, *d_out = nullptr;
    if ((rc = staging(0, bytes, &d_in)) != SPARQ_OK) return rc;
    if ((rc = staging(3, bytes, &d_out)) != SPARQ_OK) return rc;
    if ((rc = copy(d_in, in_host, bytes, cudaMemcpyHostToDevice, st)) != SPARQ_OK) return rc;
    if ((rc = sparq_quantize((const uint8_t *)d_in, (uint8_t *)d_out, rows, row_len, p, stream)) != SPARQ_OK) return rc;
    if ((rc = copy(out_host, d_out, bytes, cudaMemcpyDeviceToHost, st)) != SPARQ_OK) return rc;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_error(e, "cudaStreamSynchronize");
    return SPARQ_OK;
}

extern "C" int sparq_gemm_s8_host(const uint8_t *A_host, int64_t lda, const int8_t *B, int64_t ldb,
                                  int64_t M, int64_t N, int64_t K,
                                  const sparq_params *p, const sparq_epilogue *e, void *stream)
{
    if (!e) return set_error(SPARQ_ERR_INVALID_ARG, "sparq_epilogue is NULL");
    if (M < 0 || N < 0 || K < 0 || lda < K) return set_error(SPARQ_ERR_INVALID_ARG, "bad dimension");
    if (M == 0 || N == 0) return SPARQ_OK;
    if (!A_host) return set_error(SPARQ_ERR_INVALID_ARG, "A_host is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    void *d_a = nullptr;
    int rc = staging(0, (size_t)M * (size_t)lda, &d_a);
    if (rc != SPARQ_OK) return rc;
    sparq_epilogue de;
    OutPlan plan;
    if ((rc = plan_outputs(e, (size_t)M * (size_t)N, &de, &plan)) != SPARQ_OK) return rc;
    if ((rc = stage_residual(e, (size_t)M * (size_t)N, &de, st)) != SPARQ_OK) return rc;
    if ((rc = copy(d_a, A_host, (size_t)M * (size_t)lda, cudaMemcpyHostToDevice, st)) != SPARQ_OK) return rc;
    if ((rc = sparq_gemm_s8((const uint8_t *)d_a, lda, B, ldb, M, N, K, p, &de, stream)) != SPARQ_OK) return rc;
    return copy_back_and_sync(plan, st);
}

extern "C" int sparq_conv2d_nhwc_s8_host(const uint8_t *x_host, int n, int h, int w, int c,
                                         const int8_t *wgt, int cout, int r, int s,
                                         int stride_h, int stride_w, int pad_h, int pad_w,
                                         const sparq_params *p, const sparq_epilogue *e, void *stream)
{
    if (!e) return set_error(SPARQ_ERR_INVALID_ARG, "sparq_epilogue is NULL");
    if (n < 0 || h < 0 || w < 0 || c < 0 || cout < 0 || r < 1 || s < 1 || stride_h < 1 || stride_w < 1 ||
        pad_h < 0 || pad_w < 0 || h + 2 * pad_h < r || w + 2 * pad_w < s)
        return set_error(SPARQ_ERR_INVALID_ARG, "bad convolution geometry");
    if (n == 0 || cout == 0) return SPARQ_OK;
    if (!x_host) return set_error(SPARQ_ERR_INVALID_ARG, "x_host is NULL");
    const int ho = (h + 2 * pad_h - r) / stride_h + 1;
    const int wo = (w + 2 * pad_w - s) / stride_w + 1;
    const size_t in_bytes = (size_t)n * h * w * c;
    const size_t out_elems = (size_t)n * ho * wo * cout;
    cudaStream_t st = (cudaStream_t)stream;
    void *d_x = nullptr;
    int rc = staging(0, in_bytes, &d_x);
    if (rc != SPARQ_OK) return rc;
    sparq_epilogue de;
    OutPlan plan;
    if ((rc = plan_outputs(e, out_elems, &de, &plan)) != SPARQ_OK) return rc;
    if ((rc = stage_residual(e, out_elems, &de, st)) != SPARQ_OK) return rc;
    if ((rc = copy(d_x, x_host, in_bytes, cudaMemcpyHostToDevice, st)) != SPARQ_OK) return rc;
    rc = sparq_conv2d_nhwc_s8((const uint8_t *)d_x, n, h, w, c, wgt, cout, r, s, stride_h, stride_w, pad_h, pad_w,
                              p, &de, stream);
    if (rc != SPARQ_OK) return rc;
    return copy_back_and_sync(plan, st);
}
