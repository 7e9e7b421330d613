// Host-buffer forms of the entry points: stage the input on the device, run the device
// entry point, copy the outputs back, synchronize.  Large problems are cut into a few chunks
// of independent rows (images) so that the copy in of chunk i+1, the kernel of chunk i and the
// copy out of chunk i-1 overlap: the two copy directions and the kernels run on three streams.
#include <functional>
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

constexpr int kMaxChunks = 4;
constexpr size_t kChunkMinBytes = (size_t)1 << 20;     // below this one chunk: the overlap would not pay for the extra launches

// Per device: a stream per copy direction and the events that order them with the caller's stream.
struct Pipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr, in_done[kMaxChunks] = {}, run_done[kMaxChunks] = {}, out_done = nullptr;
};

std::mutex g_mu;
Staging g_staging[kMaxDevices];
Pipe g_pipe[kMaxDevices];

int get_pipe(Pipe **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_error(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return set_error(SPARQ_ERR_UNSUPPORTED, "device ordinal %d", dev);
    std::lock_guard<std::mutex> lk(g_mu);
    Pipe &p = g_pipe[dev];
    if (!p.ready) {
        e = cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.out_done, cudaEventDisableTiming);
        for (int i = 0; i < kMaxChunks && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&p.in_done[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.run_done[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) return cuda_error(e, "stream / event creation for the host-buffer pipeline");
        p.ready = true;
    }
    *out = &p;
    return SPARQ_OK;
}

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

// What one unit (a GEMM row, an image) occupies in each buffer, and how to launch a range of units.
struct ChunkJob {
    size_t units = 0;            // independent rows / images
    size_t unit_align = 1;       // chunk sizes are multiples of this
    size_t in_unit = 0;          // input bytes per unit
    size_t out_unit = 0;         // output elements per unit
    const uint8_t *in_host = nullptr;
    uint8_t *in_dev = nullptr;
    const uint8_t *res_host = nullptr;   // residual input (u8, out_unit bytes per unit) or null
    uint8_t *res_dev = nullptr;
    OutPlan plan;                // whole-problem host / device output pairs
    // launches units [u0, u0 + count) given the device epilogue pointers advanced to u0
    std::function<int(size_t u0, size_t count)> launch;
};

int run_chunked(const ChunkJob &job, cudaStream_t st)
{
    const size_t width[3] = {4, 4, 1};
    size_t total = job.units * job.in_unit;
    for (int i = 0; i < 3; ++i) if (job.plan.host[i]) total += job.units * job.out_unit * width[i];
    int chunks = 1;
    if (total >= 2 * kChunkMinBytes) {
        chunks = (int)(total / kChunkMinBytes);
        if (chunks > kMaxChunks) chunks = kMaxChunks;
    }
    size_t per = (job.units + chunks - 1) / chunks;
    per = (per + job.unit_align - 1) / job.unit_align * job.unit_align;
    Pipe *pp = nullptr;
    int rc = get_pipe(&pp);
    if (rc != SPARQ_OK) return rc;
    Pipe &p = *pp;
    cudaError_t e = cudaEventRecord(p.start, st);               // everything below comes after the caller's earlier work
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p.s_in, p.start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p.s_out, p.start, 0);
    if (e != cudaSuccess) return cuda_error(e, "host-buffer pipeline set-up");
    int ci = 0;
    for (size_t u0 = 0; u0 < job.units; u0 += per, ++ci) {
        const size_t cnt = (job.units - u0 < per) ? job.units - u0 : per;
        if ((rc = copy(job.in_dev + u0 * job.in_unit, job.in_host + u0 * job.in_unit, cnt * job.in_unit,
                       cudaMemcpyHostToDevice, p.s_in)) != SPARQ_OK) return rc;
        if (job.res_host && (rc = copy(job.res_dev + u0 * job.out_unit, job.res_host + u0 * job.out_unit, cnt * job.out_unit,
                                       cudaMemcpyHostToDevice, p.s_in)) != SPARQ_OK) return rc;
        e = cudaEventRecord(p.in_done[ci], p.s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, p.in_done[ci], 0);
        if (e != cudaSuccess) return cuda_error(e, "host-buffer pipeline (copy in)");
        if ((rc = job.launch(u0, cnt)) != SPARQ_OK) return rc;
        e = cudaEventRecord(p.run_done[ci], st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(p.s_out, p.run_done[ci], 0);
        if (e != cudaSuccess) return cuda_error(e, "host-buffer pipeline (kernel)");
        for (int i = 0; i < 3; ++i) {
            if (!job.plan.host[i]) continue;
            const size_t off = u0 * job.out_unit * width[i];
            if ((rc = copy((uint8_t *)job.plan.host[i] + off, (const uint8_t *)job.plan.dev[i] + off,
                           cnt * job.out_unit * width[i], cudaMemcpyDeviceToHost, p.s_out)) != SPARQ_OK) return rc;
        }
    }
    e = cudaEventRecord(p.out_done, p.s_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, p.out_done, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_error(e, "host-buffer pipeline (copy out)");
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
    Pipe &p = g_pipe[dev];
    if (p.ready) {
        cudaStreamDestroy(p.s_in);
        cudaStreamDestroy(p.s_out);
        cudaEventDestroy(p.start);
        cudaEventDestroy(p.out_done);
        for (int i = 0; i < kMaxChunks; ++i) { cudaEventDestroy(p.in_done[i]); cudaEventDestroy(p.run_done[i]); }
        p = Pipe();
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
    void *d_res = nullptr;
    if (e->residual && (rc = staging(4, (size_t)M * (size_t)N, &d_res)) != SPARQ_OK) return rc;
    ChunkJob job;
    job.units = (size_t)M; job.unit_align = 128;
    job.in_unit = (size_t)lda; job.out_unit = (size_t)N;
    job.in_host = A_host; job.in_dev = (uint8_t *)d_a;
    job.res_host = e->residual; job.res_dev = (uint8_t *)d_res;
    job.plan = plan;
    job.launch = [&](size_t u0, size_t cnt) {
        sparq_epilogue ce = de;
        if (ce.acc_out) ce.acc_out += u0 * (size_t)N;
        if (ce.f32_out) ce.f32_out += u0 * (size_t)N;
        if (ce.u8_out) ce.u8_out += u0 * (size_t)N;
        if (e->residual) ce.residual = (const uint8_t *)d_res + u0 * (size_t)N;
        return sparq_gemm_s8((const uint8_t *)d_a + u0 * (size_t)lda, lda, B, ldb, (int64_t)cnt, N, K, p, &ce, stream);
    };
    return run_chunked(job, st);
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
    void *d_res = nullptr;
    if (e->residual && (rc = staging(4, out_elems, &d_res)) != SPARQ_OK) return rc;
    const size_t out_img = (size_t)ho * wo * cout;
    ChunkJob job;
    job.units = (size_t)n; job.unit_align = 1;
    job.in_unit = (size_t)h * w * c; job.out_unit = out_img;
    job.in_host = x_host; job.in_dev = (uint8_t *)d_x;
    job.res_host = e->residual; job.res_dev = (uint8_t *)d_res;
    job.plan = plan;
    job.launch = [&](size_t u0, size_t cnt) {
        sparq_epilogue ce = de;
        if (ce.acc_out) ce.acc_out += u0 * out_img;
        if (ce.f32_out) ce.f32_out += u0 * out_img;
        if (ce.u8_out) ce.u8_out += u0 * out_img;
        if (e->residual) ce.residual = (const uint8_t *)d_res + u0 * out_img;
        return sparq_conv2d_nhwc_s8((const uint8_t *)d_x + u0 * (size_t)h * w * c, (int)cnt, h, w, c, wgt, cout, r, s,
                                    stride_h, stride_w, pad_h, pad_w, p, &ce, stream);
    };
    return run_chunked(job, st);
}
