// Diagnostic entry point: makes a bounded device-side wait run out on purpose, in a kernel that
// is built from the same mbar_wait / abort-flag / tensor-memory pieces as the fused kernels, so
// that the give-up path (status word, CTA-wide abort, normal kernel exit, sparq_check) can be
// exercised without a fault, a trap or an unbounded loop.
#include "sparq_gemm_kernel.cuh"

namespace sparq {

int static_status_word(unsigned int **dptr);   // sparq_static.cu

// One CTA of four warps.  Nothing ever arrives on `bar`.
//   warp 0  waits on it with the given limit: gives up, sets the status bit and the abort flag
//   warp 1  holds 32 columns of tensor memory across the wait and frees them afterwards
//   warp 2  starts waiting later with a limit a thousand times longer: must leave through the
//           abort flag, not through its own limit
//   warp 3  records how everybody left
// out[0] = 1 when warp 0's wait returned false, out[1] = 1 when warp 2's did, out[2] = cycles
// warp 2 spent waiting, out[3] = 1 once the kernel reached its end.
__global__ void __launch_bounds__(128, 1)
selftest_wait_kernel(unsigned int *status, long long limit, unsigned int *out)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_word;
    __shared__ uint32_t gave_up[2];
    __shared__ long long waited;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile uint32_t *abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_word = 0;
        gave_up[0] = gave_up[1] = 0;
        waited = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&tmem_base_slot)), "r"(32u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp == 0 && lane == 0) {
        gave_up[0] = mbar_wait(smem_u32(&bar), 0, abort_flag, status, limit) ? 0u : 1u;
    } else if (warp == 2 && lane == 0) {
        const long long t0 = clock64();
        gave_up[1] = mbar_wait(smem_u32(&bar), 0, abort_flag, status, limit * 1000) ? 0u : 1u;
        waited = clock64() - t0;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(32u) : "memory");
    }
    if (warp == 3 && lane == 0) {
        out[0] = gave_up[0];
        out[1] = gave_up[1];
        out[2] = (unsigned int)(waited > 0xFFFFFFFFLL ? 0xFFFFFFFFLL : waited);
        out[3] = 1u;
    }
}

// MMA-only loop: one CTA per SM issues `iters` x 4 tcgen05.mma kind::i8 instructions of
// 128 x BN x 32 (u8 x s8 -> s32) on operands that stay in shared memory (a 128 x 128-byte A
// tile and a BN x 128-byte B tile, 128-byte swizzle, all zeros), alternating between two
// accumulators in tensor memory every 36 instructions, and reports the cycles from the first
// issue to the retirement of the last.  No global-memory traffic, no transform, no epilogue:
// what the tensor core sustains when fed from shared memory, the ceiling of the fused kernels.
template <int BN>
__global__ void __launch_bounds__(128, 1)
mma_rate_kernel(int iters, unsigned int *status, long long limit, long long *cycles_out)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile uint32_t *abort_flag = &abort_word;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr int kBytes = (kBM + BN) * 128;
    for (int i = threadIdx.x; i < kBytes / 16; i += blockDim.x)
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" :: "r"(smem_base + (uint32_t)i * 16u), "r"(0u) : "memory");
    fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar_done), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)(2 * BN)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp == 0) {
        const uint32_t elected = elect_one();
        constexpr uint32_t idesc = make_idesc_i8(BN);
        const uint64_t adesc = make_smem_desc<128>(smem_base);
        const uint64_t bdesc = make_smem_desc<128>(smem_base + kBM * 128);
        const long long t0 = clock64();
        int in_tile = 0;
        uint32_t acc = 0;
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                tc_mma_i8_if(tmem_base + acc * (uint32_t)BN, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                             (in_tile > 0 || k > 0) ? 1u : 0u, elected);
            if (++in_tile == 9) { in_tile = 0; acc ^= 1u; }
        }
        tc_commit_if(smem_u32(&bar_done), elected);
        mbar_wait(smem_u32(&bar_done), 0, abort_flag, status, limit, true);
        if (elected) cycles_out[blockIdx.x] = clock64() - t0;
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)(2 * BN)) : "memory");
    }
}

template <int BN>
static cudaError_t launch_mma_rate(int grid, int iters, unsigned int *status, long long *cycles_out, cudaStream_t st)
{
    constexpr int smem = (kBM + BN) * 128 + 1024;
    cudaError_t e = cudaFuncSetAttribute(mma_rate_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    mma_rate_kernel<BN><<<grid, 128, smem, st>>>(iters, status, kWaitLimitCycles, cycles_out);
    return cudaGetLastError();
}

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_selftest_mma_rate(int bn, int iters, int64_t *cycles_out, void *stream)
{
    if (bn != 64 && bn != 128 && bn != 256) return set_error(SPARQ_ERR_INVALID_ARG, "bn %d is not 64, 128 or 256", bn);
    if (iters < 1 || iters > 1000000) return set_error(SPARQ_ERR_INVALID_ARG, "iters %d must lie in [1, 1e6]", iters);
    if (!cycles_out) return set_error(SPARQ_ERR_INVALID_ARG, "cycles_out is NULL");
    int dev = 0, sms = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");
    if (major != 10) return set_error(SPARQ_ERR_UNSUPPORTED, "needs an sm_100 device (found sm_%d0)", major);
    unsigned int *status = nullptr;
    int rc = get_status_word(&status);
    if (rc != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    long long *out = reinterpret_cast<long long *>(cycles_out);
    e = bn == 64 ? launch_mma_rate<64>(sms, iters, status, out, st)
      : bn == 128 ? launch_mma_rate<128>(sms, iters, status, out, st)
                  : launch_mma_rate<256>(sms, iters, status, out, st);
    if (e != cudaSuccess) return cuda_error(e, "mma_rate_kernel launch");
    return sms;
}

extern "C" int sparq_selftest_wait_timeout(int64_t limit_cycles, int use_static_word, uint32_t *report, void *stream)
{
    if (limit_cycles < 1000 || limit_cycles > 100000000)
        return set_error(SPARQ_ERR_INVALID_ARG, "limit_cycles %lld must lie in [1e3, 1e8]", (long long)limit_cycles);
    if (!report) return set_error(SPARQ_ERR_INVALID_ARG, "report is NULL");
    unsigned int *status = nullptr;
    int rc = use_static_word ? static_status_word(&status) : get_status_word(&status);
    if (rc != SPARQ_OK) return rc;
    selftest_wait_kernel<<<1, 128, 0, (cudaStream_t)stream>>>(status, (long long)limit_cycles, report);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "selftest_wait_kernel launch");
    return SPARQ_OK;
}
