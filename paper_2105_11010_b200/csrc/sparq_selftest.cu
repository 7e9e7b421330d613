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

}  // namespace sparq

using namespace sparq;

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
