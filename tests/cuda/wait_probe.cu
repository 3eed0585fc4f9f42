// Test-only kernel (built by tests/test_gpu_timeout.py, never linked into libcdl.so): runs the library's bounded
// mbarrier wait on a barrier that receives `arrivals` of the `expected` arrivals.  With one arrival missing the wait
// gives up after limit_ns, the kernel writes the library's timeout record into `status` and returns normally.
#include "cdl_wait.cuh"

__global__ void wait_probe_kernel(int *status, unsigned long long limit_ns, int arrivals, int expected, int *outcome)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_s;
    const uint32_t b = cdl::smem_u32(&bar);
    if (threadIdx.x == 0) {
        abort_s = 0;
        cdl::mbar_init(b, (uint32_t)expected);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if ((int)threadIdx.x < arrivals) cdl::mbar_arrive(b);
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool done = cdl::mbar_wait(b, 0u, &abort_s, limit_ns);
        if (!done) cdl::record_timeout(status);
        *outcome = done ? 1 : 2;
    }
}

extern "C" int wait_probe(void *status, unsigned long long limit_ns, int arrivals, int expected, void *outcome, void *stream)
{
    if (arrivals < 0 || expected < 1 || arrivals > expected || expected > 64) return -1;
    wait_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int *>(status), limit_ns, arrivals,
                                                                       expected, static_cast<int *>(outcome));
    return cudaGetLastError() == cudaSuccess ? 0 : -6;
}
