// Test-only build (not part of liblte.so): makes a bounded mbarrier wait of the library's own wait routine run out, the
// way a lost TMA copy or a lost tensor-core commit would, without any fault: the barrier is simply never armed, the
// wait gives up after a few thousand polls, records its code and the kernel returns normally.
#include "tc_common.cuh"

using namespace lte;
using namespace lte::tc;

__device__ StatusWord g_probe_status = LTE_STATUS_INIT;

// arm = 0: nothing ever arrives on the barrier.  out[0], out[1]: cycles spent in the first and the second wait;
// out[2] = 1 once the kernel has run to its end.
__global__ void wait_probe_kernel(int arm, long long* out)
{
    __shared__ __align__(8) unsigned long long bar_mem;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (arm) mbar_arrive(bar);
        const long long t0 = clock64();
        mbar_wait_s<4096>(bar, 0, 77, &g_probe_status);           // gives up after 4096 polls when nothing arrives
        const long long t1 = clock64();
        // a second wait of the same launch: after the first one gave up it must stop early (at its first look at the
        // launch's abort mark, 1024 polls in) instead of running out its own, much longer, limit
        if (!arm) mbar_wait_s<(1u << 16)>(bar, 0, 78, &g_probe_status);
        const long long t2 = clock64();
        out[0] = t1 - t0; out[1] = t2 - t1; out[2] = 1;
    }
}

extern "C" int wait_probe_run(int arm, long long* host_out)
{
    long long* d = nullptr;
    if (cudaMalloc(&d, 3 * sizeof(long long)) != cudaSuccess) return -1;
    cudaMemset(d, 0, 3 * sizeof(long long));
    wait_probe_kernel<<<1, 32>>>(arm, d);
    const cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) cudaMemcpy(host_out, d, 3 * sizeof(long long), cudaMemcpyDeviceToHost);
    cudaFree(d);
    return e == cudaSuccess ? 0 : -(int)e;
}

// the code the probe's status word holds; reading clears it (same routine as lte_device_status uses per family)
extern "C" int wait_probe_status(void) { return status_fetch_and_clear(g_probe_status); }
