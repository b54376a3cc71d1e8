// The time-out path of the bounded waits, exercised on purpose: a kernel whose
// barrier can never complete, a short poll limit, and the report every other
// kernel of the library would make in that situation. Nothing faults, traps or
// waits without a limit; the context stays usable.
#include "kernels.cuh"

namespace placeto {

namespace {

__global__ void wait_timeout_probe_kernel(const StatusSlot status, const float *src) {
    __shared__ __align__(16) float landing[4];
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_expect(&bar, 32);                 // 32 bytes announced ...
        bulk_load(landing, src, 16, &bar);     // ... 16 ever sent: the phase cannot complete
    }
    __syncthreads();
    bool done = false;
    for (int i = 0; i < 4096 && !done; ++i) {  // far longer than a 16-byte copy takes
        unsigned ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(smem_addr(&bar)), "r"(0)
            : "memory");
        done = ok != 0;
    }
    if (!done && threadIdx.x == 0) report_status(status, PLACETO_ERR_TIMEOUT);
}

}  // namespace

cudaError_t launch_wait_timeout_probe(const StatusSlot &status, cudaStream_t stream) {
    // the 16 bytes behind the record serve as the copy's source
    const float *src = reinterpret_cast<const float *>(status.record + 1);
    wait_timeout_probe_kernel<<<1, 32, 0, stream>>>(status, src);
    count_launch();
    return cudaGetLastError();
}

}  // namespace placeto
