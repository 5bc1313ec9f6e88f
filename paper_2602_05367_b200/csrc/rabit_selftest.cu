// Self-test of the bounded-wait mechanism used by every kernel of the library: a wait that cannot
// succeed must end by itself, record that it did, and leave the context usable.
#include "rabit_internal.h"

namespace {

__global__ void bounded_wait_probe(unsigned int* status, long long limit_ns) {
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    const unsigned int bar_s = (unsigned int)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_s), "r"(1) : "memory");   // one arrival expected, none will come
    }
    __syncthreads();
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    while (true) {
        unsigned int ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(bar_s), "r"(0u) : "memory");
        if (ok) break;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        if (*(volatile int*)&abort_flag || (long long)(t - t0) > limit_ns) { abort_flag = 1; break; }
        __nanosleep(200);
    }
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(status, 1u);
}

}  // namespace

extern "C" int rabit_selftest_bounded_wait(unsigned int* status_dev, int limit_us, void* stream) {
    rabit_clear_error();
    if (!status_dev || ((uintptr_t)status_dev & 3u)) return rabit_fail(RABIT_INVALID_ARG, "rabit_selftest_bounded_wait: status_dev must be a 4-byte aligned device pointer");
    if (limit_us < 1 || limit_us > 100000) return rabit_fail(RABIT_INVALID_ARG, "rabit_selftest_bounded_wait: limit_us must be 1..100000");
    cudaStream_t st = (cudaStream_t)stream;
    RABIT_CUDA_TRY(cudaMemsetAsync(status_dev, 0, 4, st));
    bounded_wait_probe<<<1, 64, 0, st>>>(status_dev, (long long)limit_us * 1000);
    RABIT_CUDA_TRY(cudaGetLastError());
    unsigned int word = 0;
    RABIT_CUDA_TRY(cudaMemcpyAsync(&word, status_dev, 4, cudaMemcpyDeviceToHost, st));
    RABIT_CUDA_TRY(cudaStreamSynchronize(st));                 // returns: the wait ended by itself
    if (word != 1u) return rabit_fail(RABIT_DEVICE_FAULT, "rabit_selftest_bounded_wait: the kernel returned without recording the time-out");
    return RABIT_OK;
}
