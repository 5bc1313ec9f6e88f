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

// Read-only streaming probe: every thread keeps eight 128-bit streaming loads in flight and folds what it reads into
// one word, which is stored only if it has a value no data here produces (so the loads cannot be dropped).
__global__ void __launch_bounds__(512) stream_read_probe(const uint4* __restrict__ src, size_t n_vec, unsigned int* sink) {
    const size_t stride = (size_t)gridDim.x * 512 * 8;
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
    for (size_t base = (size_t)blockIdx.x * 512 * 8 + threadIdx.x; base < n_vec; base += stride) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const size_t i = base + (size_t)u * 512;
            v[u] = i < n_vec ? __ldcs(src + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) { acc.x ^= v[u].x; acc.y ^= v[u].y; acc.z ^= v[u].z; acc.w ^= v[u].w; }
    }
    if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x9E3779B9u && sink) *sink = acc.x;
}

}  // namespace

extern "C" int rabit_selftest_f16_plan(int K, int M, int N, int batch, int sms, int* bound_out, int max_out) {
    rabit_clear_error();
    if (!bound_out) return rabit_fail(RABIT_INVALID_ARG, "rabit_selftest_f16_plan: bound_out is NULL");
    const int grid = rabit_gemv_f16_plan(K, M, N, batch, sms, bound_out, max_out);
    if (grid < 0) return rabit_fail(RABIT_INVALID_ARG, "rabit_selftest_f16_plan: unsupported shape or too small an output array");
    return grid;
}

extern "C" int rabit_selftest_stream_read(const void* src_dev, size_t bytes, unsigned int* sink_dev, void* stream) {
    rabit_clear_error();
    if (!src_dev || ((uintptr_t)src_dev & 15u)) return rabit_fail(RABIT_INVALID_ARG, "rabit_selftest_stream_read: src_dev must be a 16-byte aligned device pointer");
    if (bytes < 16) return rabit_fail(RABIT_INVALID_ARG, "rabit_selftest_stream_read: bytes must be at least 16");
    int dev = 0, sms = 0;
    RABIT_CUDA_TRY(cudaGetDevice(&dev));
    RABIT_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    stream_read_probe<<<sms * 4, 512, 0, (cudaStream_t)stream>>>((const uint4*)src_dev, bytes / 16, sink_dev);
    RABIT_CUDA_TRY(cudaGetLastError());
    return RABIT_OK;
}

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
