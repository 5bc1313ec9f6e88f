// rabit_linear_static_scratch: the decode GEMV with its reduction scratch in a fixed device array
// that belongs to the library, for callers that must not allocate device memory.
//
// The GEMV needs two pieces of scratch per call: the fp32 partial sums that the CTAs of a row
// tile exchange and a status word.  rabit_linear keeps them inside the packed
// image that the caller allocated.  Here they live in a file-scope device array of a fixed size,
// so the call neither needs a scratch-bearing buffer nor allocates one.
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr size_t kScratchBytes = (size_t)4 << 20;        // 4 MiB, held by every GPU that loads the library
constexpr int kMaxDevices = 64;
constexpr size_t kStatusOffset = kScratchBytes - 256;    // one status word for all calls, at a fixed place; it starts at zero
                                                         // (static storage) and only rabit_layer_status(clear) puts it back

// Partial sums | reserved | status word.  Every call shares this array.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// Device address of the array per device, resolved on the first call on that device.
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

struct ScratchPlan {
    size_t entries;          // segment slots: n_rt * K + RABIT_MAX_GRID
    size_t partial_bytes, flags_off, flags_bytes, status_off, total;
};

ScratchPlan plan_for(const RabitGeom& G) {
    ScratchPlan p;
    p.entries = (size_t)G.n_rt * G.K + RABIT_MAX_GRID;
    p.partial_bytes = p.entries * RABIT_PARTIAL_BATCH * RABIT_TILE_ROWS * 4;
    p.flags_off = rabit_align256(p.partial_bytes);
    p.flags_bytes = p.entries * 4;
    p.status_off = p.flags_off + rabit_align256(p.flags_bytes);
    p.total = p.status_off + 256;                            // (the status word itself sits at the end of the array, see kStatusOffset)
    return p;
}

}  // namespace

// The status word of the built-in array on `device`, or nullptr if no call has set the array up there yet.
unsigned int* rabit_static_scratch_status(int device) {
    if (device < 0 || device >= kMaxDevices || !g_scratch_ptr[device]) return nullptr;
    return reinterpret_cast<unsigned int*>(g_scratch_ptr[device] + kStatusOffset);
}

extern "C" int rabit_linear_static_scratch(const rabit_layer* layer, const void* x, void* y, int batch, void* stream) {
    rabit_clear_error();
    if (!layer) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: layer is NULL");
    if (!x || !y) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: null x or y");
    if (batch < 1 || batch > RABIT_MAX_GEMV_BATCH)
        return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: batch must be 1..%d (got %d)", RABIT_MAX_GEMV_BATCH, batch);
    if ((((uintptr_t)x) & 15u) || (((uintptr_t)y) & 15u))
        return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: x and y must be 16-byte aligned");
    const RabitGeom& G = layer->geom;
    {
        const uintptr_t x0 = (uintptr_t)x, y0 = (uintptr_t)y;
        const size_t xn = (size_t)batch * G.N * 2, yn = (size_t)batch * G.M * 2;
        if (x0 < y0 + yn && y0 < x0 + xn) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: x and y overlap");
    }
    if (!rabit_gemv_mma_supports(*layer, batch))
        return rabit_fail(RABIT_UNSUPPORTED_SHAPE, "rabit_linear_static_scratch: the GEMV kernel cannot run this layer");
    const ScratchPlan plan = plan_for(G);
    if (plan.total > kStatusOffset)
        return rabit_fail(RABIT_UNSUPPORTED_SHAPE,
                          "rabit_linear_static_scratch: layer needs %zu bytes of reduction scratch, the built-in array holds %zu "
                          "(K * ceil(M/128) must stay below about %zu)",
                          plan.total, kScratchBytes, kScratchBytes / (RABIT_PARTIAL_BATCH * RABIT_TILE_ROWS * 4 + 4) - RABIT_MAX_GRID);

    int dev = -1;
    RABIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != layer->device)
        return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: the layer lives on device %d but device %d is current", layer->device, dev);
    if (dev < 0 || dev >= kMaxDevices) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_static_scratch: device index %d out of range", dev);
    if (!g_scratch_ptr[dev]) {
        // The array's name is only a host-side handle; the kernel needs its address on this device.
        unsigned char* p = nullptr;
        RABIT_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_static_scratch));
        g_scratch_ptr[dev] = p;
    }
    unsigned char* base = g_scratch_ptr[dev];
    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the last call (of any layer) left: the partial slots of this layer must
    // start in their resting state (all-ones words) and the status word at zero.
    RABIT_CUDA_TRY(cudaMemsetAsync(base, 0xFF, plan.partial_bytes, st));
    RABIT_CUDA_TRY(cudaMemsetAsync(base + plan.flags_off, 0, plan.status_off - plan.flags_off, st));

    rabit_layer view = *layer;                               // same weights and scales, scratch redirected
    view.d_partial = reinterpret_cast<float*>(base);
    view.d_flags = reinterpret_cast<unsigned int*>(base + plan.flags_off);
    view.d_status = reinterpret_cast<unsigned int*>(base + kStatusOffset);
    cudaError_t e = cudaSuccess;
    const int rows = rabit_gemv_mma_max_rows();
    for (int b0 = 0; b0 < batch && e == cudaSuccess; b0 += rows)
        e = rabit_launch_gemv_mma(view, (const char*)x + (size_t)b0 * G.N * 2, (char*)y + (size_t)b0 * G.M * 2,
                                  batch - b0 >= rows ? rows : batch - b0, st);
    if (e != cudaSuccess) return rabit_fail(RABIT_CUDA_ERROR, "rabit_linear_static_scratch: launch failed: %s", cudaGetErrorString(e));
    return RABIT_OK;
}
