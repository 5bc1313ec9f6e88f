// C ABI of the library: argument checks, pack/upload, dispatch, error strings.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "rabit_internal.h"

static thread_local char g_err[512] = {0};

int rabit_fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}
void rabit_clear_error() { g_err[0] = 0; }

extern "C" const char* rabit_last_error(void) { return g_err; }

static void bind_layer(rabit_layer* L, const RabitGeom& G, const RabitHeader& hdr, void* dev_buf, int device) {
    L->geom = G;
    L->device = device;
    L->variant = 0;
    L->sm_count = 0;
    cudaDeviceGetAttribute(&L->sm_count, cudaDevAttrMultiProcessorCount, device);
    L->dev_base = (char*)dev_buf;
    L->dev_bytes = hdr.total_bytes;
    L->d_bits = (const uint4*)(L->dev_base + hdr.off_bits);
    L->d_g = (const uint16_t*)(L->dev_base + hdr.off_g);
    L->d_h = (const uint16_t*)(L->dev_base + hdr.off_h);
    L->d_partial = (float*)(L->dev_base + hdr.off_partial);
    L->d_flags = (unsigned int*)(L->dev_base + hdr.off_flags);
    L->d_status = L->d_flags + ((size_t)G.n_rt * G.K + RABIT_MAX_GRID);
    L->d_lut = (const unsigned char*)(L->dev_base + hdr.off_lut);
    L->d_acc = (unsigned long long*)(L->dev_base + hdr.off_acc);
}

extern "C" int rabit_pack(const uint32_t* planes, const uint16_t* g, const uint16_t* h,
                          int K, int M, int N, void* dev_buf, size_t dev_bytes, void* stream,
                          rabit_layer** out) {
    rabit_clear_error();
    if (!out) return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: out is NULL");
    *out = nullptr;
    if (!planes || !g || !h || !dev_buf) return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: null pointer");
    if (((uintptr_t)dev_buf & 255u) != 0) return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: dev_buf must be 256-byte aligned");
    RabitGeom G;
    if (!rabit_make_geom(K, M, N, &G))
        return rabit_fail(RABIT_UNSUPPORTED_SHAPE, "rabit_pack: unsupported shape K=%d M=%d N=%d (need 1<=K<=3, M>=1, N%%32==0)", K, M, N);
    RabitHeader hdr;
    rabit_fill_header(G, &hdr);
    if (dev_bytes < hdr.total_bytes)
        return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_pack: dev_buf holds %zu bytes, layer needs %zu", dev_bytes, (size_t)hdr.total_bytes);

    cudaPointerAttributes attr;
    RABIT_CUDA_TRY(cudaPointerGetAttributes(&attr, dev_buf));
    if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)
        return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: dev_buf is not device memory");

    std::vector<uint8_t> image;
    try {
        image.resize(hdr.total_bytes);
    } catch (const std::bad_alloc&) {
        return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: out of host memory for the staging image");
    }
    int rc = rabit_pack_host(planes, g, h, K, M, N, image.data(), image.size());
    if (rc != RABIT_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    RABIT_CUDA_TRY(cudaMemcpyAsync(dev_buf, image.data(), hdr.total_bytes, cudaMemcpyHostToDevice, st));
    RABIT_CUDA_TRY(cudaStreamSynchronize(st));

    rabit_layer* L = new (std::nothrow) rabit_layer;
    if (!L) return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: out of host memory");
    RabitHeader packed_hdr;
    std::memcpy(&packed_hdr, image.data(), sizeof(packed_hdr));
    RabitGeom packed_geom;
    if (!rabit_geom_from_header(packed_hdr, &packed_geom)) {
        delete L;
        return rabit_fail(RABIT_INVALID_ARG, "rabit_pack: internal error, packed header unreadable");
    }
    bind_layer(L, packed_geom, packed_hdr, dev_buf, attr.device);
    *out = L;
    return RABIT_OK;
}

static bool ranges_overlap(const void* a, size_t an, const void* b, size_t bn);


extern "C" int rabit_derive_pack(const float* W_dev, const uint16_t* g, const uint16_t* h, int K, int M, int N,
                                 void* dev_buf, size_t dev_bytes, void* stream, rabit_layer** out) {
    rabit_clear_error();
    if (!out) return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: out is NULL");
    *out = nullptr;
    if (!W_dev || !g || !h || !dev_buf) return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: null pointer");
    if (((uintptr_t)dev_buf & 255u) != 0) return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: dev_buf must be 256-byte aligned");
    if (((uintptr_t)W_dev & 15u) != 0) return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: W must be 16-byte aligned");
    RabitGeom G;
    RabitHeader hdr;
    std::vector<uint8_t> tail;
    try {
        if (!rabit_build_meta(g, h, K, M, N, &G, &hdr, &tail))
            return rabit_fail(RABIT_UNSUPPORTED_SHAPE, "rabit_derive_pack: unsupported shape K=%d M=%d N=%d (need 1<=K<=3, M>=1, N%%32==0)", K, M, N);
    } catch (const std::bad_alloc&) {
        return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: out of host memory");
    }
    if (dev_bytes < hdr.total_bytes)
        return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_derive_pack: dev_buf holds %zu bytes, layer needs %zu", dev_bytes, (size_t)hdr.total_bytes);
    cudaPointerAttributes attr;
    RABIT_CUDA_TRY(cudaPointerGetAttributes(&attr, dev_buf));
    if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)
        return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: dev_buf is not device memory");
    if (ranges_overlap(W_dev, (size_t)M * N * 4, dev_buf, hdr.total_bytes))
        return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: W overlaps dev_buf");
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)dev_buf;
    // scales from the host (a few KB); the header travels as a parameter of the second kernel
    RABIT_CUDA_TRY(cudaMemcpyAsync(base + hdr.off_g, tail.data(), tail.size(), cudaMemcpyHostToDevice, st));
    cudaError_t e = rabit_launch_derive(G, W_dev, (const uint16_t*)(base + hdr.off_g), (const uint16_t*)(base + hdr.off_h),
                                        (uint4*)(base + hdr.off_bits), st);
    // the second kernel also puts the exchange buffer (all-ones words) and the flags (zero) into their resting state
    if (e == cudaSuccess)
        e = rabit_launch_tiles_to_lut(G, (const uint4*)(base + hdr.off_bits), (unsigned char*)(base + hdr.off_lut),
                                      base + hdr.off_partial, (size_t)(hdr.off_flags - hdr.off_partial),
                                      base + hdr.off_flags, (size_t)(hdr.off_lut - hdr.off_flags), &hdr, base, st);
    if (e != cudaSuccess) return rabit_fail(RABIT_CUDA_ERROR, "rabit_derive_pack: launch failed: %s", cudaGetErrorString(e));
    // The accumulate words are cleared AFTER the kernels on purpose: the decode kernels start copying weights before
    // they wait for the previous kernel in the stream (weights normally never depend on it).  A fill between the
    // kernels that write this layer's weights and its first use is an ordinary stream dependency, which such a
    // kernel cannot overtake.
    RABIT_CUDA_TRY(cudaMemsetAsync(base + hdr.off_acc, 0, (size_t)(hdr.total_bytes - hdr.off_acc), st));
    // No synchronisation: copies from pageable host memory return once the source has been staged, so the
    // local buffers may go out of scope; the layer is usable by later work on the same stream.
    rabit_layer* L = new (std::nothrow) rabit_layer;
    if (!L) return rabit_fail(RABIT_INVALID_ARG, "rabit_derive_pack: out of host memory");
    bind_layer(L, G, hdr, dev_buf, attr.device);
    *out = L;
    return RABIT_OK;
}

static bool ranges_overlap(const void* a, size_t an, const void* b, size_t bn) {
    uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bn && b0 < a0 + an;
}

extern "C" int rabit_linear(const rabit_layer* layer, const void* x, void* y, int batch, void* stream) {
    rabit_clear_error();
    if (!layer) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: layer is NULL");
    if (!x || !y) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: null x or y");
    if (batch < 1) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: batch must be >= 1 (got %d)", batch);
    if ((((uintptr_t)x) & 15u) || (((uintptr_t)y) & 15u))
        return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: x and y must be 16-byte aligned");
    const RabitGeom& G = layer->geom;
    if (ranges_overlap(x, (size_t)batch * G.N * 2, y, (size_t)batch * G.M * 2))
        return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: x and y overlap");
    cudaStream_t st = (cudaStream_t)stream;
    {
        int dev = -1;
        RABIT_CUDA_TRY(cudaGetDevice(&dev));
        if (dev != layer->device)
            return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: the layer lives on device %d but device %d is current", layer->device, dev);
    }

    int variant = layer->variant;
    if (variant == 0) {
        const double packed_mb = (double)G.K * G.Mp * G.N / 8.0e6;
        if (rabit_gemv_lut_supports(*layer, batch)) {
            variant = 5;
        } else if (batch <= 2 * RABIT_MAX_GEMV_BATCH && rabit_gemv_f16_supports(*layer, RABIT_MAX_GEMV_BATCH)) {
            variant = 6;                    // 3..16 rows: one pass over the weights with the batch in the MMA's N dimension;
                                            // 17..32: two passes, which measured faster than one GEMM launch on every shape tried
        } else if (batch <= 4 && packed_mb <= 8.0 && rabit_gemv_lut_supports(*layer, 1)) {
            variant = 5;                    // two passes of the table-driven kernel
        } else if (batch <= RABIT_MAX_GEMV_BATCH) {
            variant = rabit_gemv_mma_supports(*layer, batch) ? 2 : 1;
            // From 5 batch rows on the integer-MMA GEMV makes two to four passes over the weights; the tensor-core GEMM,
            // whose cost does not depend on the batch up to 256, is then often cheaper.  Both estimates are fits to
            // measurements on B200 (us): a GEMV pass of four rows costs 10 + max(0, packed MB - 4) / 1.3.
            if (variant == 2 && batch > 4 && rabit_gemm_tc_supports(*layer, batch)) {
                const double passes = (double)((batch + rabit_gemv_mma_max_rows() - 1) / rabit_gemv_mma_max_rows());
                const double gemv_us = passes * (10.0 + (packed_mb > 4.0 ? (packed_mb - 4.0) / 1.3 : 0.0));
                const double gemm_us = rabit_gemm_tc_estimate_us(*layer, batch);
                if (gemm_us < 0.9 * gemv_us) variant = 3;
            }
        } else {
            variant = rabit_gemm_tc_supports(*layer, batch) ? 3 : 1;
        }
    }
    cudaError_t e;
    switch (variant) {
        case 2:
            if (!rabit_gemv_mma_supports(*layer, batch))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: integer-MMA GEMV cannot run batch %d", batch);
            e = cudaSuccess;
            for (int b0 = 0; b0 < batch && e == cudaSuccess; b0 += rabit_gemv_mma_max_rows())   // up to 4 batch rows share one pass over the weights
                e = rabit_launch_gemv_mma(*layer, (const char*)x + (size_t)b0 * G.N * 2, (char*)y + (size_t)b0 * G.M * 2,
                                          batch - b0 >= rabit_gemv_mma_max_rows() ? rabit_gemv_mma_max_rows() : batch - b0, st);
            break;
        case 3:
            if (!rabit_gemm_tc_supports(*layer, batch))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: tcgen05 GEMM cannot run batch %d", batch);
            e = rabit_launch_gemm_tc(*layer, x, y, batch, st);
            break;
        case 4:
            if (!rabit_gemm_tc_supports(*layer, batch))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: tcgen05 GEMM cannot run batch %d", batch);
            e = rabit_launch_gemm_tc(*layer, x, y, batch, st, true);
            break;
        case 5: {
            if (!rabit_gemv_lut_supports(*layer, 1))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: table-driven GEMV cannot run this layer");
            const int rows = rabit_gemv_lut_supports(*layer, rabit_gemv_lut_max_rows()) ? rabit_gemv_lut_max_rows() : 1;
            e = cudaSuccess;
            for (int b0 = 0; b0 < batch && e == cudaSuccess; b0 += rows)             // up to `rows` batch rows share one pass over the weights
                e = rabit_launch_gemv_lut(*layer, (const char*)x + (size_t)b0 * G.N * 2, (char*)y + (size_t)b0 * G.M * 2,
                                          batch - b0 >= rows ? rows : batch - b0, st);
            break;
        }
        case 6:
            if (!rabit_gemv_f16_supports(*layer, batch < RABIT_MAX_GEMV_BATCH ? batch : RABIT_MAX_GEMV_BATCH))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear: f16 tensor-core GEMV cannot run this layer");
            e = cudaSuccess;
            for (int b0 = 0; b0 < batch && e == cudaSuccess; b0 += RABIT_MAX_GEMV_BATCH)   // up to 16 batch rows share one pass over the weights
                e = rabit_launch_gemv_f16(*layer, (const char*)x + (size_t)b0 * G.N * 2, (char*)y + (size_t)b0 * G.M * 2,
                                          batch - b0 >= RABIT_MAX_GEMV_BATCH ? RABIT_MAX_GEMV_BATCH : batch - b0, st);
            break;
        default:
            e = rabit_launch_plain(*layer, x, y, batch, st);
            break;
    }
    if (e != cudaSuccess) return rabit_fail(RABIT_CUDA_ERROR, "rabit_linear: launch failed: %s", cudaGetErrorString(e));
    return RABIT_OK;
}

extern "C" int rabit_linear_group(const rabit_layer* const* layers, const void* const* xs, void* const* ys,
                                  int n_layers, int batch, void* stream) {
    rabit_clear_error();
    if (!layers || !xs || !ys) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: null array");
    if (n_layers < 1) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: n_layers must be >= 1 (got %d)", n_layers);
    if (batch < 1) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: batch must be >= 1 (got %d)", batch);
    for (int l = 0; l < n_layers; ++l) {
        if (!layers[l] || !xs[l] || !ys[l]) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: null entry %d", l);
        if ((((uintptr_t)xs[l]) & 15u) || (((uintptr_t)ys[l]) & 15u))
            return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: x and y of entry %d must be 16-byte aligned", l);
        if (layers[l]->device != layers[0]->device)
            return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: entry %d lives on another device", l);
    }
    for (int a = 0; a < n_layers; ++a) {
        const size_t ya = (size_t)batch * layers[a]->geom.M * 2;
        for (int b = 0; b < n_layers; ++b) {
            if (ranges_overlap(ys[a], ya, xs[b], (size_t)batch * layers[b]->geom.N * 2))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: output %d overlaps input %d", a, b);
            if (b > a && ranges_overlap(ys[a], ya, ys[b], (size_t)batch * layers[b]->geom.M * 2))
                return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: outputs %d and %d overlap", a, b);
        }
    }
    cudaStream_t st = (cudaStream_t)stream;
    {
        int dev = -1;
        RABIT_CUDA_TRY(cudaGetDevice(&dev));
        if (dev != layers[0]->device)
            return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group: the layers live on device %d but device %d is current", layers[0]->device, dev);
    }
    {
        bool lut = rabit_gemv_lut_group_supports(layers, n_layers, batch);
        for (int l = 0; l < n_layers && lut; ++l) lut = layers[l]->variant == 0 || layers[l]->variant == 5;
        if (lut) {
            cudaError_t e = rabit_launch_gemv_lut_group(layers, n_layers, xs, ys, batch, st, nullptr, nullptr);
            if (e != cudaSuccess) return rabit_fail(RABIT_CUDA_ERROR, "rabit_linear_group: launch failed: %s", cudaGetErrorString(e));
            return RABIT_OK;
        }
    }
    {
        bool f16 = true;                                         // 3..16 rows: every layer takes the f16 tensor-core GEMV, launch by launch
        for (int l = 0; l < n_layers && f16; ++l) f16 = layers[l]->variant == 0 && rabit_gemv_f16_supports(*layers[l], batch);
        if (f16) {
            for (int l = 0; l < n_layers; ++l) {
                int rc = rabit_linear(layers[l], xs[l], ys[l], batch, stream);
                if (rc != RABIT_OK) return rc;
            }
            return RABIT_OK;
        }
    }
    for (int a = 0; a < n_layers; ++a)
        for (int b = a + 1; b < n_layers; ++b)
            if (layers[a] == layers[b]) {                        // the same layer twice would share one reduction scratch: no fused launch
                for (int l = 0; l < n_layers; ++l) {
                    int rc = rabit_linear(layers[l], xs[l], ys[l], batch, stream);
                    if (rc != RABIT_OK) return rc;
                }
                return RABIT_OK;
            }
    bool fused = rabit_gemv_mma_group_supports(layers, n_layers, batch);
    for (int l = 0; l < n_layers && fused; ++l) fused = layers[l]->variant == 0 || layers[l]->variant == 2;
    if (!fused) {
        for (int l = 0; l < n_layers; ++l) {
            int rc = rabit_linear(layers[l], xs[l], ys[l], batch, stream);
            if (rc != RABIT_OK) return rc;
        }
        return RABIT_OK;
    }
    const void* xb[8];
    void* yb[8];
    cudaError_t e = cudaSuccess;
    const int rows = rabit_gemv_mma_max_rows();
    for (int b0 = 0; b0 < batch && e == cudaSuccess; b0 += rows) {         // up to 4 batch rows share one pass over the weights
        for (int l = 0; l < n_layers; ++l) {
            xb[l] = (const char*)xs[l] + (size_t)b0 * layers[l]->geom.N * 2;
            yb[l] = (char*)ys[l] + (size_t)b0 * layers[l]->geom.M * 2;
        }
        e = rabit_launch_gemv_mma_group(layers, n_layers, xb, yb, batch - b0 >= rows ? rows : batch - b0, st);
    }
    if (e != cudaSuccess) return rabit_fail(RABIT_CUDA_ERROR, "rabit_linear_group: launch failed: %s", cudaGetErrorString(e));
    return RABIT_OK;
}

extern "C" size_t rabit_stage_bytes(const rabit_layer* layer, int batch) {
    if (!layer || batch < 1) return 0;
    return rabit_align256((size_t)batch * layer->geom.N * 2) + rabit_align256((size_t)batch * layer->geom.M * 2);
}

// Device address under which the GPU can store straight into a host buffer of `bytes` bytes (page-locked,
// mapped memory, 16-byte aligned), or nullptr if the buffer is ordinary pageable memory.
static void* mapped_output_alias(void* host_ptr, size_t bytes) {
    cudaPointerAttributes first, last;
    if (cudaPointerGetAttributes(&first, host_ptr) != cudaSuccess || cudaPointerGetAttributes(&last, (char*)host_ptr + bytes - 1) != cudaSuccess) {
        cudaGetLastError();                                              // not an error of the caller: fall back to a copy
        return nullptr;
    }
    if (first.type != cudaMemoryTypeHost || last.type != cudaMemoryTypeHost || !first.devicePointer || !last.devicePointer) return nullptr;
    if ((char*)last.devicePointer - (char*)first.devicePointer != (ptrdiff_t)(bytes - 1)) return nullptr;
    if (((uintptr_t)first.devicePointer & 15u) != 0) return nullptr;
    return first.devicePointer;
}

extern "C" int rabit_linear_host(const rabit_layer* layer, const void* x_host, void* y_host, int batch,
                                 void* dev_stage, size_t dev_stage_bytes, void* stream) {
    rabit_clear_error();
    if (!layer) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_host: layer is NULL");
    if (!x_host || !y_host || !dev_stage) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_host: null pointer");
    if (batch < 1) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_host: batch must be >= 1 (got %d)", batch);
    if (((uintptr_t)dev_stage & 255u) != 0) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_host: dev_stage must be 256-byte aligned");
    const size_t need = rabit_stage_bytes(layer, batch);
    if (dev_stage_bytes < need)
        return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_linear_host: stage holds %zu bytes, need %zu", dev_stage_bytes, need);
    const size_t xb = (size_t)batch * layer->geom.N * 2, yb = (size_t)batch * layer->geom.M * 2;
    char* dx = (char*)dev_stage;
    char* dy = dx + rabit_align256(xb);
    cudaStream_t st = (cudaStream_t)stream;
    RABIT_CUDA_TRY(cudaMemcpyAsync(dx, x_host, xb, cudaMemcpyHostToDevice, st));
    // A decode-sized result goes straight to mapped host memory from the kernel's last stores (a few KB; the
    // copy engine's latency for so small a copy is longer than the kernel); anything else through the stage.
    void* direct = batch <= RABIT_MAX_GEMV_BATCH ? mapped_output_alias(y_host, yb) : nullptr;
    int rc = rabit_linear(layer, dx, direct ? direct : dy, batch, stream);
    if (rc != RABIT_OK) return rc;
    if (!direct) RABIT_CUDA_TRY(cudaMemcpyAsync(y_host, dy, yb, cudaMemcpyDeviceToHost, st));
    return RABIT_OK;
}

extern "C" size_t rabit_group_stage_bytes(const rabit_layer* const* layers, int n_layers, int batch) {
    if (!layers || n_layers < 1 || n_layers > 8 || batch < 1) return 0;
    size_t total = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (!layers[l]) return 0;
        total += rabit_align256((size_t)batch * layers[l]->geom.N * 2) + rabit_align256((size_t)batch * layers[l]->geom.M * 2);
    }
    return total;
}

extern "C" int rabit_linear_group_host(const rabit_layer* const* layers, const void* const* xs_host, void* const* ys_host,
                                       int n_layers, int batch, void* dev_stage, size_t dev_stage_bytes, void* stream) {
    rabit_clear_error();
    if (!layers || !xs_host || !ys_host || !dev_stage) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group_host: null pointer");
    if (n_layers < 1 || n_layers > 8) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group_host: n_layers must be 1..8 (got %d)", n_layers);
    if (batch < 1) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group_host: batch must be >= 1 (got %d)", batch);
    if (((uintptr_t)dev_stage & 255u) != 0) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group_host: dev_stage must be 256-byte aligned");
    for (int l = 0; l < n_layers; ++l)
        if (!layers[l] || !xs_host[l] || !ys_host[l]) return rabit_fail(RABIT_INVALID_ARG, "rabit_linear_group_host: null entry %d", l);
    const size_t need = rabit_group_stage_bytes(layers, n_layers, batch);
    if (dev_stage_bytes < need)
        return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_linear_group_host: stage holds %zu bytes, need %zu", dev_stage_bytes, need);
    cudaStream_t st = (cudaStream_t)stream;
    char* cur = (char*)dev_stage;
    const void* dx[8];
    void* dy[8];
    for (int l = 0; l < n_layers; ++l) {
        const size_t xb = (size_t)batch * layers[l]->geom.N * 2;
        dx[l] = nullptr;
        for (int m = 0; m < l; ++m)                                      // the same host input (and width) again: reuse its copy
            if (xs_host[m] == xs_host[l] && layers[m]->geom.N == layers[l]->geom.N) { dx[l] = dx[m]; break; }
        if (!dx[l]) {
            RABIT_CUDA_TRY(cudaMemcpyAsync(cur, xs_host[l], xb, cudaMemcpyHostToDevice, st));
            dx[l] = cur;
            cur += rabit_align256(xb);
        }
    }
    bool staged[8];
    for (int l = 0; l < n_layers; ++l) {                                 // decode-sized results: straight to mapped host memory (see rabit_linear_host)
        const size_t yb = (size_t)batch * layers[l]->geom.M * 2;
        void* direct = batch <= RABIT_MAX_GEMV_BATCH ? mapped_output_alias(ys_host[l], yb) : nullptr;
        staged[l] = direct == nullptr;
        dy[l] = direct ? direct : cur;
        cur += rabit_align256(yb);
    }
    int rc = rabit_linear_group(layers, dx, dy, n_layers, batch, stream);
    if (rc != RABIT_OK) return rc;
    for (int l = 0; l < n_layers; ++l)
        if (staged[l]) RABIT_CUDA_TRY(cudaMemcpyAsync(ys_host[l], dy[l], (size_t)batch * layers[l]->geom.M * 2, cudaMemcpyDeviceToHost, st));
    return RABIT_OK;
}

extern "C" int rabit_layer_status(const rabit_layer* layer, int clear, void* stream) {
    rabit_clear_error();
    if (!layer) return rabit_fail(RABIT_INVALID_ARG, "rabit_layer_status: layer is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    // two words can record a wait that ran out: the layer's own (inside its packed image) and the one of the library's
    // built-in scratch array, which rabit_linear_static_scratch uses for every layer
    unsigned int word = 0, word_static = 0;
    unsigned int* d_static = rabit_static_scratch_status(layer->device);
    RABIT_CUDA_TRY(cudaMemcpyAsync(&word, layer->d_status, 4, cudaMemcpyDeviceToHost, st));
    if (d_static) RABIT_CUDA_TRY(cudaMemcpyAsync(&word_static, d_static, 4, cudaMemcpyDeviceToHost, st));
    RABIT_CUDA_TRY(cudaStreamSynchronize(st));
    if (word != 0 || word_static != 0) {
        if (clear) {
            // a contributor that gave up may still have published a partial sum after its finisher restored the resting
            // state: put the whole exchange buffer back, not just the word
            const size_t partial_bytes = (size_t)((const char*)layer->d_flags - (const char*)layer->d_partial);
            RABIT_CUDA_TRY(cudaMemsetAsync(layer->d_partial, 0xFF, partial_bytes, st));
            RABIT_CUDA_TRY(cudaMemsetAsync(layer->d_status, 0, 4, st));
            if (d_static) RABIT_CUDA_TRY(cudaMemsetAsync(d_static, 0, 4, st));
            RABIT_CUDA_TRY(cudaStreamSynchronize(st));
        }
        return rabit_fail(RABIT_DEVICE_FAULT, "rabit_layer_status: a kernel of this layer%s gave up on a bounded wait; the outputs of that call are invalid",
                          word_static != 0 ? " (or another layer run through the built-in scratch array)" : "");
    }
    return RABIT_OK;
}

extern "C" int rabit_unpack(const rabit_layer* layer, uint32_t* planes_out, uint16_t* g_out, uint16_t* h_out, void* stream) {
    rabit_clear_error();
    if (!layer) return rabit_fail(RABIT_INVALID_ARG, "rabit_unpack: layer is NULL");
    std::vector<uint8_t> image;
    try {
        image.resize(layer->dev_bytes);
    } catch (const std::bad_alloc&) {
        return rabit_fail(RABIT_INVALID_ARG, "rabit_unpack: out of host memory");
    }
    cudaStream_t st = (cudaStream_t)stream;
    RABIT_CUDA_TRY(cudaMemcpyAsync(image.data(), layer->dev_base, layer->dev_bytes, cudaMemcpyDeviceToHost, st));
    RABIT_CUDA_TRY(cudaStreamSynchronize(st));
    return rabit_unpack_host(image.data(), image.size(), planes_out, g_out, h_out);
}

// ---- phase tracing (only does something in a library built with -DRABIT_TRACE) -------------------
#ifdef RABIT_TRACE
static unsigned long long* g_trace_buf = nullptr;
static size_t g_trace_words = 0, g_trace_used = 0;
static std::vector<int> g_trace_ctas;                                    // CTAs of every traced launch, in launch order
#endif

unsigned long long* rabit_trace_slot(int ctas) {
#ifdef RABIT_TRACE
    if (!g_trace_buf || ctas < 1) return nullptr;
    const size_t need = (size_t)ctas * 64;
    if (g_trace_used + need > g_trace_words) return nullptr;
    unsigned long long* rec = g_trace_buf + g_trace_used;
    g_trace_used += need;
    g_trace_ctas.push_back(ctas);
    return rec;
#else
    (void)ctas;
    return nullptr;
#endif
}

extern "C" int rabit_trace_begin(void* dev_buf, size_t bytes) {
    rabit_clear_error();
#ifdef RABIT_TRACE
    if (dev_buf && (((uintptr_t)dev_buf & 7u) != 0 || bytes < 64))
        return rabit_fail(RABIT_INVALID_ARG, "rabit_trace_begin: buffer must be 8-byte aligned and hold at least 64 bytes");
    g_trace_buf = (unsigned long long*)dev_buf;
    g_trace_words = dev_buf ? bytes / 8 : 0;
    g_trace_used = 0;
    g_trace_ctas.clear();
    return RABIT_OK;
#else
    (void)dev_buf; (void)bytes;
    return rabit_fail(RABIT_UNSUPPORTED_SHAPE, "rabit_trace_begin: this library was built without RABIT_TRACE");
#endif
}

extern "C" int rabit_trace_launches(int* ctas_out, int max_launches) {
#ifdef RABIT_TRACE
    const int n = (int)g_trace_ctas.size();
    for (int i = 0; i < n && i < max_launches && ctas_out; ++i) ctas_out[i] = g_trace_ctas[i];
    return n;
#else
    (void)ctas_out; (void)max_launches;
    return 0;
#endif
}

extern "C" int rabit_layer_K(const rabit_layer* layer) { return layer ? layer->geom.K : -1; }
extern "C" int rabit_layer_M(const rabit_layer* layer) { return layer ? layer->geom.M : -1; }
extern "C" int rabit_layer_N(const rabit_layer* layer) { return layer ? layer->geom.N : -1; }

extern "C" int rabit_set_variant(rabit_layer* layer, int variant) {
    rabit_clear_error();
    if (!layer) return rabit_fail(RABIT_INVALID_ARG, "rabit_set_variant: layer is NULL");
    if (variant < 0 || variant > 6) return rabit_fail(RABIT_INVALID_ARG, "rabit_set_variant: variant must be 0..6");
    layer->variant = variant;
    return RABIT_OK;
}

extern "C" int rabit_free(rabit_layer* layer) {
    rabit_clear_error();
    delete layer;
    return RABIT_OK;
}
