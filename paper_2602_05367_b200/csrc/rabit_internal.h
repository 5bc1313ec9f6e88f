// Internal declarations shared by the library's translation units (not part of the ABI).
#ifndef RABIT_INTERNAL_H_
#define RABIT_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/rabit.h"
#include "rabit_layout.h"

struct rabit_layer {
    RabitGeom geom;
    int device;
    int variant;                 // 0 auto, 1 plain, 2 integer-MMA GEMV, 3 tcgen05 GEMM, 4 dequantised-tile GEMM, 5 table-driven GEMV, 6 f16 tensor-core GEMV
    int sm_count;
    char* dev_base;              // caller-owned packed image
    size_t dev_bytes;
    const uint4* d_bits;         // sign tiles
    const uint16_t* d_g;         // fp16 [K][Mp]
    const uint16_t* d_h;         // fp16 [K][N]
    float* d_partial;            // fp32 [n_rt*K + RABIT_MAX_GRID][RABIT_PARTIAL_BATCH][128] cross-CTA partial sums (all-ones words between calls)
    unsigned int* d_flags;       // u32 [n_rt*K + RABIT_MAX_GRID] reserved (stay zero; no kernel uses them), then one status word
    unsigned int* d_status;      // u32, non-zero once a kernel gave up on a bounded wait
    const unsigned char* d_lut;  // look-up blocks (table-driven GEMV)
    unsigned long long* d_acc;   // u64 [RABIT_LUT_MAX_BATCH][Mp] accumulate words of the table-driven GEMV (zero between calls)
};

// error reporting (thread-local message); returns `code`
int rabit_fail(int code, const char* fmt, ...);
void rabit_clear_error();
#define RABIT_CUDA_TRY(expr)                                                              \
    do {                                                                                  \
        cudaError_t e__ = (expr);                                                         \
        if (e__ != cudaSuccess)                                                           \
            return rabit_fail(RABIT_CUDA_ERROR, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

// geometry / layout (rabit_pack.cu)
bool rabit_make_geom(int K, int M, int N, RabitGeom* out);          // hmax left at 0
void rabit_fill_header(const RabitGeom& G, RabitHeader* hdr);
bool rabit_geom_from_header(const RabitHeader& hdr, RabitGeom* out); // validates magic, version and shape
void rabit_scale_meta(const uint16_t* g, const uint16_t* h, int K, int M, int N, RabitGeom* G);   // hmax and the fixed-point grid

// header + scale sections, for images whose tiles are written on the device (rabit_pack.cu)
#ifdef __cplusplus
#include <vector>
bool rabit_build_meta(const uint16_t* g, const uint16_t* h, int K, int M, int N, RabitGeom* geom, RabitHeader* hdr,
                      std::vector<uint8_t>* tail);
#endif
cudaError_t rabit_launch_derive(const RabitGeom& G, const float* W, const uint16_t* d_g, const uint16_t* d_h, uint4* d_tiles,
                                cudaStream_t stream);

// gathers the look-up blocks from the sign tiles, fills ones_bytes at d_ones with 0xFF and zero_bytes at d_zero with 0 (16-byte
// units) and, if header is not null, writes it (256 bytes, passed as a kernel parameter) to d_header
cudaError_t rabit_launch_tiles_to_lut(const RabitGeom& G, const uint4* d_tiles, unsigned char* d_lut, void* d_ones, size_t ones_bytes,
                                      void* d_zero, size_t zero_bytes, const RabitHeader* header, void* d_header, cudaStream_t stream);

// kernel launchers; each enqueues on `stream` and returns a cudaError_t from the launch
cudaError_t rabit_launch_plain(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream);
cudaError_t rabit_launch_gemv_mma(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream);
bool rabit_gemv_mma_supports(const rabit_layer& L, int batch);
int rabit_gemv_mma_max_group();
int rabit_gemv_mma_max_rows();
bool rabit_gemv_mma_group_supports(const rabit_layer* const* layers, int n_layers, int batch);
cudaError_t rabit_launch_gemv_mma_group(const rabit_layer* const* layers, int n_layers, const void* const* xs, void* const* ys,
                                        int batch, cudaStream_t stream);
unsigned int* rabit_static_scratch_status(int device);   // rabit_noalloc.cu; nullptr before the first static-scratch call on that device

// Phase tracing (rabit_api.cu): the next free record of 8 stamps x `ctas` in the caller's trace buffer, or nullptr
// when tracing is off, the buffer is full or the library was built without RABIT_TRACE.
unsigned long long* rabit_trace_slot(int ctas);

// f16 tensor-core GEMV for 3..16 batch rows (rabit_gemv_f16.cu)
cudaError_t rabit_launch_gemv_f16(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream);
bool rabit_gemv_f16_supports(const rabit_layer& L, int batch);
int rabit_gemv_f16_plan(int K, int M, int N, int batch, int sms, int* bound_out, int max_out);   // host only: the work split

// table-driven GEMV (rabit_gemv_lut.cu); acc_override / status_override redirect the scratch (nullptr: the image's own)
cudaError_t rabit_launch_gemv_lut(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream);
bool rabit_gemv_lut_supports(const rabit_layer& L, int batch);
int rabit_gemv_lut_max_rows();
bool rabit_gemv_lut_group_supports(const rabit_layer* const* layers, int n_layers, int batch);
cudaError_t rabit_launch_gemv_lut_group(const rabit_layer* const* layers, int n_layers, const void* const* xs, void* const* ys,
                                        int batch, cudaStream_t stream, unsigned long long* const* acc_override, unsigned int* status_override);
cudaError_t rabit_launch_gemm_tc(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream, bool dequantised = false);
bool rabit_gemm_tc_supports(const rabit_layer& L, int batch);
double rabit_gemm_tc_estimate_us(const rabit_layer& L, int batch);

#endif  // RABIT_INTERNAL_H_
