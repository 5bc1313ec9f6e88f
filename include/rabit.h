/*
 * rabit.h -- C ABI of the B200 residual-binary linear layer library.
 *
 * The layer (paper Section 4.1 and Eq. 2, "stacked binary weight") is
 *
 *     y[b][i] = sum_{k<K} g_k[i] * sum_{j<N} B_k[i][j] * h_k[j] * x[b][j]
 *
 * with K stacked sign matrices B_k in {-1,+1}^{M x N}, a per-output scale g_k (length M)
 * and a per-input scale h_k (length N) per path; at inference the sign matrices are frozen
 * and only bits + scales remain (end of Section 4.2).  Signs are stored one bit each,
 * +1 -> 0 and -1 -> 1 (Appendix "Weight Packing").
 *
 * Conventions
 *   - M = d_out, N = d_in, K = number of paths (1..3), batch = number of activation rows.
 *   - Every function returns RABIT_OK (0) or a negative rabit_status; none throws, prints
 *     or exits.  rabit_last_error() returns a thread-local description of the last failure.
 *   - "HOST" / "DEVICE" on a pointer says which memory it must point into.
 *   - Device memory is always owned by the caller (for example a torch tensor); the library
 *     never frees it.  A rabit_layer is a small host-side descriptor that refers to it.
 *   - All device work is enqueued on the cudaStream_t passed as `stream` (void*, may be 0).
 */
#ifndef RABIT_H_
#define RABIT_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RABIT_API __attribute__((visibility("default")))
#else
#define RABIT_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum rabit_status {
    RABIT_OK = 0,
    RABIT_INVALID_ARG = -1,        /* null pointer, misaligned pointer, aliasing, batch < 1 ... */
    RABIT_UNSUPPORTED_SHAPE = -2,  /* K outside 1..3, M < 1, N < 32 or N not a multiple of 32 */
    RABIT_BUFFER_TOO_SMALL = -3,   /* dev_bytes / out_bytes below the required size */
    RABIT_CUDA_ERROR = -4,         /* a CUDA runtime call failed; see rabit_last_error() */
    RABIT_DEVICE_FAULT = -5        /* a kernel reported an internal bounded wait that ran out */
} rabit_status;

typedef struct rabit_layer rabit_layer;   /* opaque host-side descriptor */

/* Version of the packed device layout written by rabit_pack_host (also stored in its header): 3. */
RABIT_API int rabit_layout_version(void);

/*
 * Bytes of the packed image of a K x M x N layer: header + the sign bits in two arrangements (tiles for the
 * tensor-core kernels, byte look-up blocks for the table-driven decode kernel: 2K bits per weight in device memory,
 * of which a call reads K) + padded fp16 scales + the per-layer reduction scratch.  Returns 0 for an unsupported shape.
 * (Storage accounting of Section 4.1: K bits per weight plus the scale vectors.)
 */
RABIT_API size_t rabit_packed_bytes(int K, int M, int N);

/*
 * Step "pack" (Appendix "Weight Packing", re-designed layout): permute canonical sign planes
 * and scales into the device layout, entirely on the host.
 *   planes  HOST  uint32 [K][M][N/32]; column j is bit (j % 32), LSB first, of word j / 32;
 *                 bit 1 means -1, bit 0 means +1.
 *   g       HOST  fp16 bit patterns [K][M]   (per-output scale of each path)
 *   h       HOST  fp16 bit patterns [K][N]   (per-input scale of each path)
 *   out     HOST  receives rabit_packed_bytes(K,M,N) bytes; out_bytes must be at least that.
 * Needs no GPU.  The image is byte-for-byte what rabit_pack places in device memory.
 */
RABIT_API int rabit_pack_host(const uint32_t* planes, const uint16_t* g, const uint16_t* h,
                    int K, int M, int N, void* out, size_t out_bytes);

/*
 * Inverse of rabit_pack_host on a HOST image: recovers canonical planes and scales
 * bit-exactly.  Any of planes_out / g_out / h_out may be NULL to skip it.
 */
RABIT_API int rabit_unpack_host(const void* image, size_t image_bytes,
                      uint32_t* planes_out, uint16_t* g_out, uint16_t* h_out);

/*
 * Pack (as rabit_pack_host) and copy the image into caller-owned device memory, then create
 * the descriptor.
 *   dev_buf   DEVICE  256-byte aligned, dev_bytes >= rabit_packed_bytes(K,M,N); must stay
 *                     valid and unmodified by the caller until rabit_free.
 *   stream    the copy is enqueued on it and the call returns after it has completed.
 *   out       receives the new descriptor.
 * dev_buf also holds the layer's reduction scratch, in its resting state: the fp32 exchange buffer of the tensor-core
 * GEMV is all-ones words (0xFFFFFFFF, "nothing published"), the 64-bit accumulate words of the table-driven and f16 GEMVs, the
 * reserved flags and the status word are zero.  Every call leaves it in that state, so calls on one layer must not
 * overlap in time (different layers may).  A caller that moves or restores an image must keep these values.
 */
RABIT_API int rabit_pack(const uint32_t* planes, const uint16_t* g, const uint16_t* h,
               int K, int M, int N, void* dev_buf, size_t dev_bytes, void* stream,
               rabit_layer** out);

/*
 * Derive the sign planes from a full-precision weight on the device and pack them in one pass
 * (Section 4.2, steps 1-3 / Algorithm 2: B_1 = sign(W), R_1 = W - g_1 (.) B_1 (.) h_1, B_2 = sign(R_1), ...;
 * at the end of training these planes are frozen and W is discarded, end of Section 4.2):
 *   W_dev   DEVICE fp32 [M][N] row-major, 16-byte aligned, not overlapping dev_buf
 *   g, h    HOST fp16 bit patterns [K][M], [K][N] (the trained scales)
 *   dev_buf, dev_bytes, stream, out   as rabit_pack
 * The residual is kept in fp32; g*h is exact in fp32, so each update is one rounding; sign(0) = +1.
 * The resulting layer is identical to rabit_pack of the planes that this recurrence yields.
 * Streams W once (4 bytes per weight).  Asynchronous on `stream`: g and h are read before the call
 * returns, W when the kernel runs; the layer may be used by later work on the same stream (or after a
 * synchronisation on any stream).
 */
RABIT_API int rabit_derive_pack(const float* W_dev, const uint16_t* g, const uint16_t* h, int K, int M, int N,
                      void* dev_buf, size_t dev_bytes, void* stream, rabit_layer** out);

/*
 * Run the layer (Section 4.1 forward with the Eq. 2 weight):
 *   x  DEVICE fp16 [batch][N] row-major, 16-byte aligned
 *   y  DEVICE fp16 [batch][M] row-major, 16-byte aligned, must not overlap x
 * Asynchronous on `stream`; allocates nothing, never synchronises, and may be captured in
 * a CUDA graph.  The layer's device must be the current device.  One or two batch rows run the table-driven
 * GEMV (one pass over the weights: a shared-memory table of the partial sums of h*x over eight columns, indexed by the
 * packed sign byte), 3 to 16 rows the f16 tensor-core GEMV (one pass: the signs are expanded to +-h operand tiles in
 * registers, the batch is the MMA's N dimension), 17 to 32 rows two passes of it, more the tcgen05 GEMM.  Layers those two GEMVs cannot take
 * (more than 255 slices of 256 input columns) fall back to the integer tensor-core GEMV, four rows per pass, or to one
 * GEMM launch, whichever the library's cost estimate for the shape favours.  A GEMM with few output tiles runs as
 * clusters of CTAs that share a tile's contraction.  fp32 (or exact integer) accumulation, one rounding to fp16 at the end;
 * an inf or NaN in a batch row of x makes that row of y non-finite and leaves the other rows untouched.
 */
RABIT_API int rabit_linear(const rabit_layer* layer, const void* x, void* y, int batch, void* stream);

/*
 * Several layers that do not depend on one another in ONE launch (the same operation as rabit_linear,
 * Section 4.1 forward with the Eq. 2 weight, per layer): layer l maps xs[l] ([batch][N_l]) to ys[l]
 * ([batch][M_l]).  Meant for projections that read the same activations (q|k|v, gate|up: pass the same
 * pointer several times in xs) - at batch 1 a layer lasts a few microseconds, and the fixed cost of a
 * launch (dependency wait, first memory round trips, cross-CTA reduction) is paid once per group instead
 * of once per layer.  The tiles of all layers are split evenly over the CTAs as if they were one layer.
 *   layers, xs, ys   HOST arrays of n_layers entries (1 <= n_layers <= 8); the pointers inside are as for
 *                    rabit_linear; outputs must not overlap one another nor any input; all layers on one device.
 * For batch > 16, or more than 8 layers, the layers are simply run one after the other.
 * Asynchronous on `stream`, allocates nothing, may be captured in a CUDA graph.
 */
RABIT_API int rabit_linear_group(const rabit_layer* const* layers, const void* const* xs, void* const* ys,
                       int n_layers, int batch, void* stream);

/*
 * Host-buffer form of rabit_linear (same operation, Section 4.1 forward with the Eq. 2 weight)
 * for callers whose activations live in host memory:
 *   x_host  HOST fp16 [batch][N]   (pinned memory makes the copies asynchronous)
 *   y_host  HOST fp16 [batch][M]
 *   dev_stage DEVICE, 256-byte aligned, caller-owned, at least rabit_stage_bytes(layer, batch)
 * Enqueues on `stream`: copy x to the stage, the layer kernel, copy y back.  Returns without
 * synchronising; y_host is valid once the stream has reached this point.  If y_host is page-locked,
 * mapped memory (cudaHostAlloc / cudaHostRegister, 16-byte aligned) and batch <= 16, the kernel stores
 * its result there itself and no copy back is enqueued; y_host must then not be read before the stream
 * has reached this point either.
 */
RABIT_API size_t rabit_stage_bytes(const rabit_layer* layer, int batch);
RABIT_API int rabit_linear_host(const rabit_layer* layer, const void* x_host, void* y_host, int batch,
                      void* dev_stage, size_t dev_stage_bytes, void* stream);

/*
 * The batch 1..16 layer call for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a host that hands out a
 * fixed memory budget at start-up, in a real-time loop where an allocation may block or
 * synchronise the device, or in a plug-in that is given weight, input and output buffers but no
 * allocator.  rabit_linear keeps its reduction scratch inside the caller-allocated packed image;
 * a caller that received only the weights section of an image (or a read-only mapping of it) has
 * nowhere to put that scratch.  This entry point uses a fixed 4 MiB device array that is part of
 * the library instead (every GPU that loads the library holds these 4 MiB until the process exits).
 *
 *   layer, x, y, batch, stream   as rabit_linear, with 1 <= batch <= 16; the layer's device must be
 *                                the current device.
 * Limits and rules:
 *   - The scratch a layer needs is (K * ceil(M/128) + 320) * 2052 bytes, rounded up; a layer that
 *     needs more than the 4 MiB array is refused with RABIT_UNSUPPORTED_SHAPE and a message that
 *     states both sizes (K = 2 layers up to about M = 110,000 rows fit).
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.  The first call on a
 *     device looks up the device address of the array (cudaGetSymbolAddress); make that first
 *     call before any stream capture begins.
 *   - All calls, for all layers, share the one array.  Each call first puts the part of it that this
 *     layer uses back into its resting state (memsets enqueued on `stream` ahead of the kernel).  Two calls that overlap on the
 *     GPU (different streams, or one stream per thread) race on it and give wrong results: keep
 *     all uses of this entry point on one stream, or serialise them yourself.
 *   - This entry point always runs the integer tensor-core GEMV (the kernel whose scratch is large enough to matter);
 *     rabit_linear may choose another kernel for the same call, so the two agree within the parity tolerance, not bit
 *     for bit.  A bounded wait that runs out in it is recorded in a status word inside the array, which
 *     rabit_layer_status reports (for any layer of that device) and clears.
 */
RABIT_API int rabit_linear_static_scratch(const rabit_layer* layer, const void* x, void* y, int batch, void* stream);

/*
 * Health of a layer's kernels.  Every wait inside the kernels is bounded (about one second); a wait that
 * runs out makes the kernel set a status word, skip its remaining waits and return, so the context stays
 * usable but the outputs of that call are invalid.  (Only the tensor-core kernels wait for anything: the GEMV for
 * bulk copies and for the partial sums of CTAs with a lower index - it assumes that the CTAs of a grid no larger
 * than the device holds at once all become resident while it waits, which another tenant on the GPU can delay
 * beyond the limit - and the GEMM for its copy and tensor-memory barriers.  The table-driven GEMV never waits.)
 * A grouped launch records a run-out wait in the status word of every layer of the group.
 * This call synchronises `stream`, reads the layer's word and the word of the built-in scratch array of
 * rabit_linear_static_scratch, and returns RABIT_OK or RABIT_DEVICE_FAULT.  With `clear` non-zero it also puts the
 * words and the layer's exchange buffer back into their resting state; do that before the layer is used again.
 */
RABIT_API int rabit_layer_status(const rabit_layer* layer, int clear, void* stream);

/*
 * Self-test of the bounded-wait mechanism: launches one tiny kernel that waits on a barrier nobody will
 * ever signal, with a limit of `limit_us` microseconds (1..100000), and reports whether the kernel gave
 * up in time, set its status word and left the device usable.  Returns RABIT_OK if so.  `status_dev`
 * is a DEVICE word owned by the caller (4 bytes, 4-byte aligned); it holds 1 afterwards.
 */
RABIT_API int rabit_selftest_bounded_wait(unsigned int* status_dev, int limit_us, void* stream);

/*
 * Test aid (no counterpart in the paper; host only, no GPU needed): how the f16 tensor-core GEMV of rabit_linear
 * (batch 3..16) would split a K-path layer of M x N at `batch` rows over `sms` SMs.  The layer is ceil(M/128) row tiles x
 * ceil(N/256) slices; in that order the (row tile, slice) pairs are cut into contiguous parts, two per SM (one per group
 * of eight warps).  bound_out (HOST, max_out ints) receives the starts of the parts followed by the number of pairs:
 * 2 * grid + 1 ascending values; a part may be empty.  Returns the number of CTAs (grid >= 1), or RABIT_INVALID_ARG.
 */
RABIT_API int rabit_selftest_f16_plan(int K, int M, int N, int batch, int sms, int* bound_out, int max_out);

/*
 * Measurement aid (no counterpart in the paper): one kernel that reads `bytes` bytes of device memory once with
 * 128-bit streaming loads and keeps nothing.  Timed by the caller with CUDA events over a buffer much larger than L2
 * it gives the read-only HBM bandwidth this GPU delivers to plain loads, the natural ceiling of the decode GEMV.
 *   src_dev   DEVICE, 16-byte aligned, `bytes` readable bytes (a multiple of 16 is read)
 *   sink_dev  DEVICE word or NULL; written only if the data fold to one particular value (keeps the loads alive)
 * Asynchronous on `stream`.
 */
RABIT_API int rabit_selftest_stream_read(const void* src_dev, size_t bytes, unsigned int* sink_dev, void* stream);

/*
 * Host-buffer form of rabit_linear_group: inputs and outputs live in HOST memory (pinned memory makes the
 * copies asynchronous).  An input pointer that occurs several times in xs_host is copied to the device once.
 *   dev_stage  DEVICE, 256-byte aligned, at least rabit_group_stage_bytes(layers, n_layers, batch)
 * Enqueues the input copies, one grouped launch and the output copies on `stream`; returns without
 * synchronising.  Outputs in page-locked, mapped host memory are written by the kernel itself when
 * batch <= 16 (see rabit_linear_host).
 */
RABIT_API size_t rabit_group_stage_bytes(const rabit_layer* const* layers, int n_layers, int batch);
RABIT_API int rabit_linear_group_host(const rabit_layer* const* layers, const void* const* xs_host, void* const* ys_host,
                            int n_layers, int batch, void* dev_stage, size_t dev_stage_bytes, void* stream);

/*
 * Phase tracing of the decode kernels, for profiling (no counterpart in the paper).  Only a library built with
 * -DRABIT_TRACE (python paper_2602_05367_b200/build.py --trace -> librabit_trace.so) records anything; in the
 * ordinary build rabit_trace_begin returns RABIT_UNSUPPORTED_SHAPE and rabit_trace_launches 0.
 *   rabit_trace_begin(dev_buf, bytes)  DEVICE buffer, 8-byte aligned, caller-owned; every later launch of the
 *       table-driven GEMV (also launches captured into a CUDA graph from now on) gets the next record of
 *       64 x uint64 per CTA in it until it is full; dev_buf = NULL stops tracing.  Not thread-safe.
 *   rabit_trace_launches(ctas_out, max)  number of records handed out since rabit_trace_begin; ctas_out[i]
 *       receives the CTA count of record i (records follow one another in the buffer).
 * Stamps of a CTA, taken by one thread: 0 kernel entry in nanoseconds of the GPU's global timer (coarse: it advances
 * in steps of a fraction of a microsecond); 1..7 SM clock cycles since that entry: 1 dependency wait over, 2 x and h
 * of the first table have arrived, 3 first table built, 4 first weights in registers, 5 last look-up done and last
 * atomic issued, 6 last atomic answered and y stored, 7 look-ups of the thread's first block answered; 8 + 5*i + {0..4}
 * for the thread's block i < 11: loop top, weights arrived, look-ups answered, previous atomic settled, output scales arrived.
 */
RABIT_API int rabit_trace_begin(void* dev_buf, size_t bytes);
RABIT_API int rabit_trace_launches(int* ctas_out, int max_launches);

/* Copy the packed image back from the device and unpack it (round-trip check).  Synchronises. */
RABIT_API int rabit_unpack(const rabit_layer* layer, uint32_t* planes_out, uint16_t* g_out, uint16_t* h_out,
                 void* stream);

/* Shape queries on a descriptor; return -1 on a NULL layer. */
RABIT_API int rabit_layer_K(const rabit_layer* layer);
RABIT_API int rabit_layer_M(const rabit_layer* layer);
RABIT_API int rabit_layer_N(const rabit_layer* layer);

/*
 * Choose the kernel family for subsequent rabit_linear calls of this layer:
 *   0 = automatic (default), 1 = plain sign-select kernel, 2 = integer tensor-core GEMV,
 *   3 = tcgen05 GEMM with one exact +-h_k operand tile and accumulator per path,
 *   4 = tcgen05 GEMM on the dequantised weight tile sum_k +-g_k h_k rounded to fp16 (Eq. 2 formed per tile; one
 *       contraction of length N instead of K of them; never chosen automatically: it rounds every weight to fp16),
 *   5 = table-driven GEMV (passes of up to two batch rows; N up to 65280),
 *   6 = f16 tensor-core GEMV (passes of up to 16 batch rows; N up to 65280).
 * Returns RABIT_INVALID_ARG for a variant that cannot run the layer.
 * Meant for A/B timing and profiling; results are within tolerance for every variant.
 */
RABIT_API int rabit_set_variant(rabit_layer* layer, int variant);

/* Release the descriptor only; the caller's device buffer is untouched. NULL is accepted. */
RABIT_API int rabit_free(rabit_layer* layer);

/* Thread-local, never NULL; empty string if the last call on this thread succeeded. */
RABIT_API const char* rabit_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* RABIT_H_ */
