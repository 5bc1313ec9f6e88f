// Plain sign-select kernel: the simplest correct evaluation of the layer on the packed layout.
//
//   y[b][i] = sum_k g_k[i] * sum_j B_k[i][j] * (h_k[j] * x[b][j])        (Section 4.1, Eq. 2)
//
// One CTA owns one 128-row tile and up to kBT batch rows; its eight warps take the column
// tiles round-robin.  Each lane decodes the 16 bytes it loaded (16 rows x 8 columns), adds
// +-t in fp32, the four lanes that share rows are summed with shuffles, the g_k epilogue
// accumulates the paths, and the warps are summed in shared memory in a fixed order.  It
// exists as the any-shape, any-batch variant and as the on-device cross-check of the fast
// kernels; it is not tuned (about three ALU instructions per weight).
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kBT = 2;            // batch rows per CTA
constexpr int kWarps = 8;

__global__ void __launch_bounds__(kWarps * 32)
rabit_plain_kernel(RabitGeom G, const uint4* __restrict__ bits, const __half* __restrict__ g,
                   const __half* __restrict__ h, const __half* __restrict__ x, __half* __restrict__ y, int batch) {
    __shared__ float red[kWarps][kBT][RABIT_TILE_ROWS];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int rt = blockIdx.x;
    const int b0 = blockIdx.y * kBT;
    const int gq = lane >> 2, tq = lane & 3;

    float yacc[kBT][16];          // index 2*p + alo  <->  row 16*p + gq + 8*alo
#pragma unroll
    for (int b = 0; b < kBT; ++b)
#pragma unroll
        for (int s = 0; s < 16; ++s) yacc[b][s] = 0.f;

    for (int k = 0; k < G.K; ++k) {
        float acc[kBT][16];
#pragma unroll
        for (int b = 0; b < kBT; ++b)
#pragma unroll
            for (int s = 0; s < 16; ++s) acc[b][s] = 0.f;

        for (int ct = w; ct < G.n_ct; ct += kWarps) {
            const uint4 wv = bits[rabit_tile_pos(G, rt, k, ct) * 32 + lane];
            const uint32_t wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
            for (int ah = 0; ah < 2; ++ah)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int col = ct * RABIT_TILE_COLS + 16 * ah + 4 * tq + c;
                    const float hv = __half2float(h[(size_t)k * G.N + col]);
#pragma unroll
                    for (int b = 0; b < kBT; ++b) {
                        if (b0 + b >= batch) continue;
                        const float tv = hv * __half2float(x[(size_t)(b0 + b) * G.N + col]);
#pragma unroll
                        for (int alo = 0; alo < 2; ++alo) {
                            const uint32_t byte = (wa[alo | (ah << 1)] >> (8 * c)) & 0xFFu;
#pragma unroll
                            for (int p = 0; p < 8; ++p) acc[b][2 * p + alo] += ((byte >> p) & 1u) ? -tv : tv;
                        }
                    }
                }
        }
#pragma unroll
        for (int b = 0; b < kBT; ++b)
#pragma unroll
            for (int s = 0; s < 16; ++s) {
                float v = acc[b][s];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                const int row = rt * RABIT_TILE_ROWS + 16 * (s >> 1) + gq + 8 * (s & 1);
                yacc[b][s] += __half2float(g[(size_t)k * G.Mp + row]) * v;
            }
    }
    if (tq == 0) {
#pragma unroll
        for (int b = 0; b < kBT; ++b)
#pragma unroll
            for (int s = 0; s < 16; ++s) red[w][b][16 * (s >> 1) + gq + 8 * (s & 1)] = yacc[b][s];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBT * RABIT_TILE_ROWS; i += kWarps * 32) {
        const int b = i / RABIT_TILE_ROWS, r = i % RABIT_TILE_ROWS;
        const int row = rt * RABIT_TILE_ROWS + r;
        if (b0 + b >= batch || row >= G.M) continue;
        float sum = 0.f;
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) sum += red[ww][b][r];
        y[(size_t)(b0 + b) * G.M + row] = __float2half_rn(sum);
    }
}

}  // namespace

cudaError_t rabit_launch_plain(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    dim3 grid(L.geom.n_rt, (batch + kBT - 1) / kBT);
    rabit_plain_kernel<<<grid, kWarps * 32, 0, stream>>>(L.geom, L.d_bits, (const __half*)L.d_g, (const __half*)L.d_h,
                                                         (const __half*)x, (__half*)y, batch);
    return cudaGetLastError();
}
