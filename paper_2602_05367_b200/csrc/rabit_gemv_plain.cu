// Plain sign-select kernel: the simplest correct evaluation of the layer on the packed layout.
//
//   y[b][i] = sum_k g_k[i] * sum_j B_k[i][j] * (h_k[j] * x[b][j])        (Section 4.1, Eq. 2)
//
// One warp owns one 32-row tile and walks every column group of every path; each lane
// decodes the 16 bytes it loaded (4 rows x 32 columns), adds +-t in fp32, the four lanes of
// a quad are summed with shuffles, and the g_k epilogue accumulates the paths.  It exists
// as the any-shape, any-batch variant and as the on-device cross-check of the fast kernels;
// it is not tuned (about three ALU instructions per weight).
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kBT = 4;            // batch rows per pass
constexpr int kWarps = 8;

__global__ void __launch_bounds__(kWarps * 32)
rabit_plain_kernel(RabitGeom G, const uint4* __restrict__ bits, const __half* __restrict__ g,
                   const __half* __restrict__ h, const __half* __restrict__ x, __half* __restrict__ y, int batch) {
    const int lane = threadIdx.x & 31;
    const int rt = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (rt >= G.n_rt) return;
    const int b0 = blockIdx.y * kBT;
    const int gq = lane >> 2, tq = lane & 3;

    float yacc[kBT][4];
#pragma unroll
    for (int b = 0; b < kBT; ++b)
#pragma unroll
        for (int s = 0; s < 4; ++s) yacc[b][s] = 0.f;

    for (int k = 0; k < G.K; ++k) {
        float acc[kBT][4];
#pragma unroll
        for (int b = 0; b < kBT; ++b)
#pragma unroll
            for (int s = 0; s < 4; ++s) acc[b][s] = 0.f;

        for (int s = 0; s < G.n_slices; ++s) {
            const int ncg = rabit_slice_ncg(G, s);
            for (int q = 0; q < ncg; ++q) {
                const int cg = s * G.slice_cg + q;
                const uint4 w = bits[rabit_tile_index(G, s, rt, q, k) * 32 + lane];
                const uint32_t wa[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int cs = 0; cs < 4; ++cs)
#pragma unroll
                    for (int ah = 0; ah < 2; ++ah)
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int col = cg * 128 + cs * 32 + ah * 16 + tq * 4 + c;
                            if (col >= G.N) continue;
                            const float hv = __half2float(h[(size_t)k * G.Np + col]);
#pragma unroll
                            for (int b = 0; b < kBT; ++b) {
                                if (b0 + b >= batch) continue;
                                const float tv = hv * __half2float(x[(size_t)(b0 + b) * G.N + col]);
#pragma unroll
                                for (int alo = 0; alo < 2; ++alo) {
                                    const uint32_t byte = (wa[alo | (ah << 1)] >> (8 * c)) & 0xFFu;
#pragma unroll
                                    for (int rg = 0; rg < 2; ++rg) {
                                        const bool neg = (byte >> (rg + 2 * cs)) & 1u;
                                        acc[b][alo * 2 + rg] += neg ? -tv : tv;
                                    }
                                }
                            }
                        }
            }
        }
#pragma unroll
        for (int b = 0; b < kBT; ++b)
#pragma unroll
            for (int sl = 0; sl < 4; ++sl) {
                float v = acc[b][sl];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                const int row = rt * 32 + 2 * (gq + 8 * (sl >> 1)) + (sl & 1);
                yacc[b][sl] += __half2float(g[(size_t)k * G.Mp + row]) * v;
            }
    }
    if (tq == 0) {
#pragma unroll
        for (int b = 0; b < kBT; ++b) {
            if (b0 + b >= batch) continue;
#pragma unroll
            for (int sl = 0; sl < 4; ++sl) {
                const int row = rt * 32 + 2 * (gq + 8 * (sl >> 1)) + (sl & 1);
                if (row < G.M) y[(size_t)(b0 + b) * G.M + row] = __float2half_rn(yacc[b][sl]);
            }
        }
    }
}

}  // namespace

cudaError_t rabit_launch_plain(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    dim3 grid((L.geom.n_rt + kWarps - 1) / kWarps, (batch + kBT - 1) / kBT);
    rabit_plain_kernel<<<grid, kWarps * 32, 0, stream>>>(L.geom, L.d_bits, (const __half*)L.d_g, (const __half*)L.d_h,
                                                         (const __half*)x, (__half*)y, batch);
    return cudaGetLastError();
}
