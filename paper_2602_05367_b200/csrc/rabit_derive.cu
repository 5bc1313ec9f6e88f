// Derivation of the sign planes from a full-precision weight, fused with packing.
//
//   R_0 = W,   B_k = sign(R_{k-1}),   R_k = R_{k-1} - g_k (.) B_k (.) h_k        (Section 4.2, steps 1-3; Algorithm 2)
//
// This is the step just before the inference hot path: at the end of training the sign matrices are
// derived once from the shared full-precision weight and frozen (end of Section 4.2).  Every weight
// entry is independent, so the kernel streams W once (4 bytes per weight in, K bits out) and writes the
// packed tiles of the device layout directly.  Arithmetic is fp32: the product g*h of two fp16 values is
// exact in fp32, so each residual update is one fp32 rounding; sign(0) = +1 (bit 0).
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kWarps = 8;

// One warp per (row tile, column tile); lane (gq, tq) produces the 16 bytes it owns in every path's tile.
__global__ void __launch_bounds__(kWarps * 32)
rabit_derive_kernel(RabitGeom G, const float* __restrict__ W, const __half* __restrict__ g, const __half* __restrict__ h,
                    uint4* __restrict__ tiles) {
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (wid >= (long long)G.n_rt * G.n_ct) return;
    const int rt = (int)(wid / G.n_ct), ct = (int)(wid % G.n_ct);
    const int gq = lane >> 2, tq = lane & 3;

    float hv[RABIT_MAX_K][2][4];                          // input scales of this lane's 8 columns
#pragma unroll
    for (int k = 0; k < RABIT_MAX_K; ++k)
#pragma unroll
        for (int ah = 0; ah < 2; ++ah) {
            uint2 raw = make_uint2(0u, 0u);
            if (k < G.K) raw = *reinterpret_cast<const uint2*>(h + (size_t)k * G.N + ct * RABIT_TILE_COLS + 16 * ah + 4 * tq);
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
            hv[k][ah][0] = a.x; hv[k][ah][1] = a.y; hv[k][ah][2] = b.x; hv[k][ah][3] = b.y;
        }
    uint32_t out[RABIT_MAX_K][4];
#pragma unroll
    for (int k = 0; k < RABIT_MAX_K; ++k)
#pragma unroll
        for (int a = 0; a < 4; ++a) out[k][a] = 0u;

#pragma unroll
    for (int alo = 0; alo < 2; ++alo) {
        float4 w[8][2];                                   // 16 loads of 16 bytes in flight
        float gv[RABIT_MAX_K][8];
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const int row = rt * RABIT_TILE_ROWS + 16 * p + gq + 8 * alo;
#pragma unroll
            for (int ah = 0; ah < 2; ++ah) {
                w[p][ah] = make_float4(0.f, 0.f, 0.f, 0.f);   // padded rows: +1 signs
                if (row < G.M) w[p][ah] = __ldcs(reinterpret_cast<const float4*>(W + (size_t)row * G.N + ct * RABIT_TILE_COLS + 16 * ah + 4 * tq));
            }
#pragma unroll
            for (int k = 0; k < RABIT_MAX_K; ++k) gv[k][p] = (k < G.K && row < G.M) ? __half2float(g[(size_t)k * G.Mp + row]) : 0.f;
        }
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int ah = 0; ah < 2; ++ah) {
                float r[4] = {w[p][ah].x, w[p][ah].y, w[p][ah].z, w[p][ah].w};
#pragma unroll
                for (int k = 0; k < RABIT_MAX_K; ++k) {
                    if (k >= G.K) break;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const bool neg = r[c] < 0.f;
                        out[k][alo | (ah << 1)] |= (neg ? 1u : 0u) << (8 * c + p);
                        const float gb = neg ? -gv[k][p] : gv[k][p];          // g * B, exact
                        r[c] = r[c] - gb * hv[k][ah][c];                      // the product is exact in fp32: one rounding
                    }
                }
            }
    }
#pragma unroll
    for (int k = 0; k < RABIT_MAX_K; ++k) {
        if (k >= G.K) break;
        tiles[rabit_tile_pos(G, rt, k, ct) * 32 + lane] = make_uint4(out[k][0], out[k][1], out[k][2], out[k][3]);
    }
}

// Second arrangement of the same signs: the look-up blocks (rabit_layout.h), gathered from the tiles that the
// kernel above has just written.  One warp per (path, row block of 32 rows, slice of 256 columns) = one 1 KB part;
// lane = row.  A byte of eight consecutive columns comes from two tile words (four columns each, the row's bit p
// in every byte).  Columns beyond N stay zero.
__global__ void __launch_bounds__(kWarps * 32)
rabit_tiles_to_lut_kernel(RabitGeom G, const uint32_t* __restrict__ tiles, uint4* __restrict__ lut) {
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    const long long parts = (long long)G.n_cs * G.n_rb * G.K;
    if (wid >= parts) return;
    const int k = (int)(wid % G.K);
    const long long pos = wid / G.K;
    const int rb = (int)(pos % G.n_rb), cs = (int)(pos / G.n_rb);
    const int row = rb * RABIT_LUT_ROWS + lane;
    const int rt = row >> 7, rl = row & 127, p = rl >> 4, gq = rl & 7, alo = (rl >> 3) & 1;
    uint32_t out[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) out[j] = 0u;
#pragma unroll 4
    for (int s = 0; s < 32; ++s) {
        const int group = (s + lane) & 31;                              // byte group of the slice this lane stores at step s
        const int col = cs * RABIT_LUT_COLS + 8 * group;
        uint32_t byte = 0u;
        if (col < G.N) {
            const int ct = col >> 5, cl = col & 31, ah = cl >> 4, tq0 = (cl & 15) >> 2;     // tq0 is 0 or 2
            const uint32_t* tile = tiles + rabit_tile_pos(G, rt, k, ct) * (RABIT_TILE_BYTES / 4);
            const int a = alo | (ah << 1);
            const uint32_t w0 = tile[(4 * gq + tq0) * 4 + a], w1 = tile[(4 * gq + tq0 + 1) * 4 + a];
            const uint32_t n0 = ((((w0 >> p) & 0x01010101u) * 0x01020408u) >> 24) & 0xFu;  // bit c <- byte c
            const uint32_t n1 = ((((w1 >> p) & 0x01010101u) * 0x01020408u) >> 24) & 0xFu;
            byte = n0 | (n1 << 4);
        }
        out[s >> 2] |= byte << (8 * (s & 3));
    }
    uint4* dst = lut + (size_t)wid * (RABIT_LUT_PART_BYTES / 16);
    dst[lane] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[32 + lane] = make_uint4(out[4], out[5], out[6], out[7]);
}

}  // namespace

cudaError_t rabit_launch_tiles_to_lut(const RabitGeom& G, const uint4* d_tiles, unsigned char* d_lut, cudaStream_t stream) {
    const long long warps = (long long)G.n_cs * G.n_rb * G.K;
    const long long blocks = (warps + kWarps - 1) / kWarps;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    rabit_tiles_to_lut_kernel<<<(unsigned int)blocks, kWarps * 32, 0, stream>>>(G, reinterpret_cast<const uint32_t*>(d_tiles),
                                                                               reinterpret_cast<uint4*>(d_lut));
    return cudaGetLastError();
}

cudaError_t rabit_launch_derive(const RabitGeom& G, const float* W, const uint16_t* d_g, const uint16_t* d_h, uint4* d_tiles,
                                cudaStream_t stream) {
    const long long warps = (long long)G.n_rt * G.n_ct;
    const long long blocks = (warps + kWarps - 1) / kWarps;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    rabit_derive_kernel<<<(unsigned int)blocks, kWarps * 32, 0, stream>>>(G, W, (const __half*)d_g, (const __half*)d_h, d_tiles);
    return cudaGetLastError();
}
