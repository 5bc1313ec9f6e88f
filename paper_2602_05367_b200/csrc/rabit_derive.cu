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

#include <cstring>

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
// kernel above has just written.  One CTA per (row tile, slice of 256 columns): its eight warps first copy the slice's
// 8 K sign tiles into shared memory (coalesced, every tile read once), then each warp gathers parts of 1 KB
// (path k, row block of 32 rows; lane = row).  A byte of eight consecutive columns comes from two tile words (four
// columns each, the row's bit p in every byte).  Columns beyond N stay zero.  The CTAs also share out two fills that put
// the layer's reduction scratch into its resting state: `n_ones` 16-byte units of all-ones words, `n_zero` of zeros; and
// the first CTA writes the image's header, which arrives as a kernel parameter (one host-to-device copy fewer).
struct HeaderWords {
    uint4 v[RABIT_HEADER_BYTES / 16];
};
__global__ void __launch_bounds__(kWarps * 32)
rabit_tiles_to_lut_kernel(RabitGeom G, const uint4* __restrict__ tiles, uint4* __restrict__ lut,
                          uint4* __restrict__ ones, size_t n_ones, uint4* __restrict__ zero, size_t n_zero,
                          const __grid_constant__ HeaderWords header, uint4* __restrict__ header_dst) {
    __shared__ uint4 staged[RABIT_MAX_K][kWarps][32];     // [path][column tile of the slice][lane of the tile]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && header_dst != nullptr && threadIdx.x < RABIT_HEADER_BYTES / 16) header_dst[threadIdx.x] = header.v[threadIdx.x];
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_ones; i += (size_t)gridDim.x * blockDim.x)
        ones[i] = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_zero; i += (size_t)gridDim.x * blockDim.x)
        zero[i] = make_uint4(0u, 0u, 0u, 0u);
    const int rt = blockIdx.x / G.n_cs, cs = blockIdx.x - rt * G.n_cs;
    const int ct = cs * kWarps + warp;
    for (int k = 0; k < G.K; ++k)
        staged[k][warp][lane] = ct < G.n_ct ? tiles[rabit_tile_pos(G, rt, k, ct) * 32 + lane] : make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    for (int part = warp; part < 4 * G.K; part += kWarps) {
        const int k = part % G.K, rbl = part / G.K;
        const int rl = rbl * RABIT_LUT_ROWS + lane;                     // row inside the tile
        const int p = rl >> 4, gq = rl & 7, alo = (rl >> 3) & 1;
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) o[j] = 0u;
#pragma unroll
        for (int sidx = 0; sidx < 32; ++sidx) {
            const int group = (sidx + lane) & 31;                       // byte group of the slice this lane stores at step sidx
            const int ctl = group >> 2, ah = (group >> 1) & 1, tq0 = (group & 1) * 2;
            const uint32_t* words = reinterpret_cast<const uint32_t*>(&staged[k][ctl][4 * gq + tq0]);
            const uint32_t w0 = words[alo | (ah << 1)], w1 = words[4 + (alo | (ah << 1))];
            const uint32_t n0 = ((((w0 >> p) & 0x01010101u) * 0x01020408u) >> 24) & 0xFu;  // bit c <- byte c
            const uint32_t n1 = ((((w1 >> p) & 0x01010101u) * 0x01020408u) >> 24) & 0xFu;
            o[sidx >> 2] |= (n0 | (n1 << 4)) << (8 * (sidx & 3));
        }
        const int rb = rt * (RABIT_TILE_ROWS / RABIT_LUT_ROWS) + rbl;
        uint4* dst = lut + (((size_t)cs * G.n_rb + rb) * G.K + k) * (RABIT_LUT_PART_BYTES / 16);
        dst[lane] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[32 + lane] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

}  // namespace

cudaError_t rabit_launch_tiles_to_lut(const RabitGeom& G, const uint4* d_tiles, unsigned char* d_lut, void* d_ones, size_t ones_bytes,
                                      void* d_zero, size_t zero_bytes, const RabitHeader* header, void* d_header, cudaStream_t stream) {
    static_assert(sizeof(RabitHeader) == RABIT_HEADER_BYTES, "the header travels as a kernel parameter");
    HeaderWords hw;
    std::memset(&hw, 0, sizeof(hw));
    if (header) std::memcpy(&hw, header, sizeof(RabitHeader));
    if ((ones_bytes | zero_bytes | (size_t)(uintptr_t)d_ones | (size_t)(uintptr_t)d_zero) & 15u) return cudaErrorInvalidValue;
    static_assert(kWarps * RABIT_TILE_COLS == RABIT_LUT_COLS, "one warp per column tile of a slice");
    const long long blocks = (long long)G.n_rt * G.n_cs;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    rabit_tiles_to_lut_kernel<<<(unsigned int)blocks, kWarps * 32, 0, stream>>>(G, d_tiles, reinterpret_cast<uint4*>(d_lut),
                                                                               reinterpret_cast<uint4*>(d_ones), ones_bytes / 16,
                                                                               reinterpret_cast<uint4*>(d_zero), zero_bytes / 16, hw,
                                                                               header ? reinterpret_cast<uint4*>(d_header) : nullptr);
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
