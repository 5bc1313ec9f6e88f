// Decode GEMV on the integer tensor-core path (batch 1..2).
//
//   y[b][i] = sum_k g_k[i] * sum_j B_k[i][j] * t_k[b][j],   t_k[b][j] = h_k[j] * x[b][j]     (Section 4.1, Eq. 2)
//
// At one bit per weight the sign-select arithmetic, not HBM, is the limit on B200: logic
// instructions issue at 64 lanes/clk/SM while the memory system delivers ~190 weight bits
// /clk/SM.  This kernel therefore spends one logic instruction per FOUR weights: a packed
// 32-bit word masked with 0x01010101 << p is already a valid u8 MMA operand with entries
// {0, 2^p} (see rabit_layout.h for how the bits of a byte are assigned to 2 rows x 4 column
// sets), and mma.sync.m16n8k32.u8.s8 does the additions.  The B operand holds t in exact
// fixed point: per column slice, T = round(t * 2^e) with |T| <= 2^24, shifted left by
// 2*(3 - column set) so that every product carries the same weight, and split into four
// balanced base-256 digits that occupy four of the eight MMA columns (a second batch row
// takes the other four).  With b = sign bit, sum_j B t = sum_j t - 2 sum_j b t; the int32
// accumulators give sum_j b T exactly, and the epilogue applies 2^-e, g_k and the path sum
// in fp32.  The only roundings are T (<= 2^-24 of the slice's largest |t| per term), the
// fp32 epilogue and the final fp16 store.
//
// Work split: an item is (column slice, 32-row tile); CTAs own contiguous item ranges, the
// warps of a CTA take items round-robin, so a CTA streams one contiguous byte range and
// prepares digits only for the slice(s) it touches.  Every warp prefetches its own tiles
// with cp.async into a private shared-memory ring (each lane reads back exactly the 16
// bytes it copied, so no barrier is involved).  Slices are reduced through a per-layer fp32
// partial buffer: the warp whose arrival completes a row tile sums the partials in slice
// order (deterministic) and stores fp16.
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kDepth = 12;               // tiles in flight per warp (6 KB)
constexpr int kMaxSliceCg = 8;

struct GemvParams {
    RabitGeom G;
    const uint4* bits;
    const __half* g;
    const __half* h;
    const __half* x;
    __half* y;
    float* partial;          // [batch][n_slices][Mp]
    unsigned int* counters;  // [n_rt]
    int n_items;             // n_slices * n_rt
};

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gptr) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Walks the tiles of one warp in consumption order: segments (one per slice touched by the
// CTA range [i0,i1)), inside a segment the items seg_start + w, + kWarps, ..., inside an item
// its ncg*K contiguous tiles.
struct TileWalker {
    const RabitGeom* G;
    const uint4* bits;
    int i1, w, lane;
    int seg_end, item, tiles_left;
    const uint4* p;
    bool done;

    __device__ void start_segment(int seg_start) {
        while (true) {
            if (seg_start >= i1) { done = true; return; }
            const int s = seg_start / G->n_rt;
            seg_end = min(i1, (s + 1) * G->n_rt);
            item = seg_start + w;
            if (item < seg_end) { open_item(); return; }
            seg_start = seg_end;
        }
    }
    __device__ void open_item() {
        const int s = item / G->n_rt, rt = item - s * G->n_rt;
        tiles_left = rabit_slice_ncg(*G, s) * G->K;
        p = bits + rabit_tile_index(*G, s, rt, 0, 0) * 32 + lane;
    }
    __device__ void init(const RabitGeom* g_, const uint4* bits_, int i0, int i1_, int w_, int lane_) {
        G = g_; bits = bits_; i1 = i1_; w = w_; lane = lane_; done = false;
        start_segment(i0);
    }
    // pointer of the next tile (this lane's 16 bytes) or nullptr when exhausted
    __device__ const uint4* next() {
        if (done) return nullptr;
        const uint4* r = p;
        p += 32;
        if (--tiles_left == 0) {
            item += kWarps;
            if (item < seg_end) open_item();
            else start_segment(seg_end);
        }
        return r;
    }
};

template <int NB>
__global__ void __launch_bounds__(kThreads, 1)
rabit_gemv_mma_kernel(const GemvParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const RabitGeom& G = P.G;
    constexpr int NCOL = 4 * NB;                       // MMA columns in use (digits x batch rows)
    // shared memory carve-up
    uint4* ring = reinterpret_cast<uint4*>(smem_raw);                                  // [kWarps][kDepth][32] uint4
    uint32_t* table = reinterpret_cast<uint32_t*>(smem_raw + kWarps * kDepth * 512);   // [K*ncg*4][NCOL][4][2] words
    __shared__ int s_max[NB][RABIT_MAX_K];
    __shared__ long long s_sumT[NB][RABIT_MAX_K];
    __shared__ float s_sumTf[NB][RABIT_MAX_K];
    __shared__ float s_inv[NB][RABIT_MAX_K];            // 1 / sigma

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int gq = lane >> 2, tq = lane & 3;
    const int i0 = (int)((long long)blockIdx.x * P.n_items / gridDim.x);
    const int i1 = (int)((long long)(blockIdx.x + 1) * P.n_items / gridDim.x);
    if (i0 >= i1) return;

    // ---- start streaming this warp's weights before anything else
    uint4* my_ring = ring + (size_t)w * kDepth * 32 + lane;
    const uint32_t my_ring_s = (uint32_t)__cvta_generic_to_shared(my_ring);
    TileWalker pf;
    pf.init(&G, P.bits, i0, i1, w, lane);
#pragma unroll 1
    for (int d = 0; d < kDepth; ++d) {
        const uint4* src = pf.next();
        if (src) cp_async16(my_ring_s + d * 512, src);
        cp_async_commit();
    }
    int slot = 0;

    int seg_start = i0;
    while (seg_start < i1) {
        const int s = seg_start / G.n_rt;
        const int seg_end = min(i1, (s + 1) * G.n_rt);
        const int ncg = rabit_slice_ncg(G, s);
        const int col0 = s * G.slice_cg * 128;
        const int groups = ncg * 32;                   // groups of 4 consecutive columns
        const int units = NB * G.K * groups;

        // ---- fixed-point digits of t = h*x for this slice -------------------------------
        if (tid < NB * RABIT_MAX_K) { (&s_max[0][0])[tid] = 0; (&s_sumT[0][0])[tid] = 0; }
        __syncthreads();
        for (int u = tid; u < units; u += kThreads) {      // pass 1: largest |t| per (batch row, path)
            const int grp = u % groups, bk = u / groups, k = bk % G.K, b = bk / G.K;
            const int col = col0 + grp * 4;
            float m = 0.f;
            if (col < G.N) {                               // N % 4 == 0, so a group is inside or outside
                const uint2 hx = *reinterpret_cast<const uint2*>(P.h + (size_t)k * G.Np + col);
                const uint2 xx = *reinterpret_cast<const uint2*>(P.x + (size_t)b * G.N + col);
                const float2 h01 = __half22float2(*reinterpret_cast<const __half2*>(&hx.x));
                const float2 h23 = __half22float2(*reinterpret_cast<const __half2*>(&hx.y));
                const float2 x01 = __half22float2(*reinterpret_cast<const __half2*>(&xx.x));
                const float2 x23 = __half22float2(*reinterpret_cast<const __half2*>(&xx.y));
                m = fmaxf(fmaxf(fabsf(h01.x * x01.x), fabsf(h01.y * x01.y)), fmaxf(fabsf(h23.x * x23.x), fabsf(h23.y * x23.y)));
            }
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            if (lane == 0) atomicMax(&s_max[b][k], __float_as_int(m));     // non-negative floats order as ints
        }
        __syncthreads();
        for (int u = tid; u < units; u += kThreads) {      // pass 2: T, shifted digits, fragment order
            const int grp = u % groups, bk = u / groups, k = bk % G.K, b = bk / G.K;
            const int col = col0 + grp * 4;
            const int mbits = s_max[b][k];
            // sigma = 2^(23 - floor(log2 max)) so that max * sigma lies in [2^23, 2^24); sigma = 1 if max == 0
            const int em = (mbits >> 23) & 0xFF;
            const float sigma = mbits == 0 ? 1.f : __int_as_float((127 + 23 + 127 - em) << 23);
            int T[4] = {0, 0, 0, 0};
            if (col < G.N) {
                const uint2 hx = *reinterpret_cast<const uint2*>(P.h + (size_t)k * G.Np + col);
                const uint2 xx = *reinterpret_cast<const uint2*>(P.x + (size_t)b * G.N + col);
                const float2 h01 = __half22float2(*reinterpret_cast<const __half2*>(&hx.x));
                const float2 h23 = __half22float2(*reinterpret_cast<const __half2*>(&hx.y));
                const float2 x01 = __half22float2(*reinterpret_cast<const __half2*>(&xx.x));
                const float2 x23 = __half22float2(*reinterpret_cast<const __half2*>(&xx.y));
                T[0] = __float2int_rn(h01.x * x01.x * sigma);
                T[1] = __float2int_rn(h01.y * x01.y * sigma);
                T[2] = __float2int_rn(h23.x * x23.x * sigma);
                T[3] = __float2int_rn(h23.y * x23.y * sigma);
            }
            long long tsum = (long long)T[0] + T[1] + T[2] + T[3];
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, o);
            if (lane == 0) atomicAdd(reinterpret_cast<unsigned long long*>(&s_sumT[b][k]), (unsigned long long)tsum);
            const int cl = grp * 4;                          // column inside the slice
            const int q = cl >> 7, cs = (cl >> 5) & 3, ah = (cl >> 4) & 1, tqc = (cl >> 2) & 3;
            const int sh = 2 * (3 - cs);
            uint32_t X[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) X[c] = (((uint32_t)T[c] << sh) + 0x80808080u) ^ 0x80808080u;   // bytes = balanced digits
            const uint32_t t0 = __byte_perm(X[0], X[1], 0x5140), t1 = __byte_perm(X[2], X[3], 0x5140);
            const uint32_t t2 = __byte_perm(X[0], X[1], 0x7362), t3 = __byte_perm(X[2], X[3], 0x7362);
            uint32_t dig[4];
            dig[0] = __byte_perm(t0, t1, 0x5410); dig[1] = __byte_perm(t0, t1, 0x7632);
            dig[2] = __byte_perm(t2, t3, 0x5410); dig[3] = __byte_perm(t2, t3, 0x7632);
            uint32_t* dst = table + ((size_t)((k * ncg + q) * 4 + cs) * NCOL + 4 * b) * 8 + tqc * 2 + ah;
#pragma unroll
            for (int n = 0; n < 4; ++n) dst[n * 8] = dig[n];
        }
        __syncthreads();
        if (tid < NB * G.K) {
            const int b = tid / G.K, k = tid % G.K;
            const int mbits = s_max[b][k];
            const int em = (mbits >> 23) & 0xFF;
            s_inv[b][k] = mbits == 0 ? 1.f : __int_as_float((127 - 23 - 127 + em) << 23);
            s_sumTf[b][k] = (float)s_sumT[b][k];
        }
        __syncthreads();

        // ---- this warp's items of the segment ----------------------------------------------
        for (int item = seg_start + w; item < seg_end; item += kWarps) {
            const int rt = item - s * G.n_rt;
            float yv[2][2] = {{0.f, 0.f}, {0.f, 0.f}};      // [row half][row parity], even-tq lanes only
            int acc[RABIT_MAX_K][2][4];
#pragma unroll
            for (int k = 0; k < RABIT_MAX_K; ++k)
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[k][r][c] = 0;

            for (int q = 0; q < ncg; ++q) {
#pragma unroll
                for (int k = 0; k < RABIT_MAX_K; ++k) {
                    if (k >= G.K) break;
                    cp_async_wait<kDepth - 1>();
                    const uint4 wv = my_ring[slot * 32];
                    {   // refill the slot just read
                        const uint4* src = pf.next();
                        if (src) cp_async16(my_ring_s + slot * 512, src);
                        cp_async_commit();
                        slot = slot + 1 == kDepth ? 0 : slot + 1;
                    }
                    const uint32_t* tb = table + ((size_t)((k * ncg + q) * 4) * NCOL + gq) * 8 + tq * 2;
#pragma unroll
                    for (int cs = 0; cs < 4; ++cs) {
                        uint2 bb = make_uint2(0u, 0u);
                        if (gq < NCOL) bb = *reinterpret_cast<const uint2*>(tb + (size_t)cs * NCOL * 8);
#pragma unroll
                        for (int rg = 0; rg < 2; ++rg) {
                            const uint32_t mask = 0x01010101u << (rg + 2 * cs);
                            mma_u8s8(acc[k][rg], wv.x & mask, wv.y & mask, wv.z & mask, wv.w & mask, bb.x, bb.y);
                        }
                    }
                }
            }
            // ---- epilogue: digits -> sum_j b T, then sum_j t - 2 sum_j b t, g_k, path sum
            const int b = (NB == 2) ? (tq >> 1) : 0;
#pragma unroll
            for (int k = 0; k < RABIT_MAX_K; ++k) {
                if (k >= G.K) break;
                const float inv = s_inv[b][k], sumT = s_sumTf[b][k];
#pragma unroll
                for (int rg = 0; rg < 2; ++rg) {
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        const float lo = fmaf(256.f, (float)acc[k][rg][2 * hf + 1], (float)acc[k][rg][2 * hf]);
                        const float hi = __shfl_xor_sync(0xffffffffu, lo, 1);            // digits 2,3 live in the odd lane
                        const float v = fmaf(65536.f, hi, lo);                            // 64 * 2^rg * sum_j b T
                        const float s_sigma = fmaf(v, rg ? -0.015625f : -0.03125f, sumT); // sum T - 2 sum b T
                        const int row = rt * 32 + 2 * (gq + 8 * hf) + rg;
                        yv[hf][rg] = fmaf(__half2float(P.g[(size_t)k * G.Mp + row]), s_sigma * inv, yv[hf][rg]);
                    }
                }
            }
            const bool owner = (tq & 1) == 0 && (NB == 2 || tq == 0);
            if (G.n_slices == 1) {
                if (owner) {
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                        for (int rg = 0; rg < 2; ++rg) {
                            const int row = rt * 32 + 2 * (gq + 8 * hf) + rg;
                            if (row < G.M) P.y[(size_t)b * G.M + row] = __float2half_rn(yv[hf][rg]);
                        }
                }
            } else {
                if (owner) {
                    float* dst = P.partial + ((size_t)b * G.n_slices + s) * G.Mp + rt * 32 + 2 * gq;
                    *reinterpret_cast<float2*>(dst) = make_float2(yv[0][0], yv[0][1]);
                    *reinterpret_cast<float2*>(dst + 16) = make_float2(yv[1][0], yv[1][1]);
                }
                __threadfence();
                __syncwarp();
                unsigned int old = 0;
                if (lane == 0) old = atomicAdd(P.counters + rt, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == (unsigned)G.n_slices - 1) {       // this warp completed the row tile: reduce in slice order
                    __threadfence();
                    const int row = rt * 32 + lane;
#pragma unroll
                    for (int bb = 0; bb < NB; ++bb) {
                        float sum = 0.f;
                        for (int ss = 0; ss < G.n_slices; ++ss)
                            sum += __ldcg(P.partial + ((size_t)bb * G.n_slices + ss) * G.Mp + row);
                        if (row < G.M) P.y[(size_t)bb * G.M + row] = __float2half_rn(sum);
                    }
                    if (lane == 0) P.counters[rt] = 0;       // leave the scratch clean for the next call
                }
            }
        }
        __syncthreads();                                     // the digit table is rebuilt for the next slice
        seg_start = seg_end;
    }
    cp_async_wait<0>();
}

size_t smem_bytes(const RabitGeom& G, int nb) {
    return (size_t)kWarps * kDepth * 512 + (size_t)G.K * G.slice_cg * 4 * (4 * nb) * 8 * 4;
}

}  // namespace

bool rabit_gemv_mma_supports(const rabit_layer& L, int batch) {
    return batch >= 1 && batch <= 2 && L.geom.slice_cg <= kMaxSliceCg;
}

cudaError_t rabit_launch_gemv_mma(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    GemvParams P;
    P.G = L.geom;
    P.bits = L.d_bits;
    P.g = (const __half*)L.d_g;
    P.h = (const __half*)L.d_h;
    P.x = (const __half*)x;
    P.y = (__half*)y;
    P.partial = L.d_partial;
    P.counters = L.d_counters;
    P.n_items = L.geom.n_slices * L.geom.n_rt;
    const int sms = L.sm_count > 0 ? L.sm_count : 148;
    const int grid = P.n_items < sms ? P.n_items : sms;
    const size_t smem = smem_bytes(L.geom, batch);
    static bool attr_done[2] = {false, false};
    if (batch == 1) {
        if (!attr_done[0]) {
            cudaError_t e = cudaFuncSetAttribute(rabit_gemv_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
            if (e != cudaSuccess) return e;
            attr_done[0] = true;
        }
        rabit_gemv_mma_kernel<1><<<grid, kThreads, smem, stream>>>(P);
    } else {
        if (!attr_done[1]) {
            cudaError_t e = cudaFuncSetAttribute(rabit_gemv_mma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
            if (e != cudaSuccess) return e;
            attr_done[1] = true;
        }
        rabit_gemv_mma_kernel<2><<<grid, kThreads, smem, stream>>>(P);
    }
    return cudaGetLastError();
}
