// Decode GEMV on the integer tensor-core path (batch 1..2 per launch).
//
//   y[b][i] = sum_k g_k[i] * sum_j B_k[i][j] * t_k[b][j],   t_k[b][j] = h_k[j] * x[b][j]     (Section 4.1, Eq. 2)
//
// At one bit per weight the sign-select arithmetic, not HBM, is the limit on B200: plain
// logic instructions issue at 64 lanes/clk/SM per sub-partition pair while HBM delivers
// ~180 weight bits/clk/SM.  This kernel spends one logic instruction per FOUR weights: a
// packed word masked with 0x01010101 << p is already a u8 MMA operand with entries {0, 2^p}
// (see rabit_layout.h), and mma.sync.m16n8k32.u8.s8 does the additions.  The B operand holds
// t in exact fixed point: T = round(t * sigma), sigma a power of two chosen per (path,
// batch row) from max|x| * max|h_k| so that |T| < 2^30, split into four balanced base-256
// digits that occupy four of the eight MMA columns (a second batch row takes the other
// four).  With b the sign bit, sum_j B t = sum_j t - 2 sum_j b t; the int32 accumulators
// give sum_j b T per digit exactly, and the epilogue recombines the digits, applies
// 1/sigma, g_k and the path sum in fp32.  The roundings are T (at most 2^-31 of the bound
// per term), the fp32 epilogue and the final fp16 store.
//
// Structure of a CTA (12 warps):
//   * The tiles of the layer are numbered in layout order; CTA c owns positions
//     [c*T/G, (c+1)*T/G), one contiguous byte range, so the split is even for every shape.
//   * One elected thread streams that range with bulk asynchronous copies into a ring of
//     8 KB stages (mbarrier transaction counts).  The copies for the first ring-full are
//     issued BEFORE the programmatic-dependency wait: weights never depend on the previous
//     kernel in the stream, so they stream in while that kernel is still finishing.
//   * Four builder warps turn x and h into the digit table of each stage (the B fragments,
//     in fragment order) plus the per-tile sum of T, one stage ahead of the consumers.
//   * Eight MMA warps take the tiles of a stage round-robin: one 128-bit shared-memory read
//     of weights, one 64-bit read of digits, 32 ANDs and 8 MMAs per 4096 weights.
//   * A segment is the part of the CTA range inside one (row tile, path) strip.  At a
//     segment end the warps are summed in shared memory, scaled by g_k / sigma and written
//     to a per-layer fp32 partial buffer; the CTA whose arrival completes a row tile adds
//     the partials in a fixed order (deterministic) and stores fp16.
// Every wait in the kernel is bounded; a wait that runs out sets a status word and the
// kernel drains and returns (results are then invalid, the context stays usable).
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kMmaWarps = 8;
constexpr int kBuildWarps = 4;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kThreads = (kMmaWarps + kBuildWarps) * 32;
constexpr int kStageTiles = 16;
constexpr int kRing = 8;
constexpr long long kWaitLimitCycles = 1LL << 31;       // about one second

struct GemvParams {
    RabitGeom G;
    const unsigned char* bits;
    const __half* g;
    const __half* h;
    const __half* x;
    __half* y;
    float* partial;          // [n_rt*K + grid][RABIT_PARTIAL_BATCH][128]
    unsigned int* counters;  // [n_rt]
    unsigned int* status;
    long long n_tiles;       // n_rt * K * n_ct
};

template <int NB>
struct __align__(128) Smem {
    uint4 bits[kRing][kStageTiles][32];
    uint2 table[kRing][kStageTiles][NB * 16];           // word pair of lane l (n = l >> 2, tq = l & 3) at index l
    long long sum_t[kRing][kStageTiles][NB];
    float red[kMmaWarps][NB][RABIT_TILE_ROWS];
    unsigned long long full[kRing];
    unsigned long long empty[kRing];
    unsigned int xmax_bits[NB];
    int abort_flag;
    int is_last;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitLimitCycles or as soon as any thread of the CTA gave up.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return; }
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bar_mma_warps() { asm volatile("bar.sync 1, %0;" ::"n"(kMmaThreads) : "memory"); }

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// CTA that owns tile position p when T tiles are split over G CTAs as [c*T/G, (c+1)*T/G).
__device__ __forceinline__ int cta_of(long long p, long long T, int G) { return (int)(((p + 1) * G - 1) / T); }

// sigma = 2^s with |h x| * sigma < 2^30 for every column; inv = 2^-s (NaN if the inputs are not finite).
__device__ __forceinline__ void choose_scale(unsigned int xmax_bits, float hmax, float& sigma, float& inv) {
    const float xm = __half2float(__ushort_as_half((unsigned short)xmax_bits));
    const float bound = xm * hmax;
    if (xmax_bits >= 0x7C00u || !(bound < __int_as_float(0x7F800000))) {      // inf / NaN anywhere in x or h
        sigma = 0.f; inv = __int_as_float(0x7FC00000);
        return;
    }
    if (bound == 0.f) { sigma = 1.f; inv = 1.f; return; }
    const int e = (__float_as_int(bound) >> 23) & 0xFF;                         // bound < 2^(e - 126)
    int s = 156 - e;                                                            // 30 - (e - 126)
    s = s > 120 ? 120 : s;
    sigma = __int_as_float((s + 127) << 23);
    inv = __int_as_float((127 - s) << 23);
}

template <int NB>
__global__ void __launch_bounds__(kThreads, 2)
rabit_gemv_mma_kernel(const GemvParams P) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem<NB>& S = *reinterpret_cast<Smem<NB>*>(smem_raw);
    const RabitGeom& G = P.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = G.n_ct;
    const long long T = P.n_tiles;
    const int grid = gridDim.x;
    const long long lo = (long long)blockIdx.x * T / grid;
    const long long hi = (long long)(blockIdx.x + 1) * T / grid;
    const int n_tiles = (int)(hi - lo);
    const int n_stages = (n_tiles + kStageTiles - 1) / kStageTiles;
    volatile int* abort_flag = &S.abort_flag;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(&S.full[s]), 1 + kBuildWarps);
            mbar_init(smem_u32(&S.empty[s]), kMmaWarps);
        }
        for (int b = 0; b < NB; ++b) S.xmax_bits[b] = 0;
        S.abort_flag = 0;
        S.is_last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // ---- weights of the first ring-full start streaming before anything that depends on the stream's past
    const int prefetched = n_stages < kRing ? n_stages : kRing;
    if (tid == kMmaThreads) {
        for (int i = 0; i < prefetched; ++i) {
            const int tiles = min(kStageTiles, n_tiles - i * kStageTiles);
            const uint32_t bar = smem_u32(&S.full[i]);
            mbar_expect_tx(bar, tiles * RABIT_TILE_BYTES);
            bulk_g2s(smem_u32(&S.bits[i][0][0]), P.bits + (lo + (long long)i * kStageTiles) * RABIT_TILE_BYTES,
                     tiles * RABIT_TILE_BYTES, bar);
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- largest |x| per batch row (fp16 bit patterns order like unsigned integers once the sign is cleared)
    {
        const int vec_per_row = G.N / 8;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            unsigned int m = 0;
            const uint4* xr = reinterpret_cast<const uint4*>(P.x + (size_t)b * G.N);
            for (int i = tid; i < vec_per_row; i += kThreads) {
                const uint4 v = __ldg(xr + i);
                unsigned int a = __vmaxu2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu);
                a = __vmaxu2(a, __vmaxu2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu));
                m = __vmaxu2(m, a);
            }
            m = max(m & 0xFFFFu, m >> 16);
            m = __reduce_max_sync(0xffffffffu, m);
            if (lane == 0 && m) atomicMax(&S.xmax_bits[b], m);
        }
    }
    __syncthreads();
    if (n_tiles == 0) return;

    if (warp >= kMmaWarps) {
        // =========================== builder warps (and the copy issuer) ===========================
        const int bl = tid - kMmaThreads;            // 0..127
        const int j = bl >> 3, u = bl & 7;           // tile inside the stage, group of 4 columns inside the tile
        const int tq = u & 3, half = u >> 2;
        float sigma[NB][RABIT_MAX_K];
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int k = 0; k < RABIT_MAX_K; ++k) {
                float inv;
                choose_scale(S.xmax_bits[b], k < G.K ? G.hmax[k] : 0.f, sigma[b][k], inv);
            }
        long long p0 = lo + j;
        int ct = (int)(p0 % C);
        int k = (int)((p0 / C) % G.K);
        for (int i = 0; i < n_stages; ++i) {
            const int slot = i % kRing;
            if (i >= kRing) {
                mbar_wait(smem_u32(&S.empty[slot]), ((i / kRing) - 1) & 1, abort_flag);
                if (tid == kMmaThreads) {
                    const int tiles = min(kStageTiles, n_tiles - i * kStageTiles);
                    const uint32_t bar = smem_u32(&S.full[slot]);
                    mbar_expect_tx(bar, tiles * RABIT_TILE_BYTES);
                    bulk_g2s(smem_u32(&S.bits[slot][0][0]), P.bits + (lo + (long long)i * kStageTiles) * RABIT_TILE_BYTES,
                             tiles * RABIT_TILE_BYTES, bar);
                }
            }
            const bool live = i * kStageTiles + j < n_tiles;
            const int col = ct * RABIT_TILE_COLS + 4 * u;
            uint2 hraw = make_uint2(0u, 0u);
            if (live) hraw = __ldg(reinterpret_cast<const uint2*>(P.h + (size_t)k * G.N + col));
            const float2 h01 = __half22float2(*reinterpret_cast<const __half2*>(&hraw.x));
            const float2 h23 = __half22float2(*reinterpret_cast<const __half2*>(&hraw.y));
            float sg[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) sg[b] = k == 0 ? sigma[b][0] : (k == 1 ? sigma[b][1] : sigma[b][2]);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                uint2 xraw = make_uint2(0u, 0u);
                if (live) xraw = __ldg(reinterpret_cast<const uint2*>(P.x + (size_t)b * G.N + col));
                const float2 x01 = __half22float2(*reinterpret_cast<const __half2*>(&xraw.x));
                const float2 x23 = __half22float2(*reinterpret_cast<const __half2*>(&xraw.y));
                int Tq[4];
                Tq[0] = __float2int_rn(h01.x * x01.x * sg[b]);
                Tq[1] = __float2int_rn(h01.y * x01.y * sg[b]);
                Tq[2] = __float2int_rn(h23.x * x23.x * sg[b]);
                Tq[3] = __float2int_rn(h23.y * x23.y * sg[b]);
                long long tsum = (long long)Tq[0] + Tq[1] + Tq[2] + Tq[3];
                tsum += __shfl_xor_sync(0xffffffffu, tsum, 1);
                tsum += __shfl_xor_sync(0xffffffffu, tsum, 2);
                tsum += __shfl_xor_sync(0xffffffffu, tsum, 4);
                uint32_t X[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) X[c] = ((uint32_t)Tq[c] + 0x80808080u) ^ 0x80808080u;   // bytes = balanced digits
                const uint32_t t0 = __byte_perm(X[0], X[1], 0x5140), t1 = __byte_perm(X[2], X[3], 0x5140);
                const uint32_t t2 = __byte_perm(X[0], X[1], 0x7362), t3 = __byte_perm(X[2], X[3], 0x7362);
                uint32_t dig[4];
                dig[0] = __byte_perm(t0, t1, 0x5410); dig[1] = __byte_perm(t0, t1, 0x7632);
                dig[2] = __byte_perm(t2, t3, 0x5410); dig[3] = __byte_perm(t2, t3, 0x7632);
                uint32_t* dst = reinterpret_cast<uint32_t*>(&S.table[slot][j][b * 16]) + tq * 2 + half;
#pragma unroll
                for (int d = 0; d < 4; ++d) dst[d * 8] = dig[d];                 // word pair index 4*d + tq
                if (u == 0) S.sum_t[slot][j][b] = tsum;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&S.full[slot]));
            ct += kStageTiles;
            while (ct >= C) { ct -= C; k = k + 1 == G.K ? 0 : k + 1; }
        }
        if (*abort_flag && tid == kMmaThreads) {
            // make sure no bulk copy is still in flight towards this CTA's shared memory
            for (int i = max(0, n_stages - kRing); i < n_stages; ++i) {
                const long long t0 = clock64();
                while (!mbar_try_wait(smem_u32(&S.full[i % kRing]), (i / kRing) & 1))
                    if (clock64() - t0 > kWaitLimitCycles) break;
            }
            atomicExch(P.status, 1u);
        }
        return;
    }

    // ======================================= MMA warps =======================================
    const int gq = lane >> 2, tq = lane & 3;
    const int w = warp;
    float sig_inv[RABIT_MAX_K];               // 1 / sigma of this thread's batch row at reduction time
    {
        const int b = (tid >> 7) < NB ? (tid >> 7) : 0;
#pragma unroll
        for (int k = 0; k < RABIT_MAX_K; ++k) {
            float sg;
            choose_scale(S.xmax_bits[b], k < G.K ? G.hmax[k] : 0.f, sg, sig_inv[k]);
        }
    }
    long long strip = lo / C;
    int seg_end = (int)min((long long)n_tiles, (strip + 1) * C - lo);     // relative to lo
    int k = (int)(strip % G.K);
    int rt = (int)(strip / G.K);
    const int red_b = tid >> 7, red_r = tid & 127;                         // this thread's (batch row, row) at reduction time
    float gval = 0.f;
    if (red_b < NB) gval = __half2float(P.g[(size_t)k * G.Mp + rt * RABIT_TILE_ROWS + red_r]);

    int acc[8][4];
    long long sum_t[NB];
#pragma unroll
    for (int p = 0; p < 8; ++p)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[p][c] = 0;
#pragma unroll
    for (int b = 0; b < NB; ++b) sum_t[b] = 0;

    // Segment end: reduce the eight warps, scale, publish; the last contributor of the row tile finishes y.
    auto segment_flush = [&]() {
        // digits -> 2^p * sum_j b T, then sum_j T - 2 sum_j b T per row (fp32), into shared memory
#pragma unroll
        for (int p = 0; p < 8; ++p) {
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const float lo2 = fmaf(256.f, (float)acc[p][2 * hf + 1], (float)acc[p][2 * hf]);
                const float hi2 = __shfl_xor_sync(0xffffffffu, lo2, 1);        // digits 2,3 live in the odd lane
                const int b = tq >> 1;
                if ((tq & 1) == 0 && b < NB) {
                    const float v = fmaf(65536.f, hi2, lo2);                    // 2^p * sum_j b T
                    const float st = __ll2float_rn(b == 0 ? sum_t[0] : sum_t[NB - 1]);
                    const float scale = __int_as_float((127 + 1 - p) << 23);    // 2^(1-p)
                    S.red[w][b][16 * p + gq + 8 * hf] = fmaf(-scale, v, st);
                }
            }
        }
        bar_mma_warps();
        if (red_b < NB) {
            float sum = 0.f;
#pragma unroll
            for (int ww = 0; ww < kMmaWarps; ++ww) sum += S.red[ww][red_b][red_r];
            const float inv = k == 0 ? sig_inv[0] : (k == 1 ? sig_inv[1] : sig_inv[2]);
            const long long seg_id = (long long)blockIdx.x + strip;
            P.partial[(seg_id * RABIT_PARTIAL_BATCH + red_b) * RABIT_TILE_ROWS + red_r] = gval * (sum * inv);
        }
        __threadfence();
        bar_mma_warps();
        // contributors of this row tile: for every path, the CTAs whose range meets its strip
        int first_cta[RABIT_MAX_K], last_cta[RABIT_MAX_K];
        unsigned int expected = 0;
#pragma unroll
        for (int kk = 0; kk < RABIT_MAX_K; ++kk) {
            first_cta[kk] = 0; last_cta[kk] = -1;
            if (kk < G.K) {
                const long long s0 = ((long long)rt * G.K + kk) * C;
                first_cta[kk] = cta_of(s0, T, grid);
                last_cta[kk] = cta_of(s0 + C - 1, T, grid);
                expected += (unsigned int)(last_cta[kk] - first_cta[kk] + 1);
            }
        }
        if (tid == 0) {
            const unsigned int old = atomicAdd(P.counters + rt, 1u);
            S.is_last = (old == expected - 1u);
        }
        bar_mma_warps();
        if (S.is_last) {
            __threadfence();
            if (red_b < NB) {
                float sum = 0.f;
#pragma unroll
                for (int kk = 0; kk < RABIT_MAX_K; ++kk)
                    for (int c = first_cta[kk]; c <= last_cta[kk]; ++c) {
                        const long long sid = (long long)c + (long long)rt * G.K + kk;
                        sum += __ldcg(P.partial + (sid * RABIT_PARTIAL_BATCH + red_b) * RABIT_TILE_ROWS + red_r);
                    }
                const int row = rt * RABIT_TILE_ROWS + red_r;
                if (row < G.M) P.y[(size_t)red_b * G.M + row] = __float2half_rn(sum);
            }
            if (tid == 0) P.counters[rt] = 0;                                   // leave the scratch clean for the next call
        }
        bar_mma_warps();                                                        // S.red and S.is_last are reused
    };

    auto next_segment = [&]() {
        strip += 1;
        seg_end = (int)min((long long)n_tiles, (long long)seg_end + C);
        k += 1;
        if (k == G.K) { k = 0; rt += 1; }
        gval = 0.f;
        if (red_b < NB) gval = __half2float(P.g[(size_t)k * G.Mp + rt * RABIT_TILE_ROWS + red_r]);
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[p][c] = 0;
#pragma unroll
        for (int b = 0; b < NB; ++b) sum_t[b] = 0;
    };

    // This warp's tiles are rel = w, w + 8, ...: two per full stage, so every warp releases every full stage.
    int cur_stage = -1;
#pragma unroll 1
    for (int rel = w; rel < n_tiles; rel += kMmaWarps) {
        const int i = rel / kStageTiles, j = rel % kStageTiles;
        const int slot = i % kRing;
        if (i != cur_stage) {
            if (cur_stage >= 0) {
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&S.empty[cur_stage % kRing]));
            }
            cur_stage = i;
            mbar_wait(smem_u32(&S.full[slot]), (i / kRing) & 1, abort_flag);
        }
        while (rel >= seg_end) { segment_flush(); next_segment(); }
        const uint4 wv = S.bits[slot][j][lane];
        uint2 bb = make_uint2(0u, 0u);
        if (gq < 4 * NB) bb = S.table[slot][j][lane];
#pragma unroll
        for (int b = 0; b < NB; ++b) sum_t[b] += S.sum_t[slot][j][b];
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const uint32_t mask = 0x01010101u << p;
            mma_u8s8(acc[p], wv.x & mask, wv.y & mask, wv.z & mask, wv.w & mask, bb.x, bb.y);
        }
    }
    if (cur_stage >= 0) {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&S.empty[cur_stage % kRing]));
    }
    while (true) {
        segment_flush();
        if (seg_end >= n_tiles) break;
        next_segment();
    }
}

}  // namespace

bool rabit_gemv_mma_supports(const rabit_layer& L, int batch) {
    const long long tiles = (long long)L.geom.n_rt * L.geom.K * L.geom.n_ct;
    return batch >= 1 && batch <= RABIT_MAX_GEMV_BATCH && tiles < (1LL << 31);
}

template <int NB>
static cudaError_t launch_nb(const GemvParams& P, int grid, cudaStream_t stream) {
    static bool attr_done = false;
    const size_t smem = sizeof(Smem<NB>);
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemv_mma_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rabit_gemv_mma_kernel<NB>, P);
}

cudaError_t rabit_launch_gemv_mma(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    GemvParams P;
    P.G = L.geom;
    P.bits = reinterpret_cast<const unsigned char*>(L.d_bits);
    P.g = (const __half*)L.d_g;
    P.h = (const __half*)L.d_h;
    P.x = (const __half*)x;
    P.y = (__half*)y;
    P.partial = L.d_partial;
    P.counters = L.d_counters;
    P.status = L.d_status;
    P.n_tiles = (long long)L.geom.n_rt * L.geom.K * L.geom.n_ct;
    int grid = L.sm_count > 0 ? L.sm_count : 148;
    if (grid > RABIT_MAX_GRID) grid = RABIT_MAX_GRID;
    if ((long long)grid > P.n_tiles) grid = (int)P.n_tiles;
    return batch == 1 ? launch_nb<1>(P, grid, stream) : launch_nb<2>(P, grid, stream);
}
