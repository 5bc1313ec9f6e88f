// Decode GEMV for 3..16 batch rows: the batch sits in the N dimension of an f16 tensor-core MMA.
//
//   y[b][i] = sum_k g_k[i] * sum_j (B_k[i][j] h_k[j]) * x[b][j]                              (Section 4.1, Eq. 2)
//
// The table-driven kernel (rabit_gemv_lut.cu) pays per batch row; the integer tensor-core GEMV spends four of an MMA's
// eight columns per batch row and needs a pass over x first.  Here the A operand of mma.sync.m16n8k16 is +-h_k expanded in
// registers from the sign tiles (the weight bit flips the sign bit of the fp16 input scale: exact), B is x as it is, the
// accumulators are fp32: products are exact, 8 batch rows per MMA and 16 with a second MMA on the same A, no digits, no
// scale search.  The cost is that of the expansion (five logic instructions per two A registers) and does not depend on
// the batch.
//
// Operand mapping.  A sign tile (rabit_layout.h) gives lane (gq, tq) four words w[a]; byte c of word a has in bit p the
// sign of row 16p + gq + 8(a & 1), column 16(a >> 1) + 4tq + c of the tile.  For the k-step kh = a >> 1 (16 columns) and
// the row block p, the MMA's k slots (2tq, 2tq+1, 2tq+8, 2tq+9) of lane (gq, tq) are taken to be the tile columns
// 16kh + 4tq + (0, 1, 2, 3): any fixed assignment of slots to columns is valid as long as A and B use the same one.  Then
//     a0 = +-h(cols 0,1) for row gq      from bytes 0,1 of w[2kh]         a1 = the same columns, row gq + 8, from w[2kh+1]
//     a2 = +-h(cols 2,3) for row gq      from bytes 2,3 of w[2kh]         a3 = row gq + 8, from w[2kh+1]
//     b0 = x[n = gq][cols 0,1]           b1 = x[n = gq][cols 2,3]         (one 8-byte load per lane and k-step)
// and the accumulator lane holds rows gq, gq + 8 of the block and batch rows 2tq, 2tq + 1.
//
// Work split.  A unit is (row tile of 128 rows) x (a range of whole 256-column slices), all paths.  One CTA of 8 warps per
// unit; warp w works on path w % K and shares the column tiles of the range with the other warps of that path, one
// 512-byte tile per 128-bit load per lane, several tiles ahead.  At the end every warp scales its accumulators by g_k and
// writes them to its own slot of shared memory, the CTA adds the slots in a fixed order (deterministic), and every output
// of the unit goes, as in the table-driven kernel, into the row's 64-bit accumulate word with one integer atomic
// (fixed-point grid of the packer, arrival count in bits 55..62, bit 63 = non-finite); the lane whose add completes a row
// rounds it to fp16, stores y and clears the word.  A contribution that covers s slices is shifted by s * 2^fix_bits, so
// the total shift is the same n_cs * 2^fix_bits for every split.  Nothing waits for another CTA.
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>

#include "rabit_internal.h"

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxUnits = 1 << 20;
constexpr unsigned long long kSumMask = (1ULL << 55) - 1;

struct F16Params {
    const uint4* tiles;
    const __half* g;
    const __half* h;
    const __half* x;
    __half* y;
    unsigned long long* acc;        // [16][Mp], all zero between calls
    int K, M, N, Mp, n_rt, n_ct, n_cs;
    int batch;
    int splits;                     // column ranges per row tile; range r covers slices [r * n_cs / splits, (r + 1) * n_cs / splits)
    int n_units;                    // n_rt * splits
    int fix_bits;
    float inv_unit, unit, limit;
};

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(s));
    return r;
}
// (a & 0x80008000) ^ c: the sign bits of two fp16 values, applied to a pair of input scales
__device__ __forceinline__ uint32_t flip(uint32_t a, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, 0x80008000, %2, 0x6A;" : "=r"(r) : "r"(a), "r"(c));
    return r;
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// What a warp needs besides the sign words for one column tile of its path.
template <int NH>
struct Feed {
    uint2 h[2];                      // input scales of its four columns, per k-step
    uint2 x[2][NH];                  // activations of its four columns, per k-step and half of the batch
};

// NH = halves of the batch (8 rows each) a pass carries; DEPTH = sign tiles a warp keeps in flight.
template <int NH, int DEPTH>
__global__ void __launch_bounds__(kThreads, 2)
rabit_gemv_f16_kernel(const __grid_constant__ F16Params P) {
    extern __shared__ __align__(16) float slots[];                       // [kWarps][NH * 8][128] scaled partial outputs
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tq = lane & 3;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited = false;

    for (int unit = blockIdx.x; unit < P.n_units; unit += gridDim.x) {
        const int rt = unit / P.splits, r = unit - rt * P.splits;
        const int s0 = (int)((long long)r * P.n_cs / P.splits), s1 = (int)((long long)(r + 1) * P.n_cs / P.splits);
        const int c0 = s0 * 8, c1 = min(P.n_ct, s1 * 8);                 // column tiles of the range (a slice is eight of them)
        // every warp works on ONE path: path k = warp % K, and the column tiles of the range are dealt out among the warps of
        // that path (K = 3: three, three and two warps)
        const int k = warp % P.K;
        const int n_same = (kWarps - k + P.K - 1) / P.K, j0 = warp / P.K;

        float acc[8][NH][4];
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int hf = 0; hf < NH; ++hf)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[p][hf][e] = 0.f;

        auto fetch_w = [&](int ct) {                                     // weights: never depend on the stream's past
            return ldg_stream(P.tiles + (((size_t)rt * P.K + k) * P.n_ct + ct) * 32 + lane);
        };
        auto fetch_hx = [&](int ct, Feed<NH>& f) {                       // input scales and activations of the lane's columns (L1 / L2 hits)
            const __half* hp = P.h + (size_t)k * P.N + ct * 32 + 4 * tq;
            f.h[0] = __ldg(reinterpret_cast<const uint2*>(hp));
            f.h[1] = __ldg(reinterpret_cast<const uint2*>(hp + 16));
#pragma unroll
            for (int hf = 0; hf < NH; ++hf) {
                const int b = 8 * hf + gq;
                f.x[0][hf] = make_uint2(0u, 0u);
                f.x[1][hf] = make_uint2(0u, 0u);
                if (b < P.batch) {
                    const __half* xp = P.x + (size_t)b * P.N + ct * 32 + 4 * tq;
                    f.x[0][hf] = __ldcg(reinterpret_cast<const uint2*>(xp));
                    f.x[1][hf] = __ldcg(reinterpret_cast<const uint2*>(xp + 16));
                }
            }
        };

        // weights DEPTH tiles ahead (HBM latency), scales and activations one ahead
        uint4 wq[DEPTH];
        const int ct0 = c0 + j0;
#pragma unroll
        for (int d = 0; d < DEPTH; ++d) {
            wq[d] = make_uint4(0u, 0u, 0u, 0u);
            if (ct0 + d * n_same < c1) wq[d] = fetch_w(ct0 + d * n_same);
        }
        if (!waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");            // x, y and the accumulate words only after this
            waited = true;
        }
        Feed<NH> cur, nxt;
        if (ct0 < c1) fetch_hx(ct0, cur);
        for (int base = ct0; base < c1; base += DEPTH * n_same) {
#pragma unroll
            for (int d = 0; d < DEPTH; ++d) {
                const int ct = base + d * n_same;
                if (ct >= c1) break;
                const uint4 wv = wq[d];
                if (ct + DEPTH * n_same < c1) wq[d] = fetch_w(ct + DEPTH * n_same);
                if (ct + n_same < c1) fetch_hx(ct + n_same, nxt);
                const uint32_t w[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {
                    const uint32_t h01 = cur.h[kh].x, h23 = cur.h[kh].y;
#pragma unroll
                    for (int p = 0; p < 8; ++p) {
                        const uint32_t sl = w[2 * kh] << (7 - p), sh = w[2 * kh + 1] << (7 - p);   // bit p of every byte -> bit 7
                        const uint32_t a0 = flip(prmt(sl, 0u, 0x1404), h01), a2 = flip(prmt(sl, 0u, 0x3424), h23);
                        const uint32_t a1 = flip(prmt(sh, 0u, 0x1404), h01), a3 = flip(prmt(sh, 0u, 0x3424), h23);
#pragma unroll
                        for (int hf = 0; hf < NH; ++hf) mma_f16(acc[p][hf], a0, a1, a2, a3, cur.x[kh][hf].x, cur.x[kh][hf].y);
                    }
                }
                cur = nxt;
            }
        }
        // the path's output scale, in place
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const int row = rt * RABIT_TILE_ROWS + 16 * p + gq;
            const float g_lo = __half2float(P.g[(size_t)k * P.Mp + row]), g_hi = __half2float(P.g[(size_t)k * P.Mp + row + 8]);
#pragma unroll
            for (int hf = 0; hf < NH; ++hf) {
                acc[p][hf][0] *= g_lo; acc[p][hf][1] *= g_lo;
                acc[p][hf][2] *= g_hi; acc[p][hf][3] *= g_hi;
            }
        }

        // ---- the warp's scaled partial outputs -> its slot; slot layout [batch row][row of the tile]
        float* mine = slots + (size_t)warp * (NH * 8 * 128);
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int hf = 0; hf < NH; ++hf) {
                const int b = 8 * hf + 2 * tq, row = 16 * p + gq;
                mine[(b) * 128 + row] = acc[p][hf][0];
                mine[(b + 1) * 128 + row] = acc[p][hf][1];
                mine[(b) * 128 + row + 8] = acc[p][hf][2];
                mine[(b + 1) * 128 + row + 8] = acc[p][hf][3];
            }
        __syncthreads();
        // ---- fixed-order sum over the warps, then one atomic per output of the unit
        const int n_slices = s1 - s0;
        constexpr int kPer = NH * 8 * 128 / kThreads;                    // outputs per thread (4 or 8)
        unsigned long long old[kPer], add[kPer];
        bool bad[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int o = tid + i * kThreads, b = o >> 7, rl = o & 127;
            old[i] = 0ULL; add[i] = 0ULL; bad[i] = false;
            if (b >= P.batch) continue;
            float v = 0.f;
#pragma unroll
            for (int wv = 0; wv < kWarps; ++wv) v += slots[(size_t)wv * (NH * 8 * 128) + o];
            const float scaled = v * P.inv_unit;
            bad[i] = !(fabsf(scaled) < P.limit * (float)n_slices);       // inf or NaN: finite inputs cannot get here
            const long long q = bad[i] ? 0LL : __float2ll_rn(scaled);
            add[i] = (unsigned long long)(q + ((long long)n_slices << P.fix_bits)) + (1ULL << 55);
            unsigned long long* word = P.acc + (size_t)b * P.Mp + rt * RABIT_TILE_ROWS + rl;
            if (bad[i]) atomicOr(word, 1ULL << 63);
            old[i] = atomicAdd(word, add[i]);
        }
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int o = tid + i * kThreads, b = o >> 7, rl = o & 127;
            if (b >= P.batch) continue;
            if ((int)((old[i] >> 55) & 0xFFu) != P.splits - 1) continue;  // other column ranges are still to come
            const unsigned long long sum = (old[i] & kSumMask) + (add[i] & kSumMask);
            const long long total = (long long)sum - ((long long)P.n_cs << P.fix_bits);
            const bool poisoned = bad[i] || (old[i] >> 63) != 0;
            const float v = poisoned ? __int_as_float(0x7FC00000) : __ll2float_rn(total) * P.unit;
            const int row = rt * RABIT_TILE_ROWS + rl;
            if (row < P.M) P.y[(size_t)b * P.M + row] = __float2half_rn(v);
            P.acc[(size_t)b * P.Mp + row] = 0ULL;                         // resting state for the next call
        }
        __syncthreads();                                                 // the slots are free for the next unit
    }
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <int NH, int DEPTH>
cudaError_t launch(const F16Params& P, int grid, int device, cudaStream_t stream) {
    static bool attr_done[64] = {false};
    const size_t smem = (size_t)kWarps * NH * 8 * 128 * sizeof(float);
    const int slot = device >= 0 && device < 64 ? device : 0;
    if (!attr_done[slot] || slot != device) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemv_f16_kernel<NH, DEPTH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done[slot] = true;
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
    return cudaLaunchKernelEx(&cfg, rabit_gemv_f16_kernel<NH, DEPTH>, P);
}

}  // namespace

bool rabit_gemv_f16_supports(const rabit_layer& L, int batch) {
    if (batch < 1 || batch > RABIT_MAX_GEMV_BATCH) return false;
    if (L.geom.n_cs > RABIT_LUT_MAX_SLICES || L.d_acc == nullptr) return false;
    return (long long)L.geom.n_rt * L.geom.n_cs < kMaxUnits;
}

// One launch, 1..16 batch rows (x: [batch][N], y: [batch][M]).
cudaError_t rabit_launch_gemv_f16(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    if (!rabit_gemv_f16_supports(L, batch)) return cudaErrorInvalidValue;
    const RabitGeom& G = L.geom;
    F16Params P;
    P.tiles = L.d_bits;
    P.g = (const __half*)L.d_g;
    P.h = (const __half*)L.d_h;
    P.x = (const __half*)x;
    P.y = (__half*)y;
    P.acc = L.d_acc;
    P.K = G.K; P.M = G.M; P.N = G.N; P.Mp = G.Mp; P.n_rt = G.n_rt; P.n_ct = G.n_ct; P.n_cs = G.n_cs;
    P.batch = batch;
    P.fix_bits = G.fix_bits;
    P.unit = ldexpf(1.f, G.unit_exp);
    P.inv_unit = ldexpf(1.f, -G.unit_exp);
    P.limit = ldexpf(1.f, G.fix_bits);
    const int sms = L.sm_count > 0 ? L.sm_count : 148;
    const int resident = 2 * sms;                                        // two CTAs per SM
    // Column ranges per row tile: the split that minimises  waves x (slices per unit + 1)  (a unit's fixed cost, its
    // reduction and atomics, is about one slice's worth of tiles).
    int splits = 1;
    long long best = -1;
    for (int s = 1; s <= G.n_cs; ++s) {
        const long long units = (long long)G.n_rt * s;
        const long long waves = (units + resident - 1) / resident;
        const long long cost = waves * ((G.n_cs + s - 1) / s + 1);
        if (best < 0 || cost < best) { best = cost; splits = s; }
    }
    P.splits = splits;
    P.n_units = G.n_rt * splits;
    const int grid = P.n_units < resident ? P.n_units : resident;
    return batch <= 8 ? launch<1, 4>(P, grid, L.device, stream) : launch<2, 2>(P, grid, L.device, stream);
}
