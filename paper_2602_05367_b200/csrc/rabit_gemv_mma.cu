// Decode GEMV on the integer tensor-core path (1, 2 or 4 batch rows per launch; the dispatcher uses it for batches
// 3..16, the table-driven kernel of rabit_gemv_lut.cu takes batches 1..2).
//
//   y[b][i] = sum_k g_k[i] * sum_j B_k[i][j] * t_k[b][j],   t_k[b][j] = h_k[j] * x[b][j]     (Section 4.1, Eq. 2)
//
// At one bit per weight the sign-select arithmetic, not HBM, is the limit on B200: plain
// logic instructions issue at 64 lanes/clk/SM per sub-partition pair while HBM delivers
// ~180 weight bits/clk/SM.  This kernel spends one logic instruction per FOUR weights: a
// packed word masked with 0x01010101 << p is already a u8 MMA operand with entries {0, 2^p}
// (see rabit_layout.h), and mma.sync.m16n8k32.u8.s8 does the additions.  The B operand holds
// t in exact fixed point: T = round(t * sigma), sigma a power of two chosen per (path,
// batch row) from max|x| * max|h_k| so that |T| < 2^28, split into four balanced base-256
// digits that occupy four of the eight MMA columns (a second batch row takes the other
// four).  With b the sign bit, sum_j B t = sum_j t - 2 sum_j b t; the int32 accumulators
// give sum_j b T per digit exactly, and the epilogue recombines the digits, applies
// 1/sigma, g_k and the path sum in fp32.  The roundings are T (at most 2^-29 of the bound
// per term), the fp32 epilogue and the final fp16 store.
//
// Structure of a CTA (8 MMA warps plus 2 builder warps and two CTAs per SM up to two batch rows; 4 builder warps and
// one CTA per SM at four):
//   * The tiles of the layer are numbered in layout order; CTA c owns positions
//     [c*T/G, (c+1)*T/G), one contiguous byte range, so the split is even for every shape.
//   * One elected thread streams that range with bulk asynchronous copies into a ring of
//     8 KB stages (mbarrier transaction counts).  The copies for the first ring-full are
//     issued BEFORE the programmatic-dependency wait: weights never depend on the previous
//     kernel in the stream, so they stream in while that kernel is still finishing.
//   * Two builder warps turn x and h into the digit table of each stage (the B fragments,
//     in fragment order) plus the per-tile sum of T, one stage ahead of the consumers.
//   * Eight MMA warps take the tiles of a stage round-robin: one 128-bit shared-memory read
//     of weights, one 64-bit read of digits, 32 ANDs and 8 MMAs per 4096 weights.
//   * A segment is the part of the CTA range inside one (row tile, path) strip.  At a
//     segment end the warps are summed in shared memory, scaled by g_k / sigma and written to
//     a per-layer fp32 partial buffer whose resting content is a sentinel bit pattern (all
//     ones, a NaN no arithmetic here produces): the data is its own "published" flag.  The
//     CTA that owns the last tile of a row tile finishes it: each of its threads reads the
//     partials of its row from the other contributors (all of them CTAs with a lower index,
//     so the waits cannot form a cycle as long as those CTAs are resident or become resident while it
//     waits: the grid is never larger than what the device holds at once, but CUDA does not promise the
//     order in which CTAs start, and another kernel or tenant on the GPU can delay them; the wait is
//     bounded, so that case ends as a recorded time-out with invalid outputs, not as a hang), waiting
//     (bounded) while it still sees the sentinel,
//     puts the sentinel back, adds in a fixed order (deterministic) and stores fp16.
// Every wait in the kernel is bounded; a wait that runs out sets a status word and the
// kernel drains and returns (results are then invalid, the context stays usable).
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kMmaWarps = 8;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kStageTiles = 16;
constexpr int kHeadStages = kMmaWarps / 2;              // first stages, built by the (still idle) MMA warps, one warp pair each

// Per batch width NB (rows of x handled in one pass over the weights): every A fragment feeds (NB+1)/2
// MMAs (two batch rows each).  NB <= 2 runs two CTAs per SM; NB = 4 needs more registers (one CTA per SM)
// and twice the builder warps (each pair converts half of the batch rows).  (NB = 8 would need 128
// accumulator registers per thread and spills at this thread count, so a launch takes at most 4 rows.)
template <int NB>
struct Cfg {
    static constexpr int kPairs = (NB + 1) / 2;
    static constexpr int kBuildWarps = NB <= 2 ? 2 : 4;
    static constexpr int kBuildRows = NB <= 2 ? NB : NB / 2;        // batch rows one builder lane converts
    static constexpr int kThreads = (kMmaWarps + kBuildWarps) * 32;
    static constexpr int kRing = NB <= 4 ? 8 : 6;
    static constexpr int kMinBlocks = NB <= 2 ? 2 : 1;
};
constexpr int kBuildAhead = 3;                          // stages of raw x / h a builder lane keeps in flight
constexpr long long kWaitLimitCycles = 1LL << 31;       // about one second
constexpr unsigned int kSentinel = 0xFFFFFFFFu;         // resting content of the partial buffer ("not written yet")

// Division of a 31-bit dividend by a constant known at launch: n / d = (umulhi(n, mul) + n) >> shr.
struct FastDiv {
    unsigned int mul, shr, d;
};
__host__ inline FastDiv make_fastdiv(unsigned int d) {
    FastDiv f;
    f.d = d;
    unsigned int l = 0;
    while ((1ull << l) < d) ++l;                      // ceil(log2 d)
    f.shr = l;
    f.mul = (unsigned int)((((1ull << l) - d) << 32) / d + 1);
    return f;
}
__device__ __forceinline__ int fdiv(int n, const FastDiv& f) { return (int)((__umulhi((unsigned int)n, f.mul) + (unsigned int)n) >> f.shr); }
__device__ __forceinline__ int fmod(int n, const FastDiv& f) { return n - fdiv(n, f) * (int)f.d; }

struct GemvParams {
    RabitGeom G;
    const unsigned char* bits;
    const __half* g;
    const __half* h;
    const __half* x;
    __half* y;
    float* partial;          // [n_rt*K + grid][RABIT_PARTIAL_BATCH][128]
                             // segment (CTA c, strip s) uses slot c + s; every word rests at kSentinel between calls
    int n_tiles;             // n_rt * K * n_ct (< 2^31)
    int cta0, n_cta;         // the CTAs blockIdx.x = cta0 .. cta0 + n_cta - 1 work on this layer
    int q, r;                // n_tiles = q * n_cta + r: the layer's CTAs 0..r-1 own q+1 tiles, the others q
    FastDiv div_c, div_k, div_kc, div_q, div_q1;   // by n_ct, K, K * n_ct, q, q + 1
};

// A launch runs up to kMaxGroup layers that do not depend on one another (for example the
// projections that read the same activations).  The CTAs of the grid are shared out among the
// layers in proportion to their tiles, so every CTA works on exactly one layer and the tiles of
// a layer are split evenly over its CTAs.
constexpr int kMaxGroup = 8;
struct GroupParams {
    int n_layers;
    unsigned int* status[kMaxGroup];   // the status word of every layer of the group: a wait that runs out is recorded in all of them
    int nb;                  // batch rows actually present (<= the kernel's NB); the others are neither read nor written
    GemvParams layer[kMaxGroup];
};

template <int NB>
struct __align__(128) Smem {
    uint4 bits[Cfg<NB>::kRing][kStageTiles][32];
    uint2 table[Cfg<NB>::kRing][kStageTiles][NB * 16];  // batch row b, digit d, lane quad tq: pair index 16*b + 4*d + tq
    int sum_t[Cfg<NB>::kRing][kStageTiles][NB][4];      // sum of T over columns 8v .. 8v+7 of the tile, v = 0..3
    float red[kMmaWarps][NB][RABIT_TILE_ROWS];
    unsigned long long full[Cfg<NB>::kRing];
    unsigned long long empty[Cfg<NB>::kRing];
    unsigned int xmax_bits[NB];
    int abort_flag;
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
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
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
    unsigned int ns = 32;
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return; }
        __nanosleep(ns);                                   // a waiting warp must not eat the issue slots of the working ones
        if (ns < 256) ns *= 2;
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

// Even split of the tile positions: CTA c owns [c*q + min(c, r), (c+1)*q + min(c+1, r)).
__device__ __forceinline__ int range_lo(int c, int q, int r) { return c * q + min(c, r); }
// The CTA (counted inside its layer) that owns tile position p of that layer.
__device__ __forceinline__ int cta_of(int p, const GemvParams& P) {
    const int big = P.r * (P.q + 1);             // positions owned by the CTAs that have q+1 tiles
    return p < big ? fdiv(p, P.div_q1) : P.r + fdiv(p - big, P.div_q);
}

// sigma = 2^s with |h x| * sigma < 2^28 for every column; inv = 2^-s (NaN if the inputs are not finite).
__device__ __forceinline__ void choose_scale(unsigned int xmax_bits, float hmax, float& sigma, float& inv) {
    const float xm = __half2float(__ushort_as_half((unsigned short)xmax_bits));
    const float bound = xm * hmax;
    if (xmax_bits >= 0x7C00u || !(bound < __int_as_float(0x7F800000))) {      // inf / NaN anywhere in x or h
        sigma = 0.f; inv = __int_as_float(0x7FC00000);
        return;
    }
    if (bound == 0.f) { sigma = 1.f; inv = 1.f; return; }
    const int e = (__float_as_int(bound) >> 23) & 0xFF;                         // bound < 2^(e - 126)
    int s = 154 - e;                                                            // 28 - (e - 126)
    s = s > 120 ? 120 : s;
    sigma = __int_as_float((s + 127) << 23);
    inv = __int_as_float((127 - s) << 23);
}


// The 32 words of a tile's table row (per batch row) span all 32 banks, and the lanes of a builder warp write the
// same few words of eight different tiles at once: unrotated that is an 8-way bank conflict on every store.  Row j
// is therefore rotated by table_rot_pairs(j) word pairs, which spreads the eight tiles over distinct banks; a
// reader of tile j adds the same rotation to its pair index.
__device__ __forceinline__ int table_rot_pairs(int j) { return (j & 1) + ((j >> 1) & 3) * 4; }

// One lane's share of a stage: columns 8*bv .. +7 of tile j for ROWS batch rows starting at b0
// -> digit words in fragment order + the sum of T over those columns.
template <int NB, int ROWS>
__device__ __forceinline__ void build_rows(Smem<NB>& S, int slot, int j, int bv, int kk, int b0, const uint4& hraw,
                                           const uint4 (&xraw)[ROWS], const float (&sg_rows)[ROWS][RABIT_MAX_K]) {
    const uint32_t hw[4] = {hraw.x, hraw.y, hraw.z, hraw.w};
#pragma unroll
    for (int rr = 0; rr < ROWS; ++rr) {
        const float sg = kk == 0 ? sg_rows[rr][0] : (kk == 1 ? sg_rows[rr][1] : sg_rows[rr][2]);
        const uint32_t xw[4] = {xraw[rr].x, xraw[rr].y, xraw[rr].z, xraw[rr].w};
        int Tq[8];
#pragma unroll
        for (int c2 = 0; c2 < 4; ++c2) {
            const float2 hf = __half22float2(*reinterpret_cast<const __half2*>(&hw[c2]));
            const float2 xf = __half22float2(*reinterpret_cast<const __half2*>(&xw[c2]));
            Tq[2 * c2] = __float2int_rn(hf.x * xf.x * sg);
            Tq[2 * c2 + 1] = __float2int_rn(hf.y * xf.y * sg);
        }
        int tsum = 0;                        // |T| < 2^28, so eight of them fit
#pragma unroll
        for (int c = 0; c < 8; ++c) tsum += Tq[c];
        uint32_t* tbl = reinterpret_cast<uint32_t*>(&S.table[slot][j][(b0 + rr) * 16]);
        const int rot = table_rot_pairs(j) * 2;
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {  // columns 8*bv + 4*hlf .. +3  <->  group u = 2*bv + hlf
            const int u = 2 * bv + hlf;
            uint32_t X[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) X[c] = ((uint32_t)Tq[4 * hlf + c] + 0x80808080u) ^ 0x80808080u;   // bytes = balanced digits
            const uint32_t t0 = __byte_perm(X[0], X[1], 0x5140), t1 = __byte_perm(X[2], X[3], 0x5140);
            const uint32_t t2 = __byte_perm(X[0], X[1], 0x7362), t3 = __byte_perm(X[2], X[3], 0x7362);
            const int at = (u & 3) * 2 + (u >> 2) + rot;              // word pair index 4*digit + tq, rotated by the tile's offset
            tbl[at & 31] = __byte_perm(t0, t1, 0x5410);
            tbl[(at + 8) & 31] = __byte_perm(t0, t1, 0x7632);
            tbl[(at + 16) & 31] = __byte_perm(t2, t3, 0x5410);
            tbl[(at + 24) & 31] = __byte_perm(t2, t3, 0x7632);
        }
        S.sum_t[slot][j][b0 + rr][bv] = tsum;
    }
}

template <int NB>
__global__ void __launch_bounds__(Cfg<NB>::kThreads, Cfg<NB>::kMinBlocks)
rabit_gemv_mma_kernel(const __grid_constant__ GroupParams GP) {
    constexpr int kRing = Cfg<NB>::kRing;
    constexpr int kBuildWarps = Cfg<NB>::kBuildWarps;
    constexpr int kBuildRows = Cfg<NB>::kBuildRows;
    constexpr int kThreads = Cfg<NB>::kThreads;
    constexpr int kPairs = Cfg<NB>::kPairs;
    constexpr int kRed = (NB + 1) / 2;                   // (batch row, row) words one reducer thread owns: rows red_b0, red_b0 + 2, ...
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem<NB>& S = *reinterpret_cast<Smem<NB>*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nb = GP.nb;
    volatile int* abort_flag = &S.abort_flag;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(&S.full[s]), 1 + kBuildWarps);
            mbar_init(smem_u32(&S.empty[s]), kMmaWarps);
        }
        for (int b = 0; b < NB; ++b) S.xmax_bits[b] = 0;
        S.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // The layer this CTA works on (the loop body runs once; it is written as passes with a running stage
    // counter `it0`, so ring slots and barrier phases would simply continue if a CTA ever took several layers).
    int it0 = 0;
    bool first_pass = true;
    for (int li = 0; li < GP.n_layers; ++li) {
    const GemvParams& P = GP.layer[li];
    if ((int)blockIdx.x < P.cta0 || (int)blockIdx.x >= P.cta0 + P.n_cta) continue;
    const RabitGeom& G = P.G;
    const int C = G.n_ct;
    const int me = (int)blockIdx.x - P.cta0;                               // this CTA's index among the layer's CTAs
    const int lo = range_lo(me, P.q, P.r);                                 // its tile range, in the layer's own numbering
    const int n_tiles = range_lo(me + 1, P.q, P.r) - lo;
    const int n_stages = (n_tiles + kStageTiles - 1) / kStageTiles;
    if (!first_pass) {                                                     // every warp is done with the previous pass
        __syncthreads();
        if (tid < NB) S.xmax_bits[tid] = 0;
        __syncthreads();
    }

    // ---- everything that does not depend on the stream's past starts now: the first ring-full of
    //      weights, the first input scales of the builder lanes, the first output scales
    if (tid == kMmaThreads) {
        const int prefetched = n_stages < kRing ? n_stages : kRing;
        for (int i = 0; i < prefetched; ++i) {
            const int it = it0 + i, slot = it % kRing;
            if (it >= kRing) mbar_wait(smem_u32(&S.empty[slot]), ((it / kRing) - 1) & 1, abort_flag);
            const int tiles = min(kStageTiles, n_tiles - i * kStageTiles);
            const uint32_t bar = smem_u32(&S.full[slot]);
            mbar_expect_tx(bar, tiles * RABIT_TILE_BYTES);
            bulk_g2s(smem_u32(&S.bits[slot][0][0]), P.bits + ((size_t)lo + (size_t)i * kStageTiles) * RABIT_TILE_BYTES,
                     tiles * RABIT_TILE_BYTES, bar);
        }
    }
    // Conversion lanes: lane index bi = 0..63 of a warp pair takes tile bi >> 2 of a stage and columns
    // 8*(bi & 3) .. +7 of it.  The first kHeadStages stages are converted by the MMA warps (pair warp >> 1
    // takes stage warp >> 1, all batch rows), which have nothing else to do until a table exists; the
    // builder warps start behind them (with four builder warps each pair takes half of the batch rows).
    const int bi = ((warp & 1) << 5) | lane;
    const int bj = bi >> 2, bv = bi & 3;
    const int bw = warp - kMmaWarps;
    const int brow0 = (warp >= kMmaWarps && kBuildWarps == 4) ? (bw >> 1) * kBuildRows : 0;   // first batch row of a builder lane
    int pf_ct = 0, pf_k = 0;                          // (column tile, path) of the next prefetch / of the head stage
    int pf_stage = warp >= kMmaWarps ? kHeadStages : (warp >> 1);
    uint4 hq[kBuildAhead];
    {
        const int p0 = lo + pf_stage * kStageTiles + bj;
        const int st0 = fdiv(p0, P.div_c);
        pf_ct = p0 - st0 * C;
        pf_k = fmod(st0, P.div_k);
    }
    auto prefetch_h = [&](int d) {                   // input scales: static data, may be read before the wait
        hq[d] = make_uint4(0u, 0u, 0u, 0u);
        if (pf_stage < n_stages && pf_stage * kStageTiles + bj < n_tiles)
            hq[d] = __ldg(reinterpret_cast<const uint4*>(P.h + (size_t)pf_k * G.N + pf_ct * RABIT_TILE_COLS + 8 * bv));
    };
    // MMA thread state: first segment and its output scales
    int strip = fdiv(lo, P.div_c);
    int seg_end = min(n_tiles, (strip + 1) * C - lo);                       // relative to lo
    int rt = fdiv(strip, P.div_k);
    int k = strip - rt * G.K;
    const int red_b0 = (tid >> 7) & 1, red_r = tid & 127;                  // this thread reduces batch rows red_b0, red_b0 + 2, ... of row red_r
    const bool reducer = warp < kMmaWarps && red_b0 < nb;
    float gval = 0.f;
    prefetch_h(0);                                   // builder: its first stage; MMA warp: its head stage
    if (reducer) gval = __half2float(P.g[(size_t)k * G.Mp + rt * RABIT_TILE_ROWS + red_r]);

    if (first_pass) asm volatile("griddepcontrol.wait;" ::: "memory");
    first_pass = false;

    uint4 head_x[NB];                                // MMA warps: activations of the head stage, in flight during the max pass
#pragma unroll
    for (int b = 0; b < NB; ++b) head_x[b] = make_uint4(0u, 0u, 0u, 0u);
    const bool head_live = warp < kMmaWarps && pf_stage < n_stages && pf_stage * kStageTiles + bj < n_tiles;
    if (head_live) {
#pragma unroll
        for (int b = 0; b < NB; ++b)
            if (b < nb) head_x[b] = __ldg(reinterpret_cast<const uint4*>(P.x + (size_t)b * G.N + pf_ct * RABIT_TILE_COLS + 8 * bv));
    }

    // ---- largest |x| per batch row (fp16 bit patterns order like unsigned integers once the sign is cleared)
    {
        const int vec_per_row = G.N / 8;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (b >= nb) break;
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

    if (warp >= kMmaWarps) {
        // =========================== builder warps (and the copy issuer) ===========================
        const int j = bj;
        float sg_rows[kBuildRows][RABIT_MAX_K];
#pragma unroll
        for (int rr = 0; rr < kBuildRows; ++rr)
#pragma unroll
            for (int kk = 0; kk < RABIT_MAX_K; ++kk) {
                float inv;
                choose_scale(S.xmax_bits[brow0 + rr], kk < G.K ? G.hmax[kk] : 0.f, sg_rows[rr][kk], inv);
            }
        // a queue of kBuildAhead stages of raw inputs hides the load latency
        uint4 xq[kBuildAhead][kBuildRows];
        int kq[kBuildAhead];
        auto prefetch_x = [&](int d) {
            kq[d] = pf_k;
#pragma unroll
            for (int rr = 0; rr < kBuildRows; ++rr) xq[d][rr] = make_uint4(0u, 0u, 0u, 0u);
            if (pf_stage < n_stages && pf_stage * kStageTiles + bj < n_tiles) {
#pragma unroll
                for (int rr = 0; rr < kBuildRows; ++rr)
                    if (brow0 + rr < nb)
                        xq[d][rr] = __ldg(reinterpret_cast<const uint4*>(P.x + (size_t)(brow0 + rr) * G.N + pf_ct * RABIT_TILE_COLS + 8 * bv));
            }
            pf_stage += 1;
            pf_ct += kStageTiles;
            while (pf_ct >= C) { pf_ct -= C; pf_k = pf_k + 1 == G.K ? 0 : pf_k + 1; }
        };
#pragma unroll
        for (int d = 0; d < kBuildAhead; ++d) {          // the first stage's h part was fetched before the wait
            if (d > 0) prefetch_h(d);
            prefetch_x(d);
        }

        const bool issuer = tid == kMmaThreads;          // one lane issues the copies
        for (int i0 = kHeadStages; i0 < n_stages; i0 += kBuildAhead) {
#pragma unroll
            for (int d = 0; d < kBuildAhead; ++d) {
                const int i = i0 + d;
                if (i >= n_stages) break;
                const int slot = (it0 + i) % kRing;
                if (i >= kRing) {
                    mbar_wait(smem_u32(&S.empty[slot]), (((it0 + i) / kRing) - 1) & 1, abort_flag);
                    if (issuer) {
                        const int tiles = min(kStageTiles, n_tiles - i * kStageTiles);
                        const uint32_t bar = smem_u32(&S.full[slot]);
                        mbar_expect_tx(bar, tiles * RABIT_TILE_BYTES);
                        bulk_g2s(smem_u32(&S.bits[slot][0][0]), P.bits + ((size_t)lo + (size_t)i * kStageTiles) * RABIT_TILE_BYTES,
                                 tiles * RABIT_TILE_BYTES, bar);
                    }
                }
                build_rows<NB, kBuildRows>(S, slot, j, bv, kq[d], brow0, hq[d], xq[d], sg_rows);
                prefetch_h(d);
                prefetch_x(d);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&S.full[slot]));
            }
        }
    } else {
    // ======================================= MMA warps =======================================
    const int gq = lane >> 2, tq = lane & 3;
    const int w = warp;
    const int tbl_lane = (lane & 16) | ((lane + table_rot_pairs(w)) & 15);   // this warp's tiles are j = w and w + 8: same rotation
    float sig_inv[kRed][RABIT_MAX_K];         // 1 / sigma of the batch rows this thread reduces
    {
        float sg_all[NB][RABIT_MAX_K], inv_all[NB][RABIT_MAX_K];
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int kk = 0; kk < RABIT_MAX_K; ++kk)
                choose_scale(S.xmax_bits[b], kk < G.K ? G.hmax[kk] : 0.f, sg_all[b][kk], inv_all[b][kk]);
        if (pf_stage < n_stages) {            // head stage of this warp pair (its slot's earlier use ended with the previous pass)
            const int hslot = (it0 + pf_stage) % kRing;
            if (head_live) build_rows<NB, NB>(S, hslot, bj, bv, pf_k, 0, hq[0], head_x, sg_all);
            __syncwarp();
            if (lane == 0) mbar_arrive_n(smem_u32(&S.full[hslot]), kBuildWarps / 2);
        }
#pragma unroll
        for (int i = 0; i < kRed; ++i)
#pragma unroll
            for (int kk = 0; kk < RABIT_MAX_K; ++kk) {
                float v = inv_all[2 * i][kk];
                if (2 * i + 1 < NB && red_b0) v = inv_all[2 * i + 1 < NB ? 2 * i + 1 : 0][kk];
                sig_inv[i][kk] = v;
            }
    }

    int acc[kPairs][8][4];
    long long sum_t[NB];
#pragma unroll
    for (int jp = 0; jp < kPairs; ++jp)
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[jp][p][c] = 0;
#pragma unroll
    for (int b = 0; b < NB; ++b) sum_t[b] = 0;
    const int KC = G.K * C;
    bool red_in_use = false;

    // Segment end: sum the eight warps in shared memory, scale by g_k / sigma and store the partial
    // row sums; a stored word is visible to the finisher as soon as it differs from the sentinel.
    auto segment_flush = [&]() {
        if (red_in_use) bar_mma_warps();                                       // readers of the previous flush are done
        red_in_use = true;
        float st_f[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) {                                         // the four quarters live in lanes tq = 0..3
            long long t = sum_t[b];
            t += __shfl_xor_sync(0xffffffffu, t, 1);
            t += __shfl_xor_sync(0xffffffffu, t, 2);
            st_f[b] = __ll2float_rn(t);
        }
#pragma unroll
        for (int jp = 0; jp < kPairs; ++jp) {
            const int b = 2 * jp + (tq >> 1);                                  // lanes tq = 0,1 hold batch row 2*jp, lanes 2,3 row 2*jp + 1
            const float st = (2 * jp + 1 < NB && (tq >> 1)) ? st_f[2 * jp + 1 < NB ? 2 * jp + 1 : 0] : st_f[2 * jp];
#pragma unroll
            for (int p = 0; p < 8; ++p) {
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const float lo2 = fmaf(256.f, (float)acc[jp][p][2 * hf + 1], (float)acc[jp][p][2 * hf]);
                    const float hi2 = __shfl_xor_sync(0xffffffffu, lo2, 1);    // digits 2,3 live in the odd lane
                    if ((tq & 1) == 0 && b < NB) {
                        const float v = fmaf(65536.f, hi2, lo2);                // 2^p * sum_j b T
                        const float scale = __int_as_float((127 + 1 - p) << 23);    // 2^(1-p)
                        S.red[w][b][16 * p + gq + 8 * hf] = fmaf(-scale, v, st);    // sum_j T - 2 sum_j b T
                    }
                }
            }
        }
        bar_mma_warps();
        if (reducer) {
            const size_t seg_id = (size_t)me + strip;
#pragma unroll
            for (int i = 0; i < kRed; ++i) {
                const int b = red_b0 + 2 * i;
                if (b >= nb) break;
                float sum = 0.f;
#pragma unroll
                for (int ww = 0; ww < kMmaWarps; ++ww) sum += S.red[ww][b][red_r];
                const float inv = k == 0 ? sig_inv[i][0] : (k == 1 ? sig_inv[i][1] : sig_inv[i][2]);
                unsigned int bits = __float_as_uint(gval * (sum * inv));
                if (bits == kSentinel) bits = 0x7FFFFFFFu;                      // a NaN result must not look unwritten
                __stcg(reinterpret_cast<unsigned int*>(P.partial) + (seg_id * RABIT_PARTIAL_BATCH + b) * RABIT_TILE_ROWS + red_r, bits);
            }
        }
    };

    auto next_segment = [&]() {
        strip += 1;
        seg_end = min(n_tiles, seg_end + C);
        k += 1;
        if (k == G.K) { k = 0; rt += 1; }
        gval = 0.f;
        if (reducer) gval = __half2float(P.g[(size_t)k * G.Mp + rt * RABIT_TILE_ROWS + red_r]);
#pragma unroll
        for (int jp = 0; jp < kPairs; ++jp)
#pragma unroll
            for (int p = 0; p < 8; ++p)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[jp][p][c] = 0;
#pragma unroll
        for (int b = 0; b < NB; ++b) sum_t[b] = 0;
    };

    // One tile: 32 ANDs make the eight A fragments, each feeds kPairs MMAs (two batch rows each).
    auto one_tile = [&](int slot, int j) {
        const uint4 wv = S.bits[slot][j][lane];
        uint2 bb[kPairs];
#pragma unroll
        for (int jp = 0; jp < kPairs; ++jp) {
            bb[jp] = make_uint2(0u, 0u);
            if (2 * jp + (gq >> 2) < NB) bb[jp] = S.table[slot][j][jp * 32 + tbl_lane];
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) sum_t[b] += S.sum_t[slot][j][b][lane & 3];   // this lane's quarter of the tile
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const uint32_t mask = 0x01010101u << p;
            const uint32_t a0 = wv.x & mask, a1 = wv.y & mask, a2 = wv.z & mask, a3 = wv.w & mask;
#pragma unroll
            for (int jp = 0; jp < kPairs; ++jp) mma_u8s8(acc[jp][p], a0, a1, a2, a3, bb[jp].x, bb[jp].y);
        }
    };
    // This warp's tiles are rel = w, w + 8, ...: for NB <= 2 the two of a stage are taken together when both
    // lie in the current segment (the common case), which gives the scheduler two independent chains.
#pragma unroll 1
    for (int i = 0; i < n_stages; ++i) {
        const int slot = (it0 + i) % kRing;
        const int rel0 = i * kStageTiles + w, rel1 = rel0 + kMmaWarps;
        if (rel0 >= n_tiles) break;
        mbar_wait(smem_u32(&S.full[slot]), ((it0 + i) / kRing) & 1, abort_flag);
        if (NB <= 2 && rel1 < seg_end) {
            const uint4 wa = S.bits[slot][w][lane];
            const uint4 wb = S.bits[slot][w + kMmaWarps][lane];
            uint2 ba = make_uint2(0u, 0u), bb = make_uint2(0u, 0u);
            if (gq < 4 * NB) { ba = S.table[slot][w][tbl_lane]; bb = S.table[slot][w + kMmaWarps][tbl_lane]; }
#pragma unroll
            for (int b = 0; b < NB; ++b) sum_t[b] += S.sum_t[slot][w][b][lane & 3] + S.sum_t[slot][w + kMmaWarps][b][lane & 3];
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                const uint32_t mask = 0x01010101u << p;
                mma_u8s8(acc[0][p], wa.x & mask, wa.y & mask, wa.z & mask, wa.w & mask, ba.x, ba.y);
            }
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                const uint32_t mask = 0x01010101u << p;
                mma_u8s8(acc[0][p], wb.x & mask, wb.y & mask, wb.z & mask, wb.w & mask, bb.x, bb.y);
            }
        } else {
            while (rel0 >= seg_end) { segment_flush(); next_segment(); }
            one_tile(slot, w);
            if (rel1 < n_tiles) {
                while (rel1 >= seg_end) { segment_flush(); next_segment(); }
                one_tile(slot, w + kMmaWarps);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&S.empty[slot]));
    }
    while (true) {
        segment_flush();
        if (seg_end >= n_tiles) break;
        next_segment();
    }

    // ---- finish the row tiles whose last tile this CTA owns.  The two halves of the MMA threads share the
    //      paths (half = path & 1).  Thread (half, r) reads row r's word of every contributor's partial of its
    //      paths, for all batch rows at once (up to 8 contributors x NB words in flight), waits (bounded) while a
    //      word still holds the sentinel, restores the sentinel for the next call and adds in that fixed order.
    //      The halves meet in shared memory and the first one stores fp16.  No fence is involved: a partial
    //      word carries no other data with it.
    {
        constexpr size_t kStride = (size_t)RABIT_PARTIAL_BATCH * RABIT_TILE_ROWS;
        constexpr int kFan = 8;
        const int half = (tid >> 7) & 1;
        const bool two_halves = G.K > 1;
        for (int rt_f = fdiv(lo, P.div_kc); (rt_f + 1) * KC - 1 < lo + n_tiles; ++rt_f) {
            float part[NB];
#pragma unroll
            for (int b = 0; b < NB; ++b) part[b] = 0.f;
#pragma unroll 1
            for (int kk = half; kk < G.K; kk += 2) {
                const int s0 = (rt_f * G.K + kk) * C;
                const int c0 = cta_of(s0, P), c1 = cta_of(s0 + C - 1, P);
                unsigned int* src = reinterpret_cast<unsigned int*>(P.partial) +
                                    ((size_t)c0 + (size_t)rt_f * G.K + kk) * kStride + red_r;
#pragma unroll 1
                for (int c = c0; c <= c1; c += kFan) {
                    unsigned int v[NB][kFan];
#pragma unroll
                    for (int b = 0; b < NB; ++b)
#pragma unroll
                        for (int u = 0; u < kFan; ++u) {
                            v[b][u] = 0u;
                            if (b < nb && c + u <= c1)
                                asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v[b][u]) : "l"(src + u * kStride + b * RABIT_TILE_ROWS) : "memory");
                        }
#pragma unroll
                    for (int u = 0; u < kFan; ++u) {
                        if (c + u > c1) break;
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            if (b >= nb) break;
                            unsigned int* word = src + u * kStride + b * RABIT_TILE_ROWS;
                            if (v[b][u] == kSentinel) {
                                const long long t0 = clock64();
                                do {
                                    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v[b][u]) : "l"(word) : "memory");
                                    if (v[b][u] != kSentinel) break;
                                    if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; break; }
                                } while (true);
                            }
                            __stcg(word, kSentinel);
                            part[b] += __uint_as_float(v[b][u]);
                        }
                    }
                    src += kFan * kStride;
                }
            }
            if (two_halves) {
                bar_mma_warps();                                               // the last flush's readers are done with S.red
                if (half) {
#pragma unroll
                    for (int b = 0; b < NB; ++b) S.red[0][b][red_r] = part[b];
                }
                bar_mma_warps();
            }
            if (!half) {
                const int row = rt_f * RABIT_TILE_ROWS + red_r;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b >= nb) break;
                    const float sum = two_halves ? part[b] + S.red[0][b][red_r] : part[b];
                    if (row < G.M) P.y[(size_t)b * G.M + row] = __float2half_rn(sum);
                }
            }
        }
    }
    }                                                                          // MMA warps
    it0 += n_stages;
    }                                                                          // passes

    __syncthreads();                                                           // abort_flag of every warp is final
    if (*abort_flag && tid == kMmaThreads) {
        // make sure no bulk copy is still in flight towards this CTA's shared memory
        for (int it = max(0, it0 - kRing); it < it0; ++it) {
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&S.full[it % kRing]), (it / kRing) & 1))
                if (clock64() - t0 > kWaitLimitCycles) break;
        }
        for (int l = 0; l < GP.n_layers; ++l) atomicExch(GP.status[l], 1u);
    }
}

}  // namespace

bool rabit_gemv_mma_supports(const rabit_layer& L, int batch) {
    const long long tiles = (long long)L.geom.n_rt * L.geom.K * L.geom.n_ct;
    return batch >= 1 && batch <= RABIT_MAX_GEMV_BATCH && tiles < (1LL << 31);
}

template <int NB>
static cudaError_t launch_nb(const GroupParams& GP, int grid, int device, cudaStream_t stream) {
    static bool attr_done[64] = {false};                                          // function attributes are per device
    const int dev_slot = device >= 0 && device < 64 ? device : 0;
    const size_t smem = sizeof(Smem<NB>);
    if (!attr_done[dev_slot] || dev_slot != device) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemv_mma_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done[dev_slot] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(Cfg<NB>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rabit_gemv_mma_kernel<NB>, GP);
}

int rabit_gemv_mma_max_group() { return kMaxGroup; }

// Largest number of batch rows one launch takes (the dispatcher walks the batch in such chunks).
int rabit_gemv_mma_max_rows() { return 4; }

bool rabit_gemv_mma_group_supports(const rabit_layer* const* layers, int n_layers, int batch) {
    if (n_layers < 1 || n_layers > kMaxGroup || batch < 1 || batch > RABIT_MAX_GEMV_BATCH) return false;
    long long tiles = 0;
    for (int l = 0; l < n_layers; ++l) tiles += (long long)layers[l]->geom.n_rt * layers[l]->geom.K * layers[l]->geom.n_ct;
    return tiles < (1LL << 31);
}

// One launch for n_layers independent layers and 1..4 batch rows (x_l: [batch][N_l], y_l: [batch][M_l]).
cudaError_t rabit_launch_gemv_mma_group(const rabit_layer* const* layers, int n_layers, const void* const* xs, void* const* ys,
                                        int batch, cudaStream_t stream) {
    if (batch < 1 || batch > 4) return cudaErrorInvalidValue;
    GroupParams GP;
    GP.n_layers = n_layers;
    for (int l = 0; l < kMaxGroup; ++l) GP.status[l] = layers[l < n_layers ? l : 0]->d_status;
    GP.nb = batch;
    long long total = 0;
    for (int l = 0; l < n_layers; ++l) {
        const rabit_layer& L = *layers[l];
        GemvParams& P = GP.layer[l];
        P.G = L.geom;
        P.bits = reinterpret_cast<const unsigned char*>(L.d_bits);
        P.g = (const __half*)L.d_g;
        P.h = (const __half*)L.d_h;
        P.x = (const __half*)xs[l];
        P.y = (__half*)ys[l];
        P.partial = L.d_partial;
        P.n_tiles = L.geom.n_rt * L.geom.K * L.geom.n_ct;
        P.div_c = make_fastdiv((unsigned int)L.geom.n_ct);
        P.div_k = make_fastdiv((unsigned int)L.geom.K);
        P.div_kc = make_fastdiv((unsigned int)(L.geom.K * L.geom.n_ct));
        total += P.n_tiles;
    }
    const int sms = layers[0]->sm_count > 0 ? layers[0]->sm_count : 148;
    long long grid_ll = (long long)(batch <= 2 ? 2 : 1) * sms;   // as many CTAs as are resident at once (two per SM up to two batch rows)
    if (grid_ll > RABIT_MAX_GRID) grid_ll = RABIT_MAX_GRID;
    if (grid_ll > total) grid_ll = total;
    if (grid_ll < n_layers) grid_ll = n_layers;
    const int grid = (int)grid_ll;
    // share the CTAs out in proportion to the tiles: floor first (at least one each, at most one per tile),
    // then hand the rest to the layers with the most tiles per CTA
    int given = 0;
    for (int l = 0; l < n_layers; ++l) {
        GemvParams& P = GP.layer[l];
        long long n = (long long)grid * P.n_tiles / total;
        if (n < 1) n = 1;
        if (n > P.n_tiles) n = P.n_tiles;
        P.n_cta = (int)n;
        given += P.n_cta;
    }
    while (given > grid) {                                   // the "at least one" floor can overshoot: take from the best-served layer
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (GP.layer[l].n_cta > 1 && (best < 0 || (long long)GP.layer[l].n_tiles * GP.layer[best].n_cta < (long long)GP.layer[best].n_tiles * GP.layer[l].n_cta)) best = l;
        if (best < 0) break;
        GP.layer[best].n_cta -= 1; given -= 1;
    }
    while (given < grid) {
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (GP.layer[l].n_cta < GP.layer[l].n_tiles && (best < 0 || (long long)GP.layer[l].n_tiles * GP.layer[best].n_cta > (long long)GP.layer[best].n_tiles * GP.layer[l].n_cta)) best = l;
        if (best < 0) break;
        GP.layer[best].n_cta += 1; given += 1;
    }
    int c0 = 0;
    for (int l = 0; l < n_layers; ++l) {
        GemvParams& P = GP.layer[l];
        P.cta0 = c0;
        c0 += P.n_cta;
        P.q = P.n_tiles / P.n_cta;
        P.r = P.n_tiles % P.n_cta;
        P.div_q = make_fastdiv((unsigned int)P.q);
        P.div_q1 = make_fastdiv((unsigned int)P.q + 1u);
    }
    for (int l = n_layers; l < kMaxGroup; ++l) { GP.layer[l] = GP.layer[0]; GP.layer[l].n_cta = 0; }
    const int launch_grid = c0;
    const int device = layers[0]->device;
    if (batch == 1) return launch_nb<1>(GP, launch_grid, device, stream);
    if (batch == 2) return launch_nb<2>(GP, launch_grid, device, stream);
    return launch_nb<4>(GP, launch_grid, device, stream);
}

cudaError_t rabit_launch_gemv_mma(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    const rabit_layer* one = &L;
    return rabit_launch_gemv_mma_group(&one, 1, &x, &y, batch, stream);
}
