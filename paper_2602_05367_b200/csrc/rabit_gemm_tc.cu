// Large-batch form of the layer on the tcgen05 tensor cores (batch > 16, and smaller batches where it is cheaper).
//
//   y[b][i] = sum_k g_k[i] * sum_j (B_k[i][j] * h_k[j]) * x[b][j]                       (Section 4.1, Eq. 2)
//
// For many activation rows the layer is a dense contraction.  Per path k the A operand is the
// sign tile with the input scale folded in, A_k[i][j] = +-h_k[j]: an fp16 value with its sign
// bit flipped by the weight bit, so the expansion is exact.  The B operand is x itself (fp16,
// loaded by TMA, shared by all paths), products are exact in fp32 and accumulate in fp32 in
// tensor memory; the epilogue applies g_k, adds the paths and rounds once to fp16.
//
// One CTA per SM, persistent over output tiles of 128 weight rows x 256 batch rows:
//   warp 0      producer: per 64-column step, one TMA tile of x (128B swizzle) plus bulk copies of
//               the packed sign tiles and the h slices of that step, into a ring of up to 8 steps
//   warp 1      allocates tensor memory, issues tcgen05.mma (M=128, N=256, K=16, kind::f16) for every
//               path into that path's accumulator, commits stages back to the producer
//   warps 2..9  expand packed signs to +-h fp16 in the canonical K-major 128B-swizzled layout (two A stages), then
//               (same warps) read the accumulators with tcgen05.ld for the epilogue
// Every wait is bounded; on a time-out the CTA sets the status word, skips the remaining waits,
// frees its tensor memory and returns.
//
// Two more forms of the same kernel:
//   * split contraction: when a launch has fewer tiles than half the SMs, clusters of 2, 4 or 8 CTAs share the 64-column
//     steps of one tile and add their partial results through distributed shared memory (fixed order, no atomics);
//     tiles left over beyond whole waves of the persistent form are launched that way too;
//   * DEQ: the expander forms the dequantised weight sum_k +-g_k h_k in fp16 and one contraction serves all paths
//     (rabit_set_variant 4; half the tensor work, one fp16 rounding per partial product and weight).
#include <cuda.h>
#include <cuda_fp16.h>

#include "rabit_internal.h"

namespace {

constexpr int kTileM = 128;                 // weight rows per output tile
// batch rows per output tile (MMA N) and paths: TB = 256 with up to 2 paths or TB = 128 with 3 (template parameters):
// paths x TB accumulator columns must fit the 512 columns of tensor memory
constexpr int kStepCols = 64;               // input columns per pipeline step (128 bytes of fp16: one swizzle row)
// Expanded A tiles: double-buffered, or four stages where there is one tile per step (KA == 1, the dequantised form),
// whose expander warps work as two groups on alternate steps.
__host__ __device__ constexpr int a_stages(int ka) { return ka == 1 ? 4 : 2; }
constexpr int kExpandWarps = 8;
constexpr int kThreads = (2 + kExpandWarps) * 32;
constexpr long long kWaitLimitCycles = 1LL << 31;

// What the copy engine brings per 64-column step (deep ring: it hides the global-memory latency) ...
template <int TB, int KP>
struct __align__(1024) InStage {
    __half x[TB * kStepCols];                         // 8..32 KB, swizzled by TMA
    uint4 bits[KP][2][32];                            // packed sign tiles: 2 column tiles per step per path
    __half h[KP][kStepCols];
};
// ... and what the expander warps make of it (two steps: one being multiplied, one being written).
template <int KA>
struct __align__(1024) AStage {
    __half a[KA][kTileM * kStepCols];                 // 16 KB per expanded operand tile (one per path, or one in all), swizzled
};

// Input-ring depth: as many steps as fit beside the A ring in 222 KB, at most 8.
template <int TB, int KP, int KA>
struct GemmCfg {
    static constexpr int kInBytes = (int)sizeof(InStage<TB, KP>);
    static constexpr int kFit = (222 * 1024 - a_stages(KA) * (int)sizeof(AStage<KA>)) / kInBytes;
    static constexpr int kStages = kFit > 8 ? 8 : kFit;
};

template <int TB, int KP, int KA>
struct Smem {
    AStage<KA> astage[a_stages(KA)];
    InStage<TB, KP> stage[GemmCfg<TB, KP, KA>::kStages];
    unsigned long long full[8];                       // TMA bytes landed (x, bits, h)
    unsigned long long empty[8];                      // MMAs that read the input stage retired
    unsigned long long a_ready[4];                    // expanders done (a_stages(KA) in use)
    unsigned long long a_empty[4];                    // MMAs that read the A stage retired
    unsigned long long acc_ready;                     // all MMAs of the tile retired
    unsigned long long acc_empty;                     // epilogue has read the accumulators
    uint32_t tmem_base;
    int abort_flag;
};

struct GemmParams {
    RabitGeom G;
    const unsigned char* bits;
    const __half* g;
    const __half* h;
    __half* y;
    unsigned int* status;
    int batch;
    int n_bt;                                         // batch tiles
    int tile_lo, tile_hi;                             // this launch covers tiles tile_lo .. tile_hi - 1 of the n_rt * n_bt
    int split;                                        // CTAs (one cluster) that share the contraction of one tile: 1, 2, 4 or 8
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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes, 128-byte swizzle,
// 8-row groups 1024 bytes apart; descriptor version 1.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    uint64_t d = (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                        // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset
    d |= (uint64_t)1 << 46;                        // descriptor version
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B fp16, both K-major, N = batch tile, M = 128.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}

// DEQ = false: one operand tile +-h_k and one accumulator per path (exact products, g_k applied in the epilogue).
// DEQ = true:  one operand tile holding the dequantised weight sum_k +-g_k h_k rounded to fp16 and one accumulator:
//              half the tensor-core work and half the shared-memory operand traffic, at the price of one fp16
//              rounding per partial product and per weight (relative 2^-11 each).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t cluster_map(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

template <int TB, int KP, bool DEQ>
__global__ void __launch_bounds__(kThreads, 1)
rabit_gemm_tc_kernel(const GemmParams P, const __grid_constant__ CUtensorMap x_map) {
    constexpr int KA = DEQ ? 1 : KP;
    using Stage = InStage<TB, KP>;
    using Smem = Smem<TB, KP, KA>;
    constexpr int kStages = GemmCfg<TB, KP, KA>::kStages;
    constexpr int kAStages = a_stages(KA);
    constexpr int kGroupWarps = DEQ ? kExpandWarps / 2 : kExpandWarps;   // expander warps that build one step's operand
    constexpr int kTileB = TB;
    constexpr int kMaxPaths = KP;
    extern __shared__ unsigned char smem_raw[];
    // the swizzled operand tiles need 1024-byte alignment; the launch reserves the slack
    Smem& S = *reinterpret_cast<Smem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    const RabitGeom& G = P.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = G.K;
    const int n_steps = (G.N + kStepCols - 1) / kStepCols;        // N % 32 == 0: the last step may hold one column tile only
    volatile int* abort_flag = &S.abort_flag;
    // Split contraction: the `split` CTAs of a cluster work on the same output tile, rank r taking the r-th part of
    // the 64-column steps; their partial results meet through distributed shared memory at the end.  Each CTA
    // then has exactly one tile.  split == 1 is the persistent form (a CTA walks tiles blockIdx.x, +gridDim.x, ...).
    const int split = P.split;
    uint32_t crank = 0;
    if (split > 1) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    const int t_first = P.tile_lo + (split > 1 ? (int)blockIdx.x / split : (int)blockIdx.x);
    const int t_stride = split > 1 ? P.tile_hi - P.tile_lo : (int)gridDim.x;
    const int s_lo = split > 1 ? (int)((long long)n_steps * crank / split) : 0;
    const int s_hi = split > 1 ? (int)((long long)n_steps * (crank + 1) / split) : n_steps;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&S.full[s]), 1);
            mbar_init(smem_u32(&S.empty[s]), 1);
        }
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(smem_u32(&S.a_ready[s]), kGroupWarps);
            mbar_init(smem_u32(&S.a_empty[s]), 1);
        }
        mbar_init(smem_u32(&S.acc_ready), 1);
        mbar_init(smem_u32(&S.acc_empty), kExpandWarps);
        S.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                            // one warp allocates all 512 columns of tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&S.tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = S.tmem_base;

    if (warp == 0) {
        // ===================================== producer =====================================
        if (lane == 0) {
            int it = 0;                                          // global step counter of this CTA
            for (int t = t_first; t < P.tile_hi; t += t_stride) {
                const int rt = t / P.n_bt, bt = t % P.n_bt;
                for (int s = s_lo; s < s_hi; ++s, ++it) {
                    const int slot = it % kStages;
                    if (it >= kStages) mbar_wait(smem_u32(&S.empty[slot]), ((it / kStages) - 1) & 1, abort_flag);
                    Stage& st = S.stage[slot];
                    const int cts = min(2, G.n_ct - 2 * s);      // column tiles in this step
                    const uint32_t bar = smem_u32(&S.full[slot]);
                    const uint32_t bytes = (uint32_t)(kTileB * kStepCols * 2) + (uint32_t)K * cts * (RABIT_TILE_BYTES + RABIT_TILE_COLS * 2);
                    mbar_expect_tx(bar, bytes);
                    tma_load_2d(smem_u32(st.x), &x_map, s * kStepCols, bt * kTileB, bar);
                    for (int k = 0; k < K; ++k) {
                        bulk_g2s(smem_u32(&st.bits[k][0][0]), P.bits + rabit_tile_pos(G, rt, k, 2 * s) * RABIT_TILE_BYTES,
                                 cts * RABIT_TILE_BYTES, bar);
                        bulk_g2s(smem_u32(&st.h[k][0]), P.h + (size_t)k * G.N + (size_t)s * kStepCols, cts * RABIT_TILE_COLS * 2, bar);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ===================================== MMA issuer =====================================
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(kTileB);
            int it = 0, tile_i = 0;
            for (int t = t_first; t < P.tile_hi; t += t_stride, ++tile_i) {
                if (tile_i > 0) mbar_wait(smem_u32(&S.acc_empty), (tile_i - 1) & 1, abort_flag);   // epilogue has drained the accumulators
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int s = s_lo; s < s_hi; ++s, ++it) {
                    const int slot = it % kStages, aslot = it % kAStages;
                    mbar_wait(smem_u32(&S.full[slot]), (it / kStages) & 1, abort_flag);
                    mbar_wait(smem_u32(&S.a_ready[aslot]), (it / kAStages) & 1, abort_flag);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    Stage& st = S.stage[slot];
                    const int ksub = min(2, G.n_ct - 2 * s) * 2;                                   // MMAs of K = 16 in this step (2 per column tile)
                    const uint64_t bdesc = umma_desc(smem_u32(st.x));
                    const int n_acc = DEQ ? 1 : K;
                    for (int k = 0; k < n_acc; ++k) {
                        const uint64_t adesc = umma_desc(smem_u32(S.astage[aslot].a[k]));
                        for (int kk = 0; kk < ksub; ++kk)
                            umma_f16(tmem_base + (uint32_t)k * kTileB, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc,
                                     (s > s_lo || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&S.empty[slot]));                                         // frees both stages when these MMAs retire
                    umma_commit(smem_u32(&S.a_empty[aslot]));
                }
                umma_commit(smem_u32(&S.acc_ready));
            }
        }
    } else {
        // ============================ expanders, then epilogue ============================
        const int e = warp - 2;                               // 0..7
        const int quarter = warp & 3;                         // tensor-memory lanes this warp may read: 32*quarter .. +31
        const int col_half = e >> 2;                          // which half of the tile's batch columns this warp drains
        // expander role of this thread, the same in every step: one packed word position per path
        // (dequantised form: the warps are two groups that take alternate steps; a thread then covers both column tiles of its step)
        const int grp = e >> 2;
        // Exact form: warp e takes the words of packed lanes gq = e; its lanes spread over both column tiles, the two column
        // halves, the four tq and the two row halves, so that one 8-byte store per lane covers two whole 128-byte rows of
        // the swizzled tile.  An 8-byte store is served half a warp at a time: lanes 0..15 must fill ONE row (16 x 8 bytes,
        // all 32 banks once), so the row half is chosen by lane bit 4 and the position in the row by bits 0..3 (with the
        // row half in bit 0 every half warp wrote two half rows on the same banks: 25 M of 42 M wavefronts were conflicts).
        // Dequantised form: a group has four warps, so warp e & 3 takes gq = 2*(e & 3) and 2*(e & 3) + 1 in turn.
        const int x_ct2 = (lane >> 3) & 1;
        const int x_a = 2 * ((lane >> 2) & 1) + (lane >> 4);
        const int x_tq = lane & 3;
        const int x_gq = DEQ ? 2 * (e & 3) : e;
        const int x_l = 4 * x_gq + x_tq;
        const int x_hoff = 32 * x_ct2 + 16 * (x_a >> 1) + 4 * x_tq;
        const uint32_t x_aoff = (uint32_t)((x_gq + 8 * (x_a & 1)) * 128 + (((4 * x_ct2 + 2 * (x_a >> 1) + (x_tq >> 1)) ^ x_gq) << 4) + 8 * (x_tq & 1));
        int it = 0, tile_i = 0;
        for (int t = t_first; t < P.tile_hi; t += t_stride, ++tile_i) {
            const int rt = t / P.n_bt, bt = t % P.n_bt;
            __half2 g_rows[kMaxPaths][2][8];                  // DEQ: output scales of this thread's 2 x 8 rows, both halves alike
            if (DEQ) {
#pragma unroll
                for (int k = 0; k < kMaxPaths; ++k)
#pragma unroll
                    for (int gi = 0; gi < 2; ++gi)
#pragma unroll
                        for (int p = 0; p < 8; ++p) {
                            const int r = rt * kTileM + 16 * p + x_gq + gi + 8 * (x_a & 1);
                            g_rows[k][gi][p] = __half2half2((k < K && r < G.Mp) ? P.g[(size_t)k * G.Mp + r] : __float2half(0.f));
                        }
            }
            for (int s = s_lo; s < s_hi; ++s, ++it) {
                if (DEQ && (it & 1) != grp) continue;                 // the other group's step
                const int slot = it % kStages, aslot = it % kAStages;
                mbar_wait(smem_u32(&S.full[slot]), (it / kStages) & 1, abort_flag);
                if (it >= kAStages) mbar_wait(smem_u32(&S.a_empty[aslot]), ((it / kAStages) - 1) & 1, abort_flag);
                Stage& st = S.stage[slot];
                AStage<KA>& ast = S.astage[aslot];
                const int cts = min(2, G.n_ct - 2 * s);
                if (DEQ) {
                    // dequantised operand: for each of this thread's 8 rows and 4 columns, sum_k +-g_k[row] h_k[col],
                    // accumulated from the last (smallest) path to the first with one fused multiply-add per path
#pragma unroll
                    for (int gi = 0; gi < 2; ++gi) {
                        const int gq = x_gq + gi, l = x_l + 4 * gi;
                        uint32_t u01[kMaxPaths], u23[kMaxPaths];
                        uint2 hv[kMaxPaths];
#pragma unroll
                        for (int k = 0; k < kMaxPaths; ++k) {
                            uint32_t w = 0;
                            hv[k] = make_uint2(0u, 0u);
                            if (k < K && x_ct2 < cts) {
                                w = reinterpret_cast<const uint32_t*>(&st.bits[k][x_ct2][l])[x_a];
                                hv[k] = *reinterpret_cast<const uint2*>(&st.h[k][x_hoff]);
                            }
                            u01[k] = __byte_perm(w, 0u, 0x1404);
                            u23[k] = __byte_perm(w, 0u, 0x3424);
                        }
                        const uint32_t aoff = (uint32_t)((gq + 8 * (x_a & 1)) * 128 + (((4 * x_ct2 + 2 * (x_a >> 1) + (x_tq >> 1)) ^ gq) << 4) + 8 * (x_tq & 1));
                        const uint32_t dst = smem_u32(ast.a[0]) + aoff;
#pragma unroll
                        for (int p = 0; p < 8; ++p) {
                            __half2 s01 = __float2half2_rn(0.f), s23 = __float2half2_rn(0.f);
#pragma unroll
                            for (int k = kMaxPaths - 1; k >= 0; --k) {
                                if (k >= K) continue;
                                const uint32_t ox = hv[k].x ^ ((u01[k] << (7 - p)) & 0x80008000u);   // +-h: sign flipped where the weight is -1
                                const uint32_t oy = hv[k].y ^ ((u23[k] << (7 - p)) & 0x80008000u);
                                s01 = __hfma2(g_rows[k][gi][p], *reinterpret_cast<const __half2*>(&ox), s01);
                                s23 = __hfma2(g_rows[k][gi][p], *reinterpret_cast<const __half2*>(&oy), s23);
                            }
                            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(dst + p * 16 * 128), "r"(*reinterpret_cast<const uint32_t*>(&s01)),
                                         "r"(*reinterpret_cast<const uint32_t*>(&s23)) : "memory");
                        }
                    }
                } else
                {
                // This thread's packed word (column tile ct2, lane l, word a) of every path: rows 16*p + gq + 8*(a&1),
                // columns 32*ct2 + 16*(a>>1) + 4*tq + c (c = 0..3) = bytes 0..7 of 16-byte chunk 4*ct2 + 2*(a>>1) + (tq>>1)
                // of the row (second half if tq is odd); the chunk is XOR-swizzled with the row.
#pragma unroll
                for (int k = 0; k < kMaxPaths; ++k) {
                    if (k >= K) break;
                    uint32_t w = 0;
                    uint2 hv = make_uint2(0u, 0u);
                    if (x_ct2 < cts) {
                        w = reinterpret_cast<const uint32_t*>(&st.bits[k][x_ct2][x_l])[x_a];
                        hv = *reinterpret_cast<const uint2*>(&st.h[k][x_hoff]);
                    }
                    const uint32_t u01 = __byte_perm(w, 0u, 0x1404);                       // bytes [0, c0, 0, c1]: bit p of a column -> bit 8+p / 24+p
                    const uint32_t u23 = __byte_perm(w, 0u, 0x3424);                       // bytes [0, c2, 0, c3]
                    const uint32_t dst = smem_u32(ast.a[k]) + x_aoff;
#pragma unroll
                    for (int p = 0; p < 8; ++p) {
                        const uint32_t ox = hv.x ^ ((u01 << (7 - p)) & 0x80008000u);       // flip the fp16 sign where the weight is -1
                        const uint32_t oy = hv.y ^ ((u23 << (7 - p)) & 0x80008000u);
                        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(dst + p * 16 * 128), "r"(ox), "r"(oy) : "memory");
                    }
                }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");              // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&S.a_ready[aslot]));
            }
            if (split > 1) break;                              // the cluster's epilogue follows the role branches
            // ---- epilogue of this tile
            mbar_wait(smem_u32(&S.acc_ready), tile_i & 1, abort_flag);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int row = rt * kTileM + quarter * 32 + lane;
            float gk[kMaxPaths];
#pragma unroll
            for (int k = 0; k < kMaxPaths; ++k) gk[k] = (k < K && row < G.Mp) ? __half2float(P.g[(size_t)k * G.Mp + row]) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < kTileB / 2; c0 += 32) {
                const int col = col_half * (kTileB / 2) + c0;
                if (bt * kTileB + col >= P.batch) break;                          // batch rows beyond the batch: nothing to drain or store
                float v[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] = 0.f;
#pragma unroll
                for (int k = 0; k < kMaxPaths; ++k) {
                    if (k >= (DEQ ? 1 : K)) break;
                    uint32_t d[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(k * kTileB + col), d);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int c = 0; c < 32; ++c) v[c] = DEQ ? __uint_as_float(d[c]) : fmaf(gk[k], __uint_as_float(d[c]), v[c]);
                }
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int b = bt * kTileB + col + c;
                    if (b < P.batch && row < G.M) P.y[(size_t)b * G.M + row] = __float2half_rn(v[c]);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&S.acc_empty));
        }
    }

    if (split > 1) {
        // ---- epilogue of a split tile.  Every CTA of the cluster holds a partial 128 x TB result in tensor memory.
        //      CTA `o` finishes the batch columns [o*W, (o+1)*W), W = TB / split: all CTAs send it their slice of
        //      those columns (already scaled by g_k and summed over the paths), into its receive buffer
        //      recv[source rank][column][row] (the input ring's memory: nothing uses it once every CTA's MMAs have
        //      retired, which the first cluster barrier establishes).  After the second barrier each CTA adds the
        //      slices it received in rank order and stores fp16.
        const int rt = t_first / P.n_bt, bt = t_first % P.n_bt;
        const int W = kTileB / split;
        if (warp >= 2) {
            mbar_wait(smem_u32(&S.acc_ready), 0, abort_flag);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        __syncwarp();
        cluster_sync_all();
        float* recv = reinterpret_cast<float*>(&S.stage[0]);
        if (warp >= 2) {
            const int e = warp - 2, quarter = warp & 3, col_half = e >> 2;
            const int r_in = quarter * 32 + lane;                                  // row of the tile this thread reads from tensor memory
            const int row = rt * kTileM + r_in;
            float gk[kMaxPaths];
#pragma unroll
            for (int k = 0; k < kMaxPaths; ++k) gk[k] = (k < K && row < G.Mp) ? __half2float(P.g[(size_t)k * G.Mp + row]) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < kTileB / 2; c0 += 32) {
                const int col = col_half * (kTileB / 2) + c0;
                if (bt * kTileB + col >= P.batch) break;                          // batch rows beyond the batch: nothing to drain or store
                float v[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] = 0.f;
#pragma unroll
                for (int k = 0; k < kMaxPaths; ++k) {
                    if (k >= (DEQ ? 1 : K)) break;
                    uint32_t d[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(k * kTileB + col), d);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int c = 0; c < 32; ++c) v[c] = DEQ ? __uint_as_float(d[c]) : fmaf(gk[k], __uint_as_float(d[c]), v[c]);
                }
                const int owner = col / W, lc0 = col % W;                         // 32 divides W: the chunk has one owner
                const uint32_t dst = cluster_map(smem_u32(recv + ((size_t)crank * W + lc0) * kTileM + r_in), (uint32_t)owner);
#pragma unroll
                for (int c = 0; c < 32; ++c) st_cluster_f32(dst + (uint32_t)(c * kTileM * 4), v[c]);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
        __syncwarp();
        cluster_sync_all();
        if (warp >= 2) {
            const int et = (warp - 2) * 32 + lane;
            const int r_in = et & (kTileM - 1), hh = et >> 7;                     // two threads per row, half of the W columns each
            const int row = rt * kTileM + r_in;
            for (int lc = hh * (W / 2); lc < (hh + 1) * (W / 2); ++lc) {
                float sum = 0.f;
                for (int src = 0; src < split; ++src) sum += recv[((size_t)src * W + lc) * kTileM + r_in];
                const int b = bt * kTileB + (int)crank * W + lc;
                if (b < P.batch && row < G.M) P.y[(size_t)b * G.M + row] = __float2half_rn(sum);
            }
        }
    }

    // ---- teardown: everyone meets, then the allocating warp frees the tensor memory
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
    if (tid == 0 && *abort_flag) atomicExch(P.status, 1u);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

// CTAs per cluster that share one tile's contraction: doubled while every CTA keeps at least 8 steps, the
// slices stay 32 columns wide and the whole grid is resident at once.
// Clusters of 2 / 4 / 8 of these one-per-SM CTAs that the device places at once (index log2 of the size); cautious
// defaults until a launch has asked the runtime (a cluster must sit inside one GPC, so 8-CTA clusters are few).
static int g_cluster_limit[4] = {1 << 30, 64, 28, 8};

static int choose_split(int n_tiles, int N, int tb, int sms) {
    const int n_steps = (N + kStepCols - 1) / kStepCols;
    int best = 1;
    for (int lg = 1; lg <= 3; ++lg) {
        const int split = 1 << lg;
        if (n_tiles * split <= sms && n_tiles <= g_cluster_limit[lg] && n_steps / split >= 8 && tb / split >= 32) best = split;
    }
    return best;
}

// Estimated duration (us) of the exact-expansion GEMM on B200, a fit to measurements at batch <= 64:
// 11 + 0.75 * (K/2) per 64-column step of the busiest CTA, times the number of waves.
double rabit_gemm_tc_estimate_us(const rabit_layer& L, int batch) {
    const int sms = L.sm_count > 0 ? L.sm_count : 148;
    const int tb = L.geom.K > 2 ? 128 : 256;
    const int n_tiles = L.geom.n_rt * ((batch + tb - 1) / tb);
    const int split = choose_split(n_tiles, L.geom.N, tb, sms);
    const int n_steps = (L.geom.N + kStepCols - 1) / kStepCols;
    const double waves = split > 1 ? 1.0 : (double)((n_tiles + sms - 1) / sms);
    return waves * (11.0 + 0.375 * L.geom.K * (double)((n_steps + split - 1) / split));
}

bool rabit_gemm_tc_supports(const rabit_layer& L, int batch) {
    return batch >= 1 && L.geom.K <= 3 && encode_tiled_fn() != nullptr;
}

template <int TB, int KP, bool DEQ>
static cudaError_t launch_gemm(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)L.geom.N, (cuuint64_t)batch};
    const cuuint64_t strides[1] = {(cuuint64_t)L.geom.N * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kStepCols, (cuuint32_t)TB};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;

    GemmParams P;
    P.G = L.geom;
    P.bits = reinterpret_cast<const unsigned char*>(L.d_bits);
    P.g = (const __half*)L.d_g;
    P.h = (const __half*)L.d_h;
    P.y = (__half*)y;
    P.status = L.d_status;
    P.batch = batch;
    P.n_bt = (batch + TB - 1) / TB;
    const int n_tiles = L.geom.n_rt * P.n_bt;
    static bool attr_done[64] = {false};                                          // function attributes are per device
    const int dev_slot = L.device >= 0 && L.device < 64 ? L.device : 0;
    const size_t smem = sizeof(Smem<TB, KP, DEQ ? 1 : KP>) + 1024;               // slack for the 1024-byte alignment of the stages
    if (!attr_done[dev_slot] || dev_slot != L.device) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemm_tc_kernel<TB, KP, DEQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done[dev_slot] = true;
    }
    const int sms = L.sm_count > 0 ? L.sm_count : 148;
    const bool ring_holds_exchange = sizeof(InStage<TB, KP>) * GemmCfg<TB, KP, DEQ ? 1 : KP>::kStages >= (size_t)kTileM * TB * 4;   // the receive buffer lives in the input ring

    static bool limits_done[64] = {false};
    if (!limits_done[dev_slot]) {                                            // how many clusters of each size fit at once (asked once per kernel)
        for (int lg = 1; lg <= 3; ++lg) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3((unsigned int)((sms / (1 << lg)) * (1 << lg)));
            q.blockDim = dim3(kThreads);
            q.dynamicSmemBytes = smem;
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = 1u << lg;
            qa[0].val.clusterDim.y = 1;
            qa[0].val.clusterDim.z = 1;
            q.attrs = qa;
            q.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, rabit_gemm_tc_kernel<TB, KP, DEQ>, &q) == cudaSuccess && n > 0) g_cluster_limit[lg] = n;
            else cudaGetLastError();
        }
        limits_done[dev_slot] = true;
    }

    // One launch over tiles [lo, hi).  Few tiles: the CTAs of a cluster share each tile's contraction (see choose_split).
    auto launch_range = [&](int lo, int hi) -> cudaError_t {
        GemmParams Q = P;
        Q.tile_lo = lo;
        Q.tile_hi = hi;
        const int count = hi - lo;
        int grid = sms < count ? sms : count;
        int split = ring_holds_exchange ? choose_split(count, L.geom.N, TB, sms) : 1;
        Q.split = split;
        if (split > 1) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned int)(count * split));
            cfg.blockDim = dim3(kThreads);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned int)split;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, rabit_gemm_tc_kernel<TB, KP, DEQ>, Q, map) == cudaSuccess) return cudaSuccess;
            cudaGetLastError();                                    // clusters of this size cannot be placed here: one CTA per tile instead
            Q.split = 1;
        }
        rabit_gemm_tc_kernel<TB, KP, DEQ><<<grid, kThreads, smem, stream>>>(Q, map);
        return cudaGetLastError();
    };
    // A few tiles beyond whole waves would cost a whole wave of their own: they go to a second, split launch.
    const int whole = (n_tiles / sms) * sms, rest = n_tiles - whole;
    if (whole > 0 && rest > 0 && ring_holds_exchange && choose_split(rest, L.geom.N, TB, sms) >= 2) {
        cudaError_t e = launch_range(0, whole);
        if (e != cudaSuccess) return e;
        return launch_range(whole, n_tiles);
    }
    return launch_range(0, n_tiles);
}

cudaError_t rabit_launch_gemm_tc(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream, bool dequantised) {
    if (dequantised)                                                                 // one accumulator: the widest batch tile for every K
        return L.geom.K > 2 ? launch_gemm<256, 3, true>(L, x, y, batch, stream) : launch_gemm<256, 2, true>(L, x, y, batch, stream);
    if (L.geom.K > 2) return launch_gemm<128, 3, false>(L, x, y, batch, stream);   // three accumulators of 128 columns
    // Always the widest batch tile: a tcgen05.mma of M = 128 takes about 128 clocks whatever its N (measured),
    // so narrower tiles would not shorten a step, they would only expand the signs more often.
    return launch_gemm<256, 2, false>(L, x, y, batch, stream);
}
