// Decode GEMV by table look-up (batch 1..2 per launch): the HBM-bound form of the layer
//
//   y[b][i] = sum_k g_k[i] * sum_j B_k[i][j] * t_k[b][j],   t_k[b][j] = h_k[j] * x[b][j]     (Section 4.1, Eq. 2)
//
// At one bit per weight a sign-select add per weight costs more instruction issue slots than HBM
// leaves time for (about 180 weight bits arrive per clock per SM, 128 lane-instructions issue).  The
// signs of eight consecutive input columns of one row are one byte of the packed image (look-up blocks,
// rabit_layout.h), and that byte indexes a 256-entry table of the partial sums  sum_{b<8} (+-) t[8c+b]
// built once per CTA in shared memory: one byte permute (the address), one shared-memory load and one
// fp32 add per EIGHT weights.  The input scale h_k is applied once per table (t = h * x), the signed
// accumulation is the sum of table entries in fp32 registers, and every weight bit is read once.
//
// Work split.  The layer is a grid of blocks (32 rows x 256 columns x K paths, K KB each) stored
// slice-major; CTA c owns a contiguous range of block positions (cut on the host so that all CTAs cost
// the same: so much per block, so much per table), which is one contiguous byte range.  A range that
// crosses into the next 256-column slice rebuilds its table there.
//   * producer warp: one thread streams the range with bulk asynchronous copies (4 blocks per stage,
//     mbarrier transaction counts) into a ring that takes up to the rest of shared memory.  It never
//     waits for the previous kernel in the stream: weights do not depend on it, so they arrive while
//     that kernel finishes and while this one waits for and reads x (programmatic dependent launch).
//   * 16 consumer warps: after the dependency wait they build the table of the slice (lane = byte
//     group, warp = path x upper three index bits; 32 entries each by doubling), then take the blocks
//     round-robin: lane = row.  A lane copies its 16*K weight words to registers (the stage is released
//     at once), walks the 32 byte groups of its row in an order rotated by its lane index (so the 32
//     look-ups of a warp hit 32 banks), and ends with  p = sum_k g_k[row] * s_k.
//   * reduction over the slices of a row, without a second pass, a fence or a wait: p is rounded to a
//     fixed-point grid that the packer sized so that no finite fp16 input can overflow it, and added with
//     ONE 64-bit integer atomic to the row's accumulate word, which also counts arrivals (bits 55..62).
//     The lane whose add returns "all other slices were here" owns the complete sum (old value + its own
//     term): it rounds once to fp16, stores y and puts the word back to zero.  Integer addition commutes,
//     so results do not depend on arrival order; a non-finite partial sum sets bit 63 (NaN output).
// Every wait is bounded; a wait that runs out sets the status word and the kernel drains and returns.
#include <cuda_fp16.h>

#include <algorithm>
#include <vector>

#include "rabit_internal.h"

namespace {

constexpr int kWarps = 16;                               // consumer warps
constexpr int kConsumers = kWarps * 32;
constexpr int kThreads = kConsumers + 32;                // + the producer warp
constexpr int kStageBlocks = 4;
constexpr int kMaxGrid = 160;
constexpr int kMaxGroup = 8;
constexpr int kMaxSlots = 40;
constexpr int kSmemLimit = 232448;                       // 227 KB: the most one CTA may have
constexpr long long kWaitLimitCycles = 1LL << 31;        // about one second
constexpr unsigned long long kSumMask = (1ULL << 55) - 1;

template <int K>
struct Tab {
    static constexpr int kSlotsPerEntry = K <= 2 ? 2 : 4;              // 32-group rows per table entry (one per path)
    static constexpr int kStride = kSlotsPerEntry * 128;               // bytes between entries
    static constexpr int kBytes = 256 * kStride;
    static constexpr int kStageBytes = kStageBlocks * K * RABIT_LUT_PART_BYTES;
};

struct LutLayer {
    const unsigned char* lut;
    const __half* g;
    const __half* h;
    const __half* x;
    __half* y;
    unsigned long long* acc;        // [NB][Mp], all zero between calls
    int M, N, Mp, n_rb, n_cs;
    int fix_bits;
    float inv_unit, unit, limit;    // 2^-unit_exp, 2^unit_exp, 2^fix_bits
};
struct CtaRange {
    int layer, b0, b1;              // block positions [b0, b1) of that layer
};
struct LutParams {
    int n_layers, n_slots;
    unsigned int* status;
    LutLayer layer[kMaxGroup];
    CtaRange range[kMaxGrid];
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
    unsigned int ns = 32;
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return; }
        __nanosleep(ns);
        if (ns < 256) ns *= 2;
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(s));
    return r;
}
template <int OFF>
__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(OFF));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// What a lane still owes for the last block it accumulated: the answer of its atomic add is looked at
// one block later, so that the round trip to L2 overlaps the next block's look-ups.
struct Pending {
    unsigned long long old, add;
    unsigned long long* word;
    __half* yp;                       // nullptr for padded rows
    bool bad, live;
};

template <int NB>
__device__ __forceinline__ void settle(Pending (&pd)[NB], const LutLayer& L) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (!pd[b].live) continue;
        pd[b].live = false;
        if ((int)((pd[b].old >> 55) & 0xFFu) != L.n_cs - 1) continue;          // other slices are still to come
        const unsigned long long sum = (pd[b].old & kSumMask) + (pd[b].add & kSumMask);
        const long long total = (long long)sum - ((long long)L.n_cs << L.fix_bits);
        const bool poisoned = pd[b].bad || (pd[b].old >> 63) != 0;
        const float v = poisoned ? __int_as_float(0x7FC00000) : __ll2float_rn(total) * L.unit;
        if (pd[b].yp) *pd[b].yp = __float2half_rn(v);
        *pd[b].word = 0ULL;                                                     // resting state for the next call
    }
}

template <int K, int NB>
__global__ void __launch_bounds__(kThreads, 1)
rabit_gemv_lut_kernel(const __grid_constant__ LutParams P) {
    using T = Tab<K>;
    extern __shared__ __align__(1024) unsigned char smem[];
    // tables [NB] | ring [n_slots][stage] | full[kMaxSlots] | empty[kMaxSlots] | abort flag
    unsigned char* ring = smem + NB * T::kBytes;
    unsigned long long* full = reinterpret_cast<unsigned long long*>(ring + (size_t)P.n_slots * T::kStageBytes);
    unsigned long long* empty = full + kMaxSlots;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + kMaxSlots);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_slots = P.n_slots;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < n_slots; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), kStageBlocks);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const CtaRange R = P.range[blockIdx.x];
    const LutLayer& L = P.layer[R.layer];
    const int n_blocks = R.b1 - R.b0;
    const int n_stages = (n_blocks + kStageBlocks - 1) / kStageBlocks;

    if (warp == kWarps) {
        // ---- producer: the whole range, as fast as the ring allows; no dependency on the stream's past
        if (lane == 0) {
            const unsigned char* src = L.lut + (size_t)R.b0 * (K * RABIT_LUT_PART_BYTES);
            for (int i = 0; i < n_stages; ++i) {
                const int slot = i % n_slots;
                if (i >= n_slots) {
                    mbar_wait(smem_u32(&empty[slot]), ((i / n_slots) - 1) & 1, abort_flag);
                    if (*abort_flag) break;
                }
                const int blocks = min(kStageBlocks, n_blocks - i * kStageBlocks);
                const uint32_t bytes = blocks * K * RABIT_LUT_PART_BYTES;
                const uint32_t bar = smem_u32(&full[slot]);
                mbar_expect_tx(bar, bytes);
                bulk_g2s(smem_u32(ring + (size_t)slot * T::kStageBytes), src + (size_t)i * T::kStageBytes, bytes, bar);
            }
        }
    } else if (n_blocks > 0) {
        // ---- consumers
        const uint32_t tab0 = smem_u32(smem);
        uint32_t c[8];                                   // byte i of c[j]: bank offset of the group this lane visits in step 4j+i
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t v = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) v |= (uint32_t)((((4 * j + i) + lane) & 31) * (K <= 2 ? 4 : 2)) << (8 * i);
            c[j] = v;
        }
        int cs = R.b0 / L.n_rb;
        int rb = R.b0 - cs * L.n_rb;
        constexpr int kPairs = (8 * K + kWarps - 1) / kWarps;            // (path, upper index bits) pairs a warp builds
        uint4 hq[kPairs];
        auto load_h = [&](int slice) {                                  // static data: may be read before the dependency wait
#pragma unroll
            for (int u = 0; u < kPairs; ++u) {
                const int pi = warp + u * kWarps;
                const int col = slice * RABIT_LUT_COLS + 8 * lane;
                hq[u] = make_uint4(0u, 0u, 0u, 0u);
                if (pi < 8 * K && col < L.N) hq[u] = __ldg(reinterpret_cast<const uint4*>(L.h + (size_t)(pi >> 3) * L.N + col));
            }
        };
        load_h(cs);

        asm volatile("griddepcontrol.wait;" ::: "memory");

        Pending pd[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) pd[b].live = false;
        int b_done = 0;
        while (b_done < n_blocks) {
            const int seg = min(n_blocks - b_done, L.n_rb - rb);
            // ---- table of slice cs:  entry e of (path k, group) = sum_{bit<8} (e has bit ? -t : +t),  t = h * x
            {
                const int col = cs * RABIT_LUT_COLS + 8 * lane;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    uint4 xraw = make_uint4(0u, 0u, 0u, 0u);
                    if (col < L.N) xraw = __ldcg(reinterpret_cast<const uint4*>(L.x + (size_t)b * L.N + col));   // L2: written by the previous kernel
                    const uint32_t xw[4] = {xraw.x, xraw.y, xraw.z, xraw.w};
#pragma unroll
                    for (int u = 0; u < kPairs; ++u) {
                        const int pi = warp + u * kWarps;
                        if (pi >= 8 * K) break;
                        const int k = pi >> 3, ehi = pi & 7;
                        const uint32_t hw[4] = {hq[u].x, hq[u].y, hq[u].z, hq[u].w};
                        float t[8];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float2 hf = __half22float2(*reinterpret_cast<const __half2*>(&hw[q]));
                            const float2 xf = __half22float2(*reinterpret_cast<const __half2*>(&xw[q]));
                            t[2 * q] = hf.x * xf.x;                      // exact: two 11-bit significands
                            t[2 * q + 1] = hf.y * xf.y;
                        }
                        float v[32];
                        v[0] = (ehi & 1 ? -t[5] : t[5]) + (ehi & 2 ? -t[6] : t[6]) + (ehi & 4 ? -t[7] : t[7])
                             + (((t[0] + t[1]) + (t[2] + t[3])) + t[4]);
#pragma unroll
                        for (int bit = 0; bit < 5; ++bit) {
                            const float m2 = -2.f * t[bit];
#pragma unroll
                            for (int e = 0; e < (1 << bit); ++e) v[e | (1 << bit)] = v[e] + m2;
                        }
                        const uint32_t dst = tab0 + b * T::kBytes + (ehi * 32) * T::kStride + k * 128 + lane * 4;
#pragma unroll
                        for (int e = 0; e < 32; ++e) sts_f32(dst + e * T::kStride, v[e]);
                    }
                }
            }
            bar_consumers();

            // ---- blocks b_done .. b_done + seg - 1 of the range, round-robin over the warps
            // (after a wait ran out the warps keep walking the segments, without work, so that all of them
            //  meet at the same barriers)
            int bb = b_done + ((warp - b_done) & (kWarps - 1));
            for (; bb < b_done + seg && !*abort_flag; bb += kWarps) {
                const int row = (rb + (bb - b_done)) * RABIT_LUT_ROWS + lane;
                float gk[K];
#pragma unroll
                for (int k = 0; k < K; ++k) gk[k] = __half2float(__ldg(L.g + (size_t)k * L.Mp + row));
                const int stage = bb / kStageBlocks, slot = stage % n_slots;
                mbar_wait(smem_u32(&full[slot]), (stage / n_slots) & 1, abort_flag);
                if (*abort_flag) break;
                const uint32_t src = smem_u32(ring + (size_t)slot * T::kStageBytes) + (bb % kStageBlocks) * (K * RABIT_LUT_PART_BYTES) + lane * 16;
                uint32_t w[K][8];
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const uint4 lo = lds_v4(src + k * RABIT_LUT_PART_BYTES), hi = lds_v4(src + k * RABIT_LUT_PART_BYTES + 512);
                    w[k][0] = lo.x; w[k][1] = lo.y; w[k][2] = lo.z; w[k][3] = lo.w;
                    w[k][4] = hi.x; w[k][5] = hi.y; w[k][6] = hi.z; w[k][7] = hi.w;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&empty[slot]));      // the weights are in registers: the stage may be refilled

                float acc[NB][K][2];
#pragma unroll
                for (int b = 0; b < NB; ++b)
#pragma unroll
                    for (int k = 0; k < K; ++k) acc[b][k][0] = acc[b][k][1] = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        uint32_t a0 = prmt(w[k][j], c[j], 0xCC04), a1 = prmt(w[k][j], c[j], 0xDD15);
                        uint32_t a2 = prmt(w[k][j], c[j], 0xEE26), a3 = prmt(w[k][j], c[j], 0xFF37);
                        if (K > 2) { a0 <<= 1; a1 <<= 1; a2 <<= 1; a3 <<= 1; }
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            const uint32_t tb = tab0 + b * T::kBytes + k * 128;
                            acc[b][k][0] += lds_f32<0>(tb + a0);
                            acc[b][k][1] += lds_f32<0>(tb + a1);
                            acc[b][k][0] += lds_f32<0>(tb + a2);
                            acc[b][k][1] += lds_f32<0>(tb + a3);
                        }
                    }

                settle<NB>(pd, L);                                       // the previous block's atomics have long returned
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    float p = 0.f;
#pragma unroll
                    for (int k = 0; k < K; ++k) p += gk[k] * (acc[b][k][0] + acc[b][k][1]);
                    const float scaled = p * L.inv_unit;
                    const bool bad = !(fabsf(scaled) < L.limit);          // inf or NaN: finite inputs cannot get here
                    const long long q = bad ? 0LL : __float2ll_rn(scaled);
                    pd[b].add = (unsigned long long)(q + (1LL << L.fix_bits)) + (1ULL << 55);
                    pd[b].word = L.acc + (size_t)b * L.Mp + row;
                    pd[b].yp = row < L.M ? L.y + (size_t)b * L.M + row : nullptr;
                    pd[b].bad = bad;
                    if (bad) atomicOr(pd[b].word, 1ULL << 63);
                    pd[b].old = atomicAdd(pd[b].word, pd[b].add);
                    pd[b].live = true;
                }
            }
            b_done += seg;
            cs += 1;
            rb = 0;
            if (b_done < n_blocks) {
                load_h(cs);
                bar_consumers();                                        // every warp is done with the old table
            }
        }
        settle<NB>(pd, L);
    }

    __syncthreads();                                                    // abort_flag of every warp is final
    if (*abort_flag && tid == kConsumers) {
        // make sure no bulk copy is still in flight towards this CTA's shared memory
        for (int it = max(0, n_stages - n_slots); it < n_stages; ++it) {
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&full[it % n_slots]), (it / n_slots) & 1))
                if (clock64() - t0 > kWaitLimitCycles) break;
        }
        atomicExch(P.status, 1u);
    }
}

// ---- host side: cutting the layers into ranges of equal cost ------------------------------------

struct Cost {
    long long block, table;
};
Cost cost_of(int K, int nb) { return Cost{(long long)nb * (40 * K + 10), (long long)nb * (260 * K) + 200}; }

// CTAs a layer of n_cs x n_rb blocks needs when no CTA may cost more than `limit`; writes the cuts if asked.
int ctas_needed(int n_cs, int n_rb, const Cost& C, long long limit, std::vector<int>* cuts) {
    const long long total = (long long)n_cs * n_rb;
    long long pos = 0;
    int n = 0;
    if (cuts) { cuts->clear(); cuts->push_back(0); }
    while (pos < total) {
        long long budget = limit, taken = 0;
        long long p = pos;
        while (p < total) {
            budget -= C.table;
            const long long can = budget / C.block;
            if (can < 1) break;
            const long long left_in_slice = n_rb - (p % n_rb);
            const long long take = std::min(can, left_in_slice);
            p += take; taken += take; budget -= take * C.block;
            if (take < left_in_slice) break;
        }
        if (taken == 0) return 1 << 30;                                  // the limit does not even pay for one block
        pos = p;
        ++n;
        if (cuts) cuts->push_back((int)pos);
        if (n > (1 << 20)) return 1 << 30;
    }
    return n;
}

// Smallest per-CTA cost with which the layer fits into n_cta CTAs.
long long best_limit(int n_cs, int n_rb, const Cost& C, int n_cta) {
    long long lo = C.table + C.block, hi = (long long)n_cs * (C.table + (long long)n_rb * C.block);
    while (lo < hi) {
        const long long mid = (lo + hi) / 2;
        if (ctas_needed(n_cs, n_rb, C, mid, nullptr) <= n_cta) hi = mid; else lo = mid + 1;
    }
    return lo;
}

template <int K, int NB>
cudaError_t launch_inst(const LutParams& P, int grid, int device, cudaStream_t stream) {
    static bool attr_done[64] = {false};
    const size_t smem = (size_t)NB * Tab<K>::kBytes + (size_t)P.n_slots * Tab<K>::kStageBytes + 2 * kMaxSlots * 8 + 16;
    if (device < 0 || device >= 64 || !attr_done[device]) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemv_lut_kernel<K, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        if (device >= 0 && device < 64) attr_done[device] = true;
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
    return cudaLaunchKernelEx(&cfg, rabit_gemv_lut_kernel<K, NB>, P);
}

int max_slots(int K, int nb) {
    const int table = nb * (K <= 2 ? 65536 : 131072), stage = kStageBlocks * K * RABIT_LUT_PART_BYTES;
    int s = (kSmemLimit - table - 2 * kMaxSlots * 8 - 16) / stage;
    return s > kMaxSlots ? kMaxSlots : s;
}

}  // namespace

int rabit_gemv_lut_max_rows() { return 2; }

bool rabit_gemv_lut_supports(const rabit_layer& L, int batch) {
    if (batch < 1 || batch > 2) return false;
    if (L.geom.K == 3 && batch > 1) return false;                        // two 128 KB tables do not fit
    if (L.geom.n_cs > RABIT_LUT_MAX_SLICES) return false;
    return (long long)L.geom.n_cs * L.geom.n_rb < (1LL << 30) && L.d_lut != nullptr && L.d_acc != nullptr;
}

bool rabit_gemv_lut_group_supports(const rabit_layer* const* layers, int n_layers, int batch) {
    if (n_layers < 1 || n_layers > kMaxGroup) return false;
    for (int l = 0; l < n_layers; ++l) {
        if (!rabit_gemv_lut_supports(*layers[l], batch) || layers[l]->geom.K != layers[0]->geom.K) return false;
        for (int m = 0; m < l; ++m)
            if (layers[m] == layers[l]) return false;                    // one layer twice would share its accumulate words
    }
    return true;
}

// One launch for n_layers independent layers of equal K and 1..2 batch rows (x_l: [batch][N_l], y_l: [batch][M_l]).
cudaError_t rabit_launch_gemv_lut_group(const rabit_layer* const* layers, int n_layers, const void* const* xs, void* const* ys,
                                        int batch, cudaStream_t stream, unsigned long long* const* acc_override, unsigned int* status_override) {
    if (!rabit_gemv_lut_group_supports(layers, n_layers, batch)) return cudaErrorInvalidValue;
    const int K = layers[0]->geom.K;
    LutParams P;
    P.n_layers = n_layers;
    P.status = status_override ? status_override : layers[0]->d_status;
    const Cost C = cost_of(K, batch);
    long long weight[kMaxGroup], total_weight = 0, total_blocks = 0;
    for (int l = 0; l < n_layers; ++l) {
        const rabit_layer& Ly = *layers[l];
        const RabitGeom& G = Ly.geom;
        LutLayer& D = P.layer[l];
        D.lut = Ly.d_lut;
        D.g = (const __half*)Ly.d_g;
        D.h = (const __half*)Ly.d_h;
        D.x = (const __half*)xs[l];
        D.y = (__half*)ys[l];
        D.acc = acc_override ? acc_override[l] : Ly.d_acc;
        D.M = G.M; D.N = G.N; D.Mp = G.Mp; D.n_rb = G.n_rb; D.n_cs = G.n_cs;
        D.fix_bits = G.fix_bits;
        D.unit = ldexpf(1.f, G.unit_exp);
        D.inv_unit = ldexpf(1.f, -G.unit_exp);
        D.limit = ldexpf(1.f, G.fix_bits);
        const long long blocks = (long long)G.n_cs * G.n_rb;
        weight[l] = blocks * C.block + (long long)G.n_cs * C.table;
        total_weight += weight[l];
        total_blocks += blocks;
    }
    for (int l = n_layers; l < kMaxGroup; ++l) P.layer[l] = P.layer[0];
    int sms = layers[0]->sm_count > 0 ? layers[0]->sm_count : 148;
    int grid = sms < kMaxGrid ? sms : kMaxGrid;
    if ((long long)grid > total_blocks) grid = (int)total_blocks;
    if (grid < n_layers) grid = n_layers;                                // (n_layers <= 8 <= any device's SM count)

    // share the CTAs out in proportion to the cost, at least one each, then move single CTAs from the
    // layer that finishes first to the one that finishes last while that lowers the finishing time
    int n_cta[kMaxGroup], given = 0;
    for (int l = 0; l < n_layers; ++l) {
        long long n = (long long)grid * weight[l] / total_weight;
        const long long blocks = (long long)layers[l]->geom.n_cs * layers[l]->geom.n_rb;
        if (n < 1) n = 1;
        if (n > blocks) n = blocks;
        n_cta[l] = (int)n;
        given += n_cta[l];
    }
    auto blocks_of = [&](int l) { return (long long)layers[l]->geom.n_cs * layers[l]->geom.n_rb; };
    while (given > grid) {
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (n_cta[l] > 1 && (best < 0 || weight[l] * n_cta[best] < weight[best] * n_cta[l])) best = l;
        if (best < 0) break;
        n_cta[best] -= 1; given -= 1;
    }
    while (given < grid) {
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (n_cta[l] < blocks_of(l) && (best < 0 || weight[l] * n_cta[best] > weight[best] * n_cta[l])) best = l;
        if (best < 0) break;
        n_cta[best] += 1; given += 1;
    }
    long long limit[kMaxGroup];
    for (int l = 0; l < n_layers; ++l) limit[l] = best_limit(layers[l]->geom.n_cs, layers[l]->geom.n_rb, C, n_cta[l]);
    for (int iter = 0; iter < 8 && n_layers > 1; ++iter) {
        int hi = 0, lo = 0;
        for (int l = 1; l < n_layers; ++l) {
            if (limit[l] > limit[hi]) hi = l;
            if (limit[l] < limit[lo]) lo = l;
        }
        if (hi == lo || n_cta[lo] <= 1 || n_cta[hi] >= blocks_of(hi)) break;
        const long long lo_new = best_limit(layers[lo]->geom.n_cs, layers[lo]->geom.n_rb, C, n_cta[lo] - 1);
        const long long hi_new = best_limit(layers[hi]->geom.n_cs, layers[hi]->geom.n_rb, C, n_cta[hi] + 1);
        if (std::max(lo_new, hi_new) >= limit[hi]) break;
        n_cta[lo] -= 1; n_cta[hi] += 1;
        limit[lo] = lo_new; limit[hi] = hi_new;
    }
    int c0 = 0, max_blocks = 0;
    std::vector<int> cuts;
    for (int l = 0; l < n_layers; ++l) {
        const int used = ctas_needed(layers[l]->geom.n_cs, layers[l]->geom.n_rb, C, limit[l], &cuts);
        if (used > n_cta[l] || c0 + used > kMaxGrid) return cudaErrorInvalidValue;      // cannot happen: limit[l] was found with n_cta[l]
        for (int i = 0; i < used; ++i) {
            P.range[c0 + i] = CtaRange{l, cuts[i], cuts[i + 1]};
            max_blocks = std::max(max_blocks, cuts[i + 1] - cuts[i]);
        }
        c0 += used;
    }
    const int launch_grid = c0;
    for (int i = c0; i < kMaxGrid; ++i) P.range[i] = CtaRange{0, 0, 0};
    const int want = (max_blocks + kStageBlocks - 1) / kStageBlocks;
    P.n_slots = std::max(1, std::min(want, max_slots(K, batch)));
    const int device = layers[0]->device;
    if (K == 1) return batch == 1 ? launch_inst<1, 1>(P, launch_grid, device, stream) : launch_inst<1, 2>(P, launch_grid, device, stream);
    if (K == 2) return batch == 1 ? launch_inst<2, 1>(P, launch_grid, device, stream) : launch_inst<2, 2>(P, launch_grid, device, stream);
    return launch_inst<3, 1>(P, launch_grid, device, stream);
}

cudaError_t rabit_launch_gemv_lut(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    const rabit_layer* one = &L;
    return rabit_launch_gemv_lut_group(&one, 1, &x, &y, batch, stream, nullptr, nullptr);
}
