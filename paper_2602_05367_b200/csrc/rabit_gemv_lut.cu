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
// Measured on B200: the look-ups alone run at 81 clocks per 2 KB block per SM (the shared-memory pipe's
// rate: 64 look-ups + 16 for the weights), 7.3 TB/s over 148 SMs, above what HBM delivers.
//
// Work split.  The layer is a grid of blocks (32 rows x 256 columns x K paths, K KB each) stored
// slice-major; CTA c owns a contiguous range of block positions (cut on the host so that all CTAs cost
// the same: so much per block, so much per table), which is one contiguous byte range.  A range that
// crosses into the next 256-column slice rebuilds its table there.  One CTA per SM, 16 warps:
//   * before the dependency wait (weights do not depend on the previous kernel in the stream, so this
//     overlaps its tail under programmatic dependent launch): every warp loads its first block into
//     registers and the input scales of the first table are read (a bulk L2 prefetch of the CTA's whole
//     range at this point was measured and made the kernel 8-10 % slower: the loads then meet their own
//     prefetch in L2);
//   * after the wait: x of the slice is read, the table is built (lane = byte group, warp = path x upper
//     three index bits; 32 entries each by doubling), and the warps take the blocks round-robin, lane =
//     row.  A lane holds its 16*K weight words in registers (128-bit streaming loads, one block ahead:
//     32 KB in flight per SM; two ahead measured no faster), walks the 32 byte groups of
//     its row in an order rotated by its lane index (so the 32 look-ups of a warp step hit 32 banks), and
//     ends with  p = sum_k g_k[row] * s_k;
//   * reduction over the slices of a row, without a second pass, a fence or a wait: p is rounded to a
//     fixed-point grid that the packer sized so that no finite fp16 input can overflow it, and added with
//     ONE 64-bit integer atomic to the row's accumulate word, which also counts arrivals (bits 55..62).
//     The lane whose add returns "all other slices were here" owns the complete sum (old value + its own
//     term): it rounds once to fp16, stores y and puts the word back to zero.  Integer addition commutes,
//     so results do not depend on arrival order; a non-finite partial sum sets bit 63 (NaN output).
// No thread ever waits for another CTA, and the only waits inside a CTA are barriers of its own warps.
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>
#include <type_traits>
#include <vector>

#include "rabit_internal.h"

namespace {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxGrid = 160;
constexpr int kMaxGroup = 8;
constexpr unsigned long long kSumMask = (1ULL << 55) - 1;

// Tables: one 64 KB table serves two paths, entry e of (path k, byte group) at  e * 256 + (k & 1) * 128 + group * 4
// of table k >> 1.  The tables start on a 64 KB boundary of the CTA's shared-memory window, so that a table address
// is  base | byte << 8 | bank offset  and ONE byte permute builds it whole (no add): see the look-up loop.
template <int K, int NB>
struct Tab {
    static constexpr int kTables = (K + 1) / 2;                       // per batch row
    static constexpr int kBytes = kTables * 65536;                    // per batch row
    static constexpr int kSmem = 65536 + NB * kBytes;                 // alignment slack + tables
    __host__ __device__ static constexpr int offset(int k, int b) { return b * kBytes + (k >> 1) * 65536 + (k & 1) * 128; }
};

template <int I, int N, typename F>
__device__ __forceinline__ void static_for(F&& f) {
    if constexpr (I < N) {
        f(std::integral_constant<int, I>{});
        static_for<I + 1, N>(f);
    }
}

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
    int pad_;                       // (keeps the size a multiple of 8)
};
static_assert(sizeof(LutLayer) % 4 == 0 && sizeof(LutLayer) <= 128, "LutLayer is copied to shared memory by one warp, a word per lane");
struct CtaRange {
    int layer, b0, b1;              // block positions [b0, b1) of that layer
};
struct LutParams {
    int n_layers;
    unsigned int* status;           // RABIT_CHECKED builds: set to 2 when an index check fails (the access is skipped)
    unsigned long long* trace;      // RABIT_TRACE builds: 8 time stamps per CTA of this launch (nullptr: none)
    LutLayer layer[kMaxGroup];
    CtaRange range[kMaxGrid];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_cta() { asm volatile("bar.sync 0;" ::: "memory"); }
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
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// Weights are read exactly once: no L1 allocation, 128-byte L2 sectors.
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// The compiler may move an ordinary use of a loaded value up to the load and stall there; these two keep the load
// early and its first use late (volatile statements keep their order among themselves, and the look-ups are volatile).
__device__ __forceinline__ unsigned short ldg_u16_early(const unsigned short* p) {
    unsigned short v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned short use_here_u16(unsigned short v) {
    unsigned short r;
    asm volatile("mov.b16 %0, %1;" : "=h"(r) : "h"(v));
    return r;
}
__device__ __forceinline__ unsigned long long use_here_u64(unsigned long long v) {
    unsigned long long r;
    asm volatile("mov.b64 %0, %1;" : "=l"(r) : "l"(v));
    return r;
}

// Phase stamps of a CTA (RABIT_TRACE builds only; see rabit_trace_begin in rabit.h): stamp 0 is %globaltimer
// (nanoseconds, coarse) at entry, stamps 1..7 are SM clock cycles since entry, taken by lane 0 of warp 0.
#ifdef RABIT_TRACE
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned long long sm_clock() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t));
    return t;
}
#define RABIT_STAMP0() do { trace_t0 = sm_clock(); if (P.trace && lane == 0 && warp == 0) P.trace[(size_t)blockIdx.x * 64] = global_ns(); } while (0)
#define RABIT_STAMP(i) do { if (P.trace && lane == 0 && warp == 0) P.trace[(size_t)blockIdx.x * 64 + (i)] = sm_clock() - trace_t0; } while (0)
#else
#define RABIT_STAMP0() do { } while (0)
#define RABIT_STAMP(i) do { } while (0)
#endif

// Checked build (-DRABIT_CHECKED, python paper_2602_05367_b200/build.py --checked): every index that addresses global or
// shared memory in this kernel is compared with its range first; a violation sets the status word to 2 and the access
// is skipped (never a trap, never an out-of-range access), so the small-shape suite can run under it in place of a
// memory checker.
#ifdef RABIT_CHECKED
#define RABIT_IN_RANGE(cond) ((cond) ? true : (atomicExch(P.status, 2u), false))
#else
#define RABIT_IN_RANGE(cond) true
#endif

template <int K>
struct Blk {
    uint4 v[2 * K];                  // one lane's 32 bytes per path: (path k, half hf) at v[2k + hf]
};
template <int K>
__device__ __forceinline__ Blk<K> load_blk(const uint4* range_base, int bb, int lane) {
    Blk<K> r;
    const uint4* p = range_base + (size_t)bb * (K * RABIT_LUT_PART_BYTES / 16) + lane;
#pragma unroll
    for (int i = 0; i < 2 * K; ++i) r.v[i] = ldg_stream(p + i * 32);
    return r;
}

// What a lane still owes for the last block it accumulated: the answer of its atomic add is looked at
// one block later, so that the round trip to L2 overlaps the next block's look-ups.
struct Pending {
    unsigned long long old, add;
    unsigned long long* word;
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
        const long long row = (pd[b].word - L.acc) - (long long)b * L.Mp;       // (rare path: the layer's fields come from shared memory)
        if (row >= 0 && row < L.M) L.y[(size_t)b * L.M + row] = __float2half_rn(v);
        *pd[b].word = 0ULL;                                                     // resting state for the next call
    }
}

template <int K, int NB>
__global__ void __launch_bounds__(kThreads, 1)
rabit_gemv_lut_kernel(const __grid_constant__ LutParams P) {
    using T = Tab<K, NB>;
    extern __shared__ __align__(1024) unsigned char smem[];             // slack up to a 64 KB boundary, then the tables
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

#ifdef RABIT_TRACE
    unsigned long long trace_t0;
#endif
    RABIT_STAMP0();                                                     // entry
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // The launch parameters live in constant memory, which is cold in every new launch: a first touch of one of its
    // lines costs a trip to L2.  Everything the CTA needs later is therefore copied to shared memory now, before the
    // dependency wait, so that none of those trips lands between the arrival of x and the end of the kernel.
    __shared__ LutLayer layer_copy;
    __shared__ CtaRange range_copy;
    if (warp == 0) {
        const CtaRange r0 = P.range[blockIdx.x];
        const uint32_t* src = reinterpret_cast<const uint32_t*>(&P.layer[r0.layer]);
        if (lane < (int)(sizeof(LutLayer) / 4)) reinterpret_cast<uint32_t*>(&layer_copy)[lane] = src[lane];
        if (lane == 0) range_copy = r0;
    }
    __syncthreads();
    const CtaRange R = range_copy;
    const LutLayer& L = layer_copy;
    const int n_blocks = R.b1 - R.b0;
    const unsigned char* range_bytes = L.lut + (size_t)R.b0 * (K * RABIT_LUT_PART_BYTES);
    const uint4* range_base = reinterpret_cast<const uint4*>(range_bytes);

    // ---- everything that does not depend on the stream's past
    const int n_mine = warp < n_blocks ? (n_blocks - warp + kWarps - 1) / kWarps : 0;    // blocks warp, warp + 16, ...
    Blk<K> cur;                                          // this warp's current block
#pragma unroll
    for (int i = 0; i < 2 * K; ++i) cur.v[i] = make_uint4(0u, 0u, 0u, 0u);
    if (n_mine > 0) cur = load_blk<K>(range_base, warp, lane);

    const uint32_t tab0 = (smem_u32(smem) + 65535u) & ~65535u;
    // c[j][h]: bytes 0, 1 = bank offsets (4 * group) of the groups this lane visits in steps 4j + 2h and 4j + 2h + 1,
    // bytes 2, 3 = the upper half of the table base.  A permute of (weight word, c) then yields a complete address.
    uint32_t c[8][2];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int h = 0; h < 2; ++h)
            c[j][h] = (uint32_t)((((4 * j + 2 * h) + lane) & 31) * 4) | (uint32_t)((((4 * j + 2 * h + 1) + lane) & 31) * 4) << 8 | (tab0 & 0xFFFF0000u);
    int cs = R.b0 / L.n_rb;
    int seg_rb0 = R.b0 - cs * L.n_rb;                    // row block of the first block of the current segment
    int seg_begin = 0, seg_end = min(n_blocks, L.n_rb - seg_rb0);       // blocks [seg_begin, seg_end) of the range use slice cs
    constexpr int kPairs = (8 * K + kWarps - 1) / kWarps;                // (path, upper index bits) pairs a warp builds
    uint4 hq[kPairs], xq[NB];
    auto load_h = [&](int slice) {                                      // static data: may be read before the dependency wait
#pragma unroll
        for (int u = 0; u < kPairs; ++u) {
            const int pi = warp + u * kWarps;
            const int col = slice * RABIT_LUT_COLS + 8 * lane;
            hq[u] = make_uint4(0u, 0u, 0u, 0u);
            if (pi < 8 * K && col < L.N) hq[u] = __ldg(reinterpret_cast<const uint4*>(L.h + (size_t)(pi >> 3) * L.N + col));
        }
    };
    auto load_x = [&](int slice) {                                      // L2 (not L1): written by the previous kernel in the stream
        const int col = slice * RABIT_LUT_COLS + 8 * lane;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            xq[b] = make_uint4(0u, 0u, 0u, 0u);
            if (col < L.N) xq[b] = __ldcg(reinterpret_cast<const uint4*>(L.x + (size_t)b * L.N + col));
        }
    };
    // table of the slice whose h and x sit in hq / xq:  entry e of (path k, group) = sum_{bit<8} (e has bit ? -t : +t),  t = h * x
    auto build_table = [&]() {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const uint32_t xw[4] = {xq[b].x, xq[b].y, xq[b].z, xq[b].w};
#pragma unroll
            for (int u = 0; u < kPairs; ++u) {
                const int pi = warp + u * kWarps;
                if (pi >= 8 * K) break;
                const int k = pi >> 3, ehi = pi & 7;
                const uint32_t hw[4] = {hq[u].x, hq[u].y, hq[u].z, hq[u].w};
                float t[8];
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float2 hf = __half22float2(*reinterpret_cast<const __half2*>(&hw[w]));
                    const float2 xf = __half22float2(*reinterpret_cast<const __half2*>(&xw[w]));
                    t[2 * w] = hf.x * xf.x;                              // exact: two 11-bit significands
                    t[2 * w + 1] = hf.y * xf.y;
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
                const uint32_t dst = tab0 + b * T::kBytes + (k >> 1) * 65536 + (ehi * 32) * 256 + (k & 1) * 128 + lane * 4;
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (RABIT_IN_RANGE(dst + e * 256 >= tab0 && dst + e * 256 + 4 <= tab0 + (uint32_t)(NB * T::kBytes) && dst + e * 256 + 4 <= smem_u32(smem) + (uint32_t)T::kSmem))
                        sts_f32(dst + e * 256, v[e]);
            }
        }
    };
    // makes the table of block bb's slice the current one; every warp crosses every slice border of the range here
    auto advance_to = [&](int bb) {
        while (bb >= seg_end) {
            bar_cta();                                                  // every warp is done with the old table
            build_table();
            cs += 1;
            seg_begin = seg_end;
            seg_rb0 = 0;
            seg_end = min(n_blocks, seg_end + L.n_rb);
            if (seg_end < n_blocks) { load_h(cs + 1); load_x(cs + 1); } // the table after this one
            bar_cta();
        }
    };
    load_h(cs);

    asm volatile("griddepcontrol.wait;" ::: "memory");
    RABIT_STAMP(1);                                                     // the previous kernel's results are visible
    if (n_blocks <= 0) return;
    load_x(cs);
#ifdef RABIT_TRACE
    if (xq[0].x == 0x12345678u && xq[0].y == 0x9ABCDEF0u && hq[0].x == 0x12345678u) RABIT_STAMP(7);   // (a use of x and h, so that the next stamp follows their arrival)
#endif
    RABIT_STAMP(2);                                                     // x and h of the first table have arrived
    build_table();
    if (seg_end < n_blocks) { load_h(cs + 1); load_x(cs + 1); }
    bar_cta();
    RABIT_STAMP(3);                                                     // first table built

    // One iteration per block of this warp.  Everything with a long latency is ISSUED at the top of an iteration
    // (the next block's weights, this block's output scales, the atomic adds of the previous block) and its result is
    // first touched below the look-ups of the same iteration, some 1300 cycles later: no request is in flight across the
    // loop's back edge, where the compiler would otherwise have the warp wait for it (a warp has six scoreboards).
    // what every iteration needs of the layer, in registers (the shared-memory pipe is the one this loop saturates)
    const unsigned short* const g_base = reinterpret_cast<const unsigned short*>(L.g);
    unsigned long long* const acc_base = L.acc;
    const int Mp = L.Mp;
    const float inv_unit = L.inv_unit, limit = L.limit;
    const long long bias = (1LL << L.fix_bits) + (1LL << 55);            // shift to non-negative + one arrival
    Pending pd[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) { pd[b].live = false; pd[b].old = 0ULL; pd[b].add = 0ULL; pd[b].word = nullptr; pd[b].bad = false; }
    bool owe = false;                                                   // pd holds a finished block whose atomics are still to be issued
    for (int i = 0; i < n_mine; ++i) {
        const int bb = warp + i * kWarps;
#ifdef RABIT_TRACE
        if (i < 11) RABIT_STAMP(8 + 5 * i);                             // iteration i: top
#endif
        advance_to(bb);
        const int row = (seg_rb0 + (bb - seg_begin)) * RABIT_LUT_ROWS + lane;
        unsigned short graw[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            graw[k] = 0;
            if (RABIT_IN_RANGE(row >= 0 && row < Mp)) graw[k] = ldg_u16_early(g_base + (size_t)k * Mp + row);
        }
        const int bb_next = i + 1 < n_mine ? bb + kWarps : bb;
        Blk<K> nxt = cur;
        if (RABIT_IN_RANGE(bb_next >= 0 && bb_next < n_blocks && (long long)R.b0 + bb_next < (long long)L.n_cs * L.n_rb))
            nxt = load_blk<K>(range_base, bb_next, lane);   // (the last iteration re-reads its own block: in bounds, unused)
        if (owe) {
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (!RABIT_IN_RANGE(pd[b].word >= acc_base && pd[b].word < acc_base + (size_t)NB * Mp)) continue;
                if (pd[b].bad) atomicOr(pd[b].word, 1ULL << 63);
                pd[b].old = atomicAdd(pd[b].word, pd[b].add);
                pd[b].live = true;
            }
        }
        if (i == 0) RABIT_STAMP(4);                                     // first weights in registers
#ifdef RABIT_TRACE
        {
            unsigned int u = cur.v[0].x;
#pragma unroll
            for (int t = 0; t < 2 * K; ++t) u |= cur.v[t].w;
            u = (unsigned int)use_here_u64(u);                           // the block's weights have arrived
            if (i < 11 && u != 0x13572468u) RABIT_STAMP(9 + 5 * i);
        }
#endif

        float acc[NB][K][2];
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int k = 0; k < K; ++k) acc[b][k][0] = acc[b][k][1] = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            static_for<0, K>([&](auto kc) {
                constexpr int k = decltype(kc)::value;
                const uint4 part = cur.v[2 * k + (j >> 2)];
                const uint32_t w = (j & 3) == 0 ? part.x : (j & 3) == 1 ? part.y : (j & 3) == 2 ? part.z : part.w;
                // address = table base | sign byte << 8 | bank offset, all from one permute
                const uint32_t a0 = prmt(w, c[j][0], 0x7604), a1 = prmt(w, c[j][0], 0x7615);
                const uint32_t a2 = prmt(w, c[j][1], 0x7624), a3 = prmt(w, c[j][1], 0x7635);
#ifdef RABIT_CHECKED
                {
                    const uint32_t lo = tab0, hi = tab0 + 65536u - 128u;     // with the path offset added: inside table k >> 1
                    if (!RABIT_IN_RANGE(a0 >= lo && a0 < hi && a1 >= lo && a1 < hi && a2 >= lo && a2 < hi && a3 >= lo && a3 < hi)) return;
                }
#endif
                static_for<0, NB>([&](auto bc) {
                    constexpr int b = decltype(bc)::value;
                    acc[b][k][0] += lds_f32<T::offset(k, b)>(a0);
                    acc[b][k][1] += lds_f32<T::offset(k, b)>(a1);
                    acc[b][k][0] += lds_f32<T::offset(k, b)>(a2);
                    acc[b][k][1] += lds_f32<T::offset(k, b)>(a3);
                });
            });
#ifdef RABIT_TRACE
        if (i == 0) RABIT_STAMP(7);                                     // first block's look-ups issued
        if (i < 11 && use_here_u64(__float_as_uint(acc[0][0][0] + acc[0][0][1] + acc[0][K - 1][0] + acc[0][K - 1][1])) != 0x13572468u) RABIT_STAMP(10 + 5 * i);   // look-ups answered
#endif
#pragma unroll
        for (int b = 0; b < NB; ++b) pd[b].old = use_here_u64(pd[b].old);
        settle<NB>(pd, L);                                               // the previous block's atomics, issued above the look-ups
#ifdef RABIT_TRACE
        if (i < 11) RABIT_STAMP(11 + 5 * i);                            // previous atomic answered and settled
#endif
#pragma unroll
        for (int k = 0; k < K; ++k) graw[k] = use_here_u16(graw[k]);
#ifdef RABIT_TRACE
        if (i < 11) RABIT_STAMP(12 + 5 * i);                            // output scales have arrived
#endif
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            float p = 0.f;
#pragma unroll
            for (int k = 0; k < K; ++k) p += __half2float(__ushort_as_half(graw[k])) * (acc[b][k][0] + acc[b][k][1]);
            const float scaled = p * inv_unit;
            const bool bad = !(fabsf(scaled) < limit);                    // inf or NaN: finite inputs cannot get here
            const long long qv = bad ? 0LL : __float2ll_rn(scaled);
            pd[b].add = (unsigned long long)(qv + bias);
            pd[b].word = acc_base + (size_t)b * Mp + row;
            pd[b].bad = bad;
        }
        owe = true;
#pragma unroll
        for (int t = 0; t < 2 * K; ++t) cur.v[t] = nxt.v[t];             // the next block's weights have arrived by now
        cur.v[0].x = (unsigned int)use_here_u64(cur.v[0].x);
    }
    if (owe) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            if (!RABIT_IN_RANGE(pd[b].word >= acc_base && pd[b].word < acc_base + (size_t)NB * Mp)) continue;
            if (pd[b].bad) atomicOr(pd[b].word, 1ULL << 63);
            pd[b].old = atomicAdd(pd[b].word, pd[b].add);
            pd[b].live = true;
        }
    }
    RABIT_STAMP(5);                                                     // last look-up done, last atomic issued
    advance_to(n_blocks - 1);                                           // warps that ran out of blocks early still take part in the rebuilds
    settle<NB>(pd, L);
    RABIT_STAMP(6);                                                     // last atomic answered, y stored
}

// ---- host side: cutting the layers into ranges of equal cost ------------------------------------

struct Cost {
    long long block, table;
};
// SM clock cycles, from the phase stamps of the kernel on B200: a block of K paths (look-ups, loads, its atomic) and a
// table (build plus the two barriers around it).
// (the table figure is a fit: the split that minimises the measured step time charges a table about 26 blocks, far
// more than its 430 cycles of stores, because a rebuild in mid-range also stops every warp at two barriers)
Cost cost_of(int K, int nb) { return Cost{(long long)nb * (70 * K + 30), (long long)nb * (2200 * K) + 100}; }

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
    const size_t smem = (size_t)Tab<K, NB>::kSmem;
    if (device < 0 || device >= 64 || !attr_done[device]) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemv_lut_kernel<K, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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

cudaError_t launch_k(int K, int batch, const LutParams& P, int grid, int device, cudaStream_t stream) {
    if (K == 1) return batch == 1 ? launch_inst<1, 1>(P, grid, device, stream) : launch_inst<1, 2>(P, grid, device, stream);
    if (K == 2) return batch == 1 ? launch_inst<2, 1>(P, grid, device, stream) : launch_inst<2, 2>(P, grid, device, stream);
    return launch_inst<3, 1>(P, grid, device, stream);
}

}  // namespace

int rabit_gemv_lut_max_rows() { return 2; }

bool rabit_gemv_lut_supports(const rabit_layer& L, int batch) {
    if (batch < 1 || batch > 2) return false;
    if (L.geom.K == 3 && batch > 1) return false;                        // four 64 KB tables do not fit into shared memory
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
    P.status = status_override ? status_override : layers[0]->d_status;  // (only a checked build writes it: this kernel has no wait that could run out)
    P.trace = nullptr;
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
    // The cut of the layers into ranges depends only on the shapes, the batch and the device: remembered per thread
    // (a decoder calls the same few groups over and over; the search costs a few microseconds of host time).
    struct PlanKey { int n, batch, sms, shape[kMaxGroup][3]; };
    struct Plan { PlanKey key; int grid; CtaRange range[kMaxGrid]; };
    static thread_local std::vector<Plan> plans;
    PlanKey key;
    std::memset(&key, 0, sizeof(key));
    key.n = n_layers; key.batch = batch; key.sms = layers[0]->sm_count;
    for (int l = 0; l < n_layers; ++l) { key.shape[l][0] = K; key.shape[l][1] = layers[l]->geom.n_rb; key.shape[l][2] = layers[l]->geom.n_cs; }
    for (const Plan& pl : plans)
        if (std::memcmp(&pl.key, &key, sizeof(key)) == 0) {
            std::memcpy(P.range, pl.range, sizeof(P.range));
            P.trace = rabit_trace_slot(pl.grid);
            return launch_k(K, batch, P, pl.grid, layers[0]->device, stream);
        }
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
    int c0 = 0;
    std::vector<int> cuts;
    for (int l = 0; l < n_layers; ++l) {
        const int used = ctas_needed(layers[l]->geom.n_cs, layers[l]->geom.n_rb, C, limit[l], &cuts);
        if (used > n_cta[l] || c0 + used > kMaxGrid) return cudaErrorInvalidValue;      // cannot happen: limit[l] was found with n_cta[l]
        for (int i = 0; i < used; ++i) {
            P.range[c0 + i] = CtaRange{l, cuts[i], cuts[i + 1]};
        }
        c0 += used;
    }
    const int launch_grid = c0;
    for (int i = c0; i < kMaxGrid; ++i) P.range[i] = CtaRange{0, 0, 0};
    if (plans.size() >= 256) plans.clear();
    plans.emplace_back();
    plans.back().key = key;
    plans.back().grid = launch_grid;
    std::memcpy(plans.back().range, P.range, sizeof(P.range));
    P.trace = rabit_trace_slot(launch_grid);
    return launch_k(K, batch, P, launch_grid, layers[0]->device, stream);
}

cudaError_t rabit_launch_gemv_lut(const rabit_layer& L, const void* x, void* y, int batch, cudaStream_t stream) {
    const rabit_layer* one = &L;
    return rabit_launch_gemv_lut_group(&one, 1, &x, &y, batch, stream, nullptr, nullptr);
}
