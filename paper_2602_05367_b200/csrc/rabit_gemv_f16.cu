// Decode GEMV for 3..16 batch rows: the batch sits in the N dimension of an f16 tensor-core MMA.
//
//   y[b][i] = sum_k g_k[i] * sum_j (B_k[i][j] h_k[j]) * x[b][j]                              (Section 4.1, Eq. 2)
//
// The table-driven kernel (rabit_gemv_lut.cu) pays per batch row; the integer tensor-core GEMV spends four of an MMA's
// eight columns per batch row and needs a pass over x first.  Here the A operand of mma.sync.m16n8k16 is +-h_k expanded in
// registers from the sign tiles (the weight bit flips the sign bit of the fp16 input scale: exact), B is x as it is, the
// accumulators are fp32: products are exact, 8 batch rows per MMA and 16 with a second MMA on the same A, no digits, no
// scale search.  The cost is that of the expansion and does not depend on the batch.
//
// Expansion.  Shifts, byte permutes and logic instructions all issue on the half-rate integer pipe of an SM sub-partition
// (16 lanes per clock), and that pipe, not the tensor pipe, bounds this kernel.  So an A register (two fp16 values) costs
// ONE logic instruction there, (v & 0x80008000) ^ h, and the shift that brings the two weight bits to bits 15 and 31 is a
// multiplication by a power of two on the multiply-add pipe: v = w * 2^s, where the factor comes from a kernel parameter
// so that the compiler keeps it a multiplication.  The two bits must be 16 apart in the word, i.e. two columns apart:
//
// Operand mapping.  A sign tile (rabit_layout.h) gives lane (gq, tq) four words w[a]; byte c of word a has in bit p the
// sign of row 16p + gq + 8(a & 1), column 16(a >> 1) + 4tq + c of the tile.  For the k-step kh = a >> 1 (16 columns) and
// the row block p, the MMA's k slots (2tq, 2tq+1, 2tq+8, 2tq+9) of lane (gq, tq) are taken to be the tile columns
// 16kh + 4tq + (0, 2, 1, 3): any fixed assignment of slots to columns is valid as long as A and B use the same one.  Then
//     a0 = +-h(cols 0,2) for row gq      from bits p, 16+p of w[2kh] * 2^(15-p)      a1 = the same, row gq + 8, from w[2kh+1]
//     a2 = +-h(cols 1,3) for row gq      from bits 8+p, 24+p of w[2kh] * 2^(7-p)     a3 = row gq + 8, from w[2kh+1]
//     b0 = x[n = gq][cols 0,2]           b1 = x[n = gq][cols 1,3]         (one 8-byte load per lane and k-step, two permutes)
// and the accumulator lane holds rows gq, gq + 8 of the block and batch rows 2tq, 2tq + 1.
//
// Work split.  The layer is n_rt row tiles x n_cs slices of 256 columns; in that order the (row tile, slice) pairs are cut
// into one contiguous range per SM and every SM's range into two parts, by a cost model on the host (plan_ranges).  One
// CTA of 16 warps per SM; its two groups of 8 warps each take one part and share nothing but the SM (own barrier, own
// shared memory): while one group adds up a segment and waits for its atomics, the other computes.  The part of a range
// inside one row tile is a segment.  Warp w of a group works on path w % K and shares the column tiles of the segment
// with the other warps of that path.  A warp streams its tiles through a ring of its own in shared memory with
// asynchronous 16-byte copies (one per lane and tile, each lane reads back only what it copied itself, so no barrier is
// involved), kRing - 1 tiles ahead: with 16 warps per SM that keeps about 56 KB per SM in flight, which is what the HBM
// latency needs (with the tiles prefetched into registers, two to four per warp, the kernel ran at the speed of its
// memory latency, 1.1 to 1.7 TB/s).  At the end of a segment every warp writes its accumulators to its own slot of shared
// memory, the group adds the slots path by path in a fixed order (deterministic) and applies g_k to each path's sum, and
// every output of the segment goes, as in the table-driven kernel, into the row's 64-bit accumulate word with one
// integer atomic (fixed-point grid of the packer, arrival count in bits 55..62, bit 63 = non-finite); the thread whose
// add completes a row (the count reaches the number of segments of that row tile) rounds it to fp16, stores y and clears
// the word.  A contribution that covers s slices is shifted by s * 2^fix_bits, so the total shift is the same
// n_cs * 2^fix_bits for every split.  Nothing waits for another CTA or for the other group.
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>
#include <vector>

#include "rabit_internal.h"

namespace {

constexpr int kWarps = 8;                              // warps of a group
constexpr int kGroupThreads = kWarps * 32;
constexpr int kGroups = 2;                             // independent groups of a CTA (one CTA per SM)
constexpr int kThreads = kGroups * kGroupThreads;
constexpr int kRing = 8;                               // sign tiles a warp keeps in flight or in use (a power of two)
constexpr long long kMaxPairs = 1LL << 30;
constexpr int kMaxRanges = kGroups * 160;              // one range per group, up to 160 SMs
constexpr int kSlotStride = 128 + 4;                  // floats per batch row of a slot: the pad spreads a warp's store over all banks
constexpr unsigned long long kSumMask = (1ULL << 55) - 1;

struct F16Params {
    const uint4* tiles;
    const __half* g;
    const __half* h;
    const __half* x;
    __half* y;
    unsigned long long* acc;        // [16][Mp], all zero between calls
    unsigned int* status;           // RABIT_CHECKED builds: set to 2 when an index check fails (the access is skipped)
    int K, M, N, Mp, n_rt, n_ct, n_cs;
    int batch;
    int n_pairs;                    // n_rt * n_cs (row tile, slice) pairs; group q of CTA c owns pairs [bound[2c + q], bound[2c + q + 1])
    int fix_bits;
    float inv_unit, unit, limit;
    uint32_t two, two_pow_8;        // 2 and 256: multipliers the compiler cannot fold into shifts
    int bound[kMaxRanges + 1];      // ascending; bound[2 * grid] = n_pairs
};

// Checked build (-DRABIT_CHECKED, python paper_2602_05367_b200/build.py --checked): every index that addresses global or
// shared memory is compared with its range first; a violation is recorded in the layer's status word and the access is
// skipped (nothing traps).  In the ordinary build the checks compile to nothing.
#ifdef RABIT_CHECKED
#define RABIT_IN_RANGE(cond) ((cond) ? true : (atomicExch(P.status, 2u), false))
#else
#define RABIT_IN_RANGE(cond) true
#endif

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(s));
    return r;
}
// (a & 0x80008000) ^ c: the sign bits of two fp16 values, applied to a pair of input scales
__device__ __forceinline__ uint32_t flip(uint32_t a, uint32_t c) {
    uint32_t r;
    asm volatile("lop3.b32 %0, %1, 0x80008000, %2, 0x6A;" : "=r"(r) : "r"(a), "r"(c));
    return r;
}
// a * m on the multiply-add pipe (m is a power of two the compiler does not know)
__device__ __forceinline__ uint32_t mul_lo(uint32_t a, uint32_t m) {
    uint32_t r;
    asm volatile("mul.lo.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(m));
    return r;
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// 16 bytes global -> shared, asynchronous, not through L1; one group per call so that groups and tiles count alike
__device__ __forceinline__ void copy_async_16(uint32_t dst_smem, const void* src, bool valid) {
    if (valid) asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void copy_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// barrier of one group (ids 1 and 2; 0 is left to __syncthreads)
__device__ __forceinline__ void group_sync(int group) {
    asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "n"(kGroupThreads) : "memory");
}
__device__ __forceinline__ uint4 lds_128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// One output of a segment from the warps' slots: warp w holds path w % KK; the paths' sums are formed warp by warp in the
// order of the warps and scaled by the path's output scale.
template <int KK, int NH>
__device__ __forceinline__ float path_sums(const float* col, const __half (&g)[RABIT_MAX_K]) {
    float sk[KK];
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) sk[kk] = 0.f;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) sk[wv % KK] += col[(size_t)wv * (NH * 8 * kSlotStride)];
    float v = 0.f;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) v = fmaf(__half2float(g[kk]), sk[kk], v);
    return v;
}

// The range that holds pair u: the last r with bound[r] <= u (empty ranges have bound[r] == bound[r + 1] and lose to
// the non-empty one that follows them).
__device__ __forceinline__ int owner_of(const F16Params& P, int u, int n_ranges) {
    int lo = 0, hi = n_ranges - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (P.bound[mid] <= u) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// NH = halves of the batch (8 rows each) a pass carries.
template <int NH>
__global__ void __launch_bounds__(kThreads, 1)
rabit_gemv_f16_kernel(const __grid_constant__ F16Params P) {
    extern __shared__ __align__(16) float smem_f[];                      // per group: [kWarps][NH * 8][kSlotStride] partial outputs, then the warps' rings
    constexpr int kGroupFloats = kWarps * NH * 8 * kSlotStride + kWarps * kRing * 128;
    const int group = threadIdx.x / kGroupThreads;                       // the two groups share nothing but the SM
    const int tid = threadIdx.x % kGroupThreads, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tq = lane & 3;
    float* slots = smem_f + (size_t)group * kGroupFloats;
    // the lane's 16 bytes of ring slot 0 of its warp; slot r is r * 512 bytes further
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(slots) + (uint32_t)(kWarps * NH * 8 * kSlotStride * sizeof(float)) +
                          (uint32_t)((warp * kRing * 32 + lane) * 16);

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited = false;

    // every warp works on ONE path: path k = warp % K, and the column tiles of a segment are dealt out among the group's
    // warps of that path (K = 3: three, three and two warps)
    const int k = warp % P.K;
    const int n_same = (kWarps - k + P.K - 1) / P.K, j0 = warp / P.K;
    const int hk = k * P.N + 4 * tq;                                      // element offsets (K * N and 16 * N fit 31 bits: N <= 65280)
    int xb[NH];
#pragma unroll
    for (int hf = 0; hf < NH; ++hf)                                      // lanes beyond the batch read its last row; their columns are never stored
        xb[hf] = min(8 * hf + gq, P.batch - 1) * P.N + 4 * tq;

    // A segment: row tile rt, column tiles [ct0, c1) of which this warp takes every n_same-th, starting at ct0.
    struct Segment {
        int rt, n_slices, c1, ct0, n_my;
        const uint4* wsrc;                                               // the warp's first tile (this lane's 16 bytes)
    };
    const int n_ranges = kGroups * gridDim.x;
    int u = P.bound[kGroups * blockIdx.x + group];
    const int u_end = P.bound[kGroups * blockIdx.x + group + 1];
    auto next_segment = [&]() {                                          // the segment that starts at pair u; advances u
        Segment sg;
        sg.rt = u / P.n_cs;
        const int s0 = u - sg.rt * P.n_cs;
        const int s1 = min(P.n_cs, s0 + (u_end - u));
        u += s1 - s0;
        sg.n_slices = s1 - s0;
        sg.c1 = min(P.n_ct, s1 * 8);                                     // a slice is eight column tiles
        sg.ct0 = s0 * 8 + j0;
        sg.n_my = sg.ct0 < sg.c1 ? (sg.c1 - sg.ct0 + n_same - 1) / n_same : 0;
        sg.wsrc = P.tiles + (size_t)(sg.rt * P.K + k) * P.n_ct * 32 + sg.ct0 * 32 + lane;
        return sg;
    };
    auto prefill = [&](const Segment& sg) {                              // the first kRing - 1 tiles of the warp; weights never depend on the stream's past
#pragma unroll
        for (int i = 0; i < kRing - 1; ++i)
            copy_async_16(ring + i * 512, sg.wsrc + (size_t)i * n_same * 32,
                          i < sg.n_my && RABIT_IN_RANGE(sg.wsrc + (size_t)i * n_same * 32 >= P.tiles &&
                                                        sg.wsrc + (size_t)i * n_same * 32 < P.tiles + (size_t)P.n_rt * P.K * P.n_ct * 32));
    };
    bool more = u < u_end;
    Segment sg;
    if (more) {
        sg = next_segment();
        prefill(sg);
    }
    while (more) {
        const int rt = sg.rt, ct0 = sg.ct0, n_my = sg.n_my;
        const uint4* wsrc = sg.wsrc;
        float acc[8][NH][4];
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int hf = 0; hf < NH; ++hf)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[p][hf][e] = 0.f;

        // input scales and activations of the lane's four columns of k-step kh of column tile ct, as loaded (columns 0,1 | 2,3)
        auto fetch_hx = [&](int ct, int kh, uint2& fh, uint2 (&fx)[NH]) {
            const int off = ct * 32 + 16 * kh;
            if (!RABIT_IN_RANGE(off >= 0 && hk + off + 4 <= P.K * P.N)) return;
            fh = __ldg(reinterpret_cast<const uint2*>(P.h + hk + off));
#pragma unroll
            for (int hf = 0; hf < NH; ++hf)
                if (RABIT_IN_RANGE(xb[hf] + off + 4 <= P.batch * P.N)) fx[hf] = __ldcg(reinterpret_cast<const uint2*>(P.x + xb[hf] + off));
        };

        // weights kRing - 1 tiles ahead (HBM latency), scales and activations one tile ahead, k-step by k-step in place
        if (!waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");            // x, y and the accumulate words only after this
            waited = true;
        }
        uint2 fh[2], fx[2][NH];
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) fetch_hx(min(ct0, P.n_ct - 1), kh, fh[kh], fx[kh]);
        for (int i = 0; i < n_my; ++i) {
            {
                const int ct = ct0 + i * n_same;
                const int ia = i + kRing - 1;                            // the tile that takes the slot freed in the last round
                copy_async_16(ring + (ia & (kRing - 1)) * 512, wsrc + (size_t)ia * n_same * 32,
                              ia < n_my && RABIT_IN_RANGE(wsrc + (size_t)ia * n_same * 32 >= P.tiles &&
                                                          wsrc + (size_t)ia * n_same * 32 < P.tiles + (size_t)P.n_rt * P.K * P.n_ct * 32));
                copy_async_wait<kRing - 1>();                            // tile i has landed (one group per tile, also for the tiles that do not exist)
                const uint4 wv = lds_128(ring + (i & (kRing - 1)) * 512);
                const int ct_next = min(ct + n_same, P.n_ct - 1);        // beyond the segment: a valid address, never used
                const uint32_t w[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {
                    const uint32_t h02 = prmt(fh[kh].x, fh[kh].y, 0x5410), h13 = prmt(fh[kh].x, fh[kh].y, 0x7632);
                    uint32_t b0[NH], b1[NH];
#pragma unroll
                    for (int hf = 0; hf < NH; ++hf) {
                        b0[hf] = prmt(fx[kh][hf].x, fx[kh][hf].y, 0x5410);
                        b1[hf] = prmt(fx[kh][hf].x, fx[kh][hf].y, 0x7632);
                    }
                    fetch_hx(ct_next, kh, fh[kh], fx[kh]);                // the same k-step of the warp's next tile, in place
                    // u = w * 2^(7-p): bit p of bytes 1 and 3 -> bits 15 and 31;  v = u * 2^8: the same for bytes 0 and 2
                    uint32_t ul = w[2 * kh], uh = w[2 * kh + 1];
                    uint32_t vl = mul_lo(ul, P.two_pow_8), vh = mul_lo(uh, P.two_pow_8);
#pragma unroll
                    for (int p = 7; p >= 0; --p) {
                        const uint32_t a0 = flip(vl, h02), a1 = flip(vh, h02), a2 = flip(ul, h13), a3 = flip(uh, h13);
#pragma unroll
                        for (int hf = 0; hf < NH; ++hf) mma_f16(acc[p][hf], a0, a1, a2, a3, b0[hf], b1[hf]);
                        if (p > 0) {
                            ul = mul_lo(ul, P.two); uh = mul_lo(uh, P.two);
                            vl = mul_lo(vl, P.two); vh = mul_lo(vh, P.two);
                        }
                    }
                }
            }
        }
        copy_async_wait<0>();
        // the next segment's first tiles set off now: they cross HBM while this segment is added up
        const int n_slices = sg.n_slices;
        more = u < u_end;
        if (more) {
            sg = next_segment();
            prefill(sg);
        }
        constexpr int kPer = NH * 8 * 128 / kGroupThreads;                    // outputs per thread (4 or 8)
        __half gk[RABIT_MAX_K];                                           // output scales of the thread's row (the same row for all its outputs), loaded early
#pragma unroll
        for (int kk = 0; kk < RABIT_MAX_K; ++kk)
            gk[kk] = kk < P.K ? P.g[(size_t)kk * P.Mp + rt * RABIT_TILE_ROWS + (tid & 127)] : __half();
        // ---- the warp's partial outputs -> its slot; slot layout [batch row][row of the tile]
        float* mine = slots + (size_t)warp * (NH * 8 * kSlotStride);
        const bool slot_ok = RABIT_IN_RANGE(mine + (NH * 8 - 1) * kSlotStride + 127 < smem_f + kGroups * kGroupFloats);
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int hf = 0; hf < NH; ++hf) {
                if (!slot_ok) break;
                const int b = 8 * hf + 2 * tq, row = 16 * p + gq;
                mine[(b) * kSlotStride + row] = acc[p][hf][0];
                mine[(b + 1) * kSlotStride + row] = acc[p][hf][1];
                mine[(b) * kSlotStride + row + 8] = acc[p][hf][2];
                mine[(b + 1) * kSlotStride + row + 8] = acc[p][hf][3];
            }
        group_sync(group);
        // ---- fixed-order sum over the warps, then one atomic per output of the segment
        int arrivals = 0;                                                // segments of this row tile: the non-empty ranges that touch it
        for (int r = owner_of(P, rt * P.n_cs, n_ranges), r1 = owner_of(P, (rt + 1) * P.n_cs - 1, n_ranges); r <= r1; ++r)
            arrivals += P.bound[r] < P.bound[r + 1] ? 1 : 0;
        // (thread t owns row t & 127 of the tile and the batch rows (t >> 7) + 2 i; rows beyond the batch are computed from
        // whatever their MMA columns held and dropped)
        unsigned long long old[kPer], add[kPer];
        bool bad[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int o = tid + i * kGroupThreads, b = o >> 7, rl = o & 127;
            // sum_k g_k * (sum over the warps of path k), in a fixed order
            const float* col = slots + b * kSlotStride + rl;
            const float v = P.K == 2 ? path_sums<2, NH>(col, gk) : P.K == 3 ? path_sums<3, NH>(col, gk) : path_sums<1, NH>(col, gk);
            const float scaled = v * P.inv_unit;
            bad[i] = !(fabsf(scaled) < P.limit * (float)n_slices);       // inf or NaN: finite inputs cannot get here
            const long long q = bad[i] ? 0LL : __float2ll_rn(scaled);
            add[i] = (unsigned long long)(q + ((long long)n_slices << P.fix_bits)) + (1ULL << 55);
        }
        // all atomics of the thread back to back: nothing between them that could wait for an answer
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int o = tid + i * kGroupThreads, b = o >> 7, rl = o & 127;
            old[i] = 0ULL;
            if (b >= P.batch) continue;
            unsigned long long* word = P.acc + (size_t)b * P.Mp + rt * RABIT_TILE_ROWS + rl;
            if (!RABIT_IN_RANGE(rt * RABIT_TILE_ROWS + rl < P.Mp && b < RABIT_LUT_MAX_BATCH)) continue;
            if (bad[i]) atomicOr(word, 1ULL << 63);                      // sticky: the add below never carries into bit 63
            old[i] = atomicAdd(word, add[i]);
        }
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int o = tid + i * kGroupThreads, b = o >> 7, rl = o & 127;
            if (b >= P.batch) continue;
            if ((int)((old[i] >> 55) & 0xFFu) != arrivals - 1) continue;  // other segments of the row tile are still to come
            const unsigned long long sum = (old[i] & kSumMask) + (add[i] & kSumMask);
            const long long total = (long long)sum - ((long long)P.n_cs << P.fix_bits);
            const bool poisoned = bad[i] || (old[i] >> 63) != 0;
            const float v = poisoned ? __int_as_float(0x7FC00000) : __ll2float_rn(total) * P.unit;
            const int row = rt * RABIT_TILE_ROWS + rl;
            if (row < P.M) P.y[(size_t)b * P.M + row] = __float2half_rn(v);
            P.acc[(size_t)b * P.Mp + row] = 0ULL;                         // resting state for the next call
        }
        group_sync(group);                                               // the slots are free for the next segment
    }
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <int NH>
cudaError_t launch(const F16Params& P, int grid, int device, cudaStream_t stream) {
    static bool attr_done[64] = {false};
    const size_t smem = (size_t)kGroups * ((size_t)kWarps * NH * 8 * kSlotStride * sizeof(float) + (size_t)kWarps * kRing * 512);
    const int slot = device >= 0 && device < 64 ? device : 0;
    if (!attr_done[slot] || slot != device) {
        cudaError_t e = cudaFuncSetAttribute(rabit_gemv_f16_kernel<NH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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
    return cudaLaunchKernelEx(&cfg, rabit_gemv_f16_kernel<NH>, P);
}

}  // namespace

namespace {

// Cuts the n_rt * n_cs (row tile, slice) pairs, in that order, into one contiguous range per SM and every SM's range into
// two parts, one per group of its CTA.  A group's cost is its pairs plus `seg` for every segment after its first (a part
// that crosses a row-tile boundary adds up and publishes twice, and while it does so its SM runs at half strength; the last
// segment end is the same for everybody); an SM's cost is that of its slower group under the best cut between the two
// parts, which is often the row-tile boundary itself.  The SM ranges are grown greedily under a cost limit and the
// smallest limit that needs no more than `sms` ranges is found by bisection, so SMs whose range holds a boundary get
// fewer pairs.  (Equal ranges cut in the middle, the previous form, left such SMs 30-40 % late; equal-cost parts
// handed to independent CTAs, two per SM wherever the hardware put them, gave SMs unequal sums.)
// bound[] receives the starts of the 2 * grid parts (bound[2 * grid] = n_pairs); returns grid.  Plans are cached per thread.
int plan_ranges(int n_rt, int n_cs, int K, int NH, int sms, int* bound) {
    struct Plan { int n_rt, n_cs, K, NH, sms, grid; int bound[kMaxRanges + 1]; };
    static thread_local std::vector<Plan> plans;
    for (const Plan& pl : plans)
        if (pl.n_rt == n_rt && pl.n_cs == n_cs && pl.K == K && pl.NH == NH && pl.sms == sms) {
            std::memcpy(bound, pl.bound, sizeof(pl.bound));
            return pl.grid;
        }
    const long long n_pairs = (long long)n_rt * n_cs;
    const int max_grid = (int)std::min<long long>(std::min(sms, kMaxRanges / kGroups), n_pairs);
    // fitted to timelines on B200: a group works through a tile of a pair (8 K tiles) in about 0.068 us (NH = 1) or 0.085 us
    // (NH = 2), a segment end takes it 3 to 3.5 us
    const double seg = (NH == 1 ? 3.0 : 3.5) / (8.0 * K * (NH == 1 ? 0.068 : 0.085));
    auto part_cost = [&](long long a, long long b) {                     // pairs [a, b) as one group's part
        if (b <= a) return 0.0;
        const long long segments = (b - 1) / n_cs - a / n_cs + 1;
        return (double)(b - a) + seg * (double)(segments - 1);
    };
    auto best_cut = [&](long long a, long long b, double* cost) {        // the cut of [a, b) that makes the slower group fastest
        long long best = b;
        double best_cost = part_cost(a, b);
        for (long long m = a + 1; m < b; ++m) {
            const double c = std::max(part_cost(a, m), part_cost(m, b));
            if (c < best_cost) { best_cost = c; best = m; }
        }
        *cost = best_cost;
        return best;
    };
    auto cut_all = [&](double limit, int* out) {                         // greedy SM ranges under the limit; returns their number
        int n = 0;
        long long a = 0;
        while (a < n_pairs) {
            long long lo = a + 1, hi = std::min<long long>(n_pairs, a + 4 * (long long)limit + 8);   // largest b with cost <= limit
            while (lo < hi) {
                const long long mid = (lo + hi + 1) / 2;
                double c;
                best_cut(a, mid, &c);
                if (c <= limit) lo = mid; else hi = mid - 1;
            }
            if (out && n < max_grid) {
                double c;
                out[kGroups * n] = (int)a;
                out[kGroups * n + 1] = (int)best_cut(a, lo, &c);
            }
            ++n;
            if (n > max_grid && !out) return n;
            a = lo;
        }
        return n;
    };
    double lo = 1.0, hi = (double)n_pairs + seg * (n_rt + 1) + 1.0;
    if (n_pairs <= max_grid) {
        lo = hi = 0.5;                                                   // fewer pairs than SMs: one pair, one group per SM (a group alone on its SM is faster than two)
    } else if (cut_all(lo, nullptr) > max_grid) {
        for (int it = 0; it < 40; ++it) {
            const double mid = 0.5 * (lo + hi);
            if (cut_all(mid, nullptr) <= max_grid) hi = mid; else lo = mid;
        }
    } else {
        hi = lo;
    }
    int tmp[kMaxRanges + 2];
    const int grid = cut_all(hi, tmp);
    for (int r = 0; r <= kMaxRanges; ++r) bound[r] = r < kGroups * grid ? tmp[r] : (int)n_pairs;
    if (plans.size() >= 256) plans.clear();
    plans.emplace_back();
    Plan& pl = plans.back();
    pl.n_rt = n_rt; pl.n_cs = n_cs; pl.K = K; pl.NH = NH; pl.sms = sms; pl.grid = grid;
    std::memcpy(pl.bound, bound, sizeof(pl.bound));
    return grid;
}

}  // namespace

// Host-only view of the work split (for tests): the starts of the 2 * grid group parts of a K-path layer of M x N at
// `batch` rows on `sms` SMs; bound_out receives 2 * grid + 1 values, the last being the number of pairs.
int rabit_gemv_f16_plan(int K, int M, int N, int batch, int sms, int* bound_out, int max_out) {
    if (K < 1 || K > RABIT_MAX_K || M < 1 || N < 32 || (N % 32) != 0 || batch < 1 || batch > RABIT_MAX_GEMV_BATCH || sms < 1) return -1;
    const long long n_rt = ((long long)M + RABIT_TILE_ROWS - 1) / RABIT_TILE_ROWS, n_cs = ((long long)N + RABIT_LUT_COLS - 1) / RABIT_LUT_COLS;
    if (n_cs > RABIT_LUT_MAX_SLICES || n_rt * n_cs >= kMaxPairs) return -1;
    int bound[kMaxRanges + 1];
    const int grid = plan_ranges((int)n_rt, (int)n_cs, K, batch > 8 ? 2 : 1, sms, bound);
    if (max_out < kGroups * grid + 1) return -1;
    for (int r = 0; r <= kGroups * grid; ++r) bound_out[r] = bound[r];
    return grid;
}

bool rabit_gemv_f16_supports(const rabit_layer& L, int batch) {
    if (batch < 1 || batch > RABIT_MAX_GEMV_BATCH) return false;
    if (L.geom.n_cs > RABIT_LUT_MAX_SLICES || L.d_acc == nullptr) return false;
    if ((long long)L.geom.n_rt * L.geom.K * L.geom.n_ct * 32 >= (1LL << 31)) return false;   // 32-bit tile offsets in the kernel
    return (long long)L.geom.n_rt * L.geom.n_cs < kMaxPairs;
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
    P.status = L.d_status;
    P.K = G.K; P.M = G.M; P.N = G.N; P.Mp = G.Mp; P.n_rt = G.n_rt; P.n_ct = G.n_ct; P.n_cs = G.n_cs;
    P.batch = batch;
    P.fix_bits = G.fix_bits;
    P.unit = ldexpf(1.f, G.unit_exp);
    P.inv_unit = ldexpf(1.f, -G.unit_exp);
    P.limit = ldexpf(1.f, G.fix_bits);
    P.two = 2u;
    P.two_pow_8 = 256u;
    P.n_pairs = G.n_rt * G.n_cs;
    const int sms = L.sm_count > 0 ? L.sm_count : 148;
    const int grid = plan_ranges(G.n_rt, G.n_cs, G.K, batch > 8 ? 2 : 1, sms, P.bound);   // one CTA (two groups of eight warps) per SM
    return batch <= 8 ? launch<1>(P, grid, L.device, stream) : launch<2>(P, grid, L.device, stream);
}
