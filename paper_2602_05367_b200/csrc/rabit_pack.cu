// Host-side packing of canonical sign planes + scales into the device layout
// (step "pack" of the layer; Appendix "Weight Packing" of the paper fixes only the
// sign -> bit rule, the tile arrangement is described in rabit_layout.h).
#include <algorithm>
#include <cmath>
#include <cstring>
#include <thread>
#include <vector>

#include "rabit_internal.h"

static float half_bits_to_float(uint16_t v) {
    const uint32_t sign = (uint32_t)(v & 0x8000u) << 16;
    const int e = (v >> 10) & 0x1F;
    uint32_t m = v & 0x3FFu, bits;
    if (e == 0) {
        if (m == 0) bits = sign;
        else {                                  // subnormal: normalise
            int sh = 0;
            while (!(m & 0x400u)) { m <<= 1; ++sh; }
            bits = sign | ((uint32_t)(127 - 15 - sh + 1) << 23) | ((m & 0x3FFu) << 13);
        }
    } else if (e == 31) bits = sign | 0x7F800000u | (m << 13);
    else bits = sign | ((uint32_t)(e - 15 + 127) << 23) | (m << 13);
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

bool rabit_make_geom(int K, int M, int N, RabitGeom* out) {
    if (K < 1 || K > RABIT_MAX_K || M < 1 || N < 32 || (N % 32) != 0) return false;
    if ((long long)M > (1 << 24) || (long long)N > (1 << 24)) return false;
    RabitGeom G;
    G.K = K; G.M = M; G.N = N;
    G.Mp = (M + RABIT_TILE_ROWS - 1) / RABIT_TILE_ROWS * RABIT_TILE_ROWS;
    G.n_rt = G.Mp / RABIT_TILE_ROWS;
    G.n_ct = N / RABIT_TILE_COLS;
    for (int k = 0; k < RABIT_MAX_K; ++k) G.hmax[k] = 0.f;
    G.n_rb = G.Mp / RABIT_LUT_ROWS;
    G.n_cs = (N + RABIT_LUT_COLS - 1) / RABIT_LUT_COLS;
    G.fix_bits = 0;
    G.unit_exp = 0;
    *out = G;
    return true;
}

// Everything the header records about the scales: max_j |h_k[j]| per path (the integer-MMA GEMV derives its
// fixed-point scale from it) and the fixed-point grid of the table-driven GEMV's accumulate words.
//
// That GEMV adds, per output row, one partial sum per 256-column slice into a 64-bit word with an integer
// atomic.  A partial sum is bounded, for ANY finite fp16 activations, by
//     65504 * max_i sum_k |g_k[i]| * max_{k, slice} sum_{j in slice} |h_k[j]|,
// so a grid of 2^unit_exp whose 2^fix_bits steps cover twice that bound can never overflow, and with
// fix_bits = 54 - ceil(log2(slices)) the sum of all slices (each shifted to be non-negative) stays below 2^55.
// |value| of every fp16 magnitude (sign bit cleared), converted once: the scans below are table look-ups
static const float* half_magnitude_table() {
    static const std::vector<float> table = [] {
        std::vector<float> t(32768);
        for (uint32_t m = 0; m < 32768; ++m) t[m] = half_bits_to_float((uint16_t)m);
        return t;
    }();
    return table.data();
}

void rabit_scale_meta(const uint16_t* g, const uint16_t* h, int K, int M, int N, RabitGeom* G) {
    const float* mag = half_magnitude_table();
    // one pass over h: per path the largest |h| (fp16 magnitudes order like their bit patterns; the first NaN wins and
    // sticks, so a NaN scale makes the bound NaN) and per slice of 256 columns the sum of |h|, added in column order
    double hsum_max = 0.0;
    for (int k = 0; k < K; ++k) {
        const uint16_t* hk = h + (size_t)k * N;
        uint32_t top = 0, first_nan = 0;
        for (int j0 = 0; j0 < N; j0 += RABIT_LUT_COLS) {
            const int j1 = j0 + RABIT_LUT_COLS < N ? j0 + RABIT_LUT_COLS : N;
            double s = 0.0;
            for (int j = j0; j < j1; ++j) {
                const uint32_t m = hk[j] & 0x7FFFu;
                if (m > 0x7C00u && first_nan == 0) first_nan = m;
                top = m > top ? m : top;
                s += (double)mag[m];
            }
            if (s > hsum_max || s != s) hsum_max = s;
        }
        G->hmax[k] = mag[first_nan ? first_nan : top];
    }
    double gsum_max = 0.0;
    for (int i = 0; i < M; ++i) {
        double s = 0.0;
        for (int k = 0; k < K; ++k) s += (double)mag[g[(size_t)k * M + i] & 0x7FFFu];
        if (s > gsum_max || s != s) gsum_max = s;
    }
    int clog = 0;
    while ((1 << clog) < G->n_cs) ++clog;
    G->fix_bits = 54 - clog;
    const double bound = 65504.0 * gsum_max * hsum_max;
    int e = 0;
    if (bound == bound && bound > 0.0 && bound < 1e300) {
        int ex = 0;
        std::frexp(bound, &ex);                       // bound < 2^ex
        e = ex + 1;                                   // one spare bit for the fp32 roundings of the kernel
    }
    if (e < -40) e = -40;                             // keeps 2^(fix_bits - e) inside fp32
    if (e > 100) e = 100;
    G->unit_exp = e - G->fix_bits;
}

void rabit_fill_header(const RabitGeom& G, RabitHeader* hdr) {
    std::memset(hdr, 0, sizeof(RabitHeader));
    hdr->magic = RABIT_MAGIC;
    hdr->version = RABIT_LAYOUT_VERSION;
    hdr->K = G.K; hdr->M = G.M; hdr->N = G.N; hdr->Mp = G.Mp;
    hdr->n_rt = G.n_rt; hdr->n_ct = G.n_ct;
    hdr->max_grid = RABIT_MAX_GRID;
    hdr->partial_batch = RABIT_PARTIAL_BATCH;
    for (int k = 0; k < G.K; ++k) std::memcpy(&hdr->hmax_bits[k], &G.hmax[k], 4);
    hdr->n_rb = G.n_rb; hdr->n_cs = G.n_cs;
    hdr->fix_bits = (uint32_t)G.fix_bits; hdr->unit_exp = G.unit_exp;
    size_t off = RABIT_HEADER_BYTES;
    hdr->off_bits = off;     off = rabit_align256(off + (size_t)G.K * G.n_rt * G.n_ct * RABIT_TILE_BYTES);
    hdr->off_g = off;        off = rabit_align256(off + (size_t)G.K * G.Mp * 2);
    hdr->off_h = off;        off = rabit_align256(off + (size_t)G.K * G.N * 2);
    hdr->off_partial = off;  off = rabit_align256(off + ((size_t)G.n_rt * G.K + RABIT_MAX_GRID) * RABIT_PARTIAL_BATCH * RABIT_TILE_ROWS * 4);
    hdr->off_flags = off;    off = rabit_align256(off + ((size_t)G.n_rt * G.K + RABIT_MAX_GRID) * 4 + 4);   // + one status word
    hdr->off_lut = off;      off = rabit_align256(off + (size_t)G.n_cs * G.n_rb * G.K * RABIT_LUT_PART_BYTES);
    hdr->off_acc = off;      off = rabit_align256(off + (size_t)RABIT_LUT_MAX_BATCH * G.Mp * 8);
    hdr->total_bytes = off;
}

bool rabit_geom_from_header(const RabitHeader& hdr, RabitGeom* out) {
    if (hdr.magic != RABIT_MAGIC || hdr.version != RABIT_LAYOUT_VERSION) return false;
    if (!rabit_make_geom((int)hdr.K, (int)hdr.M, (int)hdr.N, out)) return false;
    if (hdr.max_grid != RABIT_MAX_GRID || hdr.partial_batch != RABIT_PARTIAL_BATCH) return false;
    for (int k = 0; k < out->K; ++k) std::memcpy(&out->hmax[k], &hdr.hmax_bits[k], 4);
    if (hdr.n_rb != (uint32_t)out->n_rb || hdr.n_cs != (uint32_t)out->n_cs) return false;
    out->fix_bits = (int)hdr.fix_bits;
    out->unit_exp = hdr.unit_exp;
    return true;
}

extern "C" int rabit_layout_version(void) { return RABIT_LAYOUT_VERSION; }

extern "C" size_t rabit_packed_bytes(int K, int M, int N) {
    RabitGeom G;
    if (!rabit_make_geom(K, M, N, &G)) return 0;
    RabitHeader hdr;
    rabit_fill_header(G, &hdr);
    return (size_t)hdr.total_bytes;
}

// bit i of the low byte of v -> least significant bit of byte i of the result
static inline uint64_t spread8(uint32_t v) {
    uint64_t m = ((uint64_t)(v & 0xFFu) * 0x0101010101010101ULL) & 0x8040201008040201ULL;
    return ((m + 0x7F7F7F7F7F7F7F7FULL) >> 7) & 0x0101010101010101ULL;
}

static void pack_tile(const RabitGeom& G, const uint32_t* plane /*[M][N/32]*/, int rt, int ct, uint8_t* dst) {
    const int words_per_row = G.N / 32;
    for (int r16 = 0; r16 < 16; ++r16) {            // r16 = gq + 8 * (a & 1): row inside a 16-row block
        // bytes[q] byte b collects, for column 8q + b of the tile, bit p <- row 16p + r16
        uint64_t bytes[4] = {0, 0, 0, 0};
        for (int p = 0; p < 8; ++p) {
            const int row = rt * RABIT_TILE_ROWS + 16 * p + r16;
            uint32_t s = 0;
            if (row < G.M) s = plane[(size_t)row * words_per_row + ct];
            for (int q = 0; q < 4; ++q) bytes[q] |= spread8(s >> (8 * q)) << p;
        }
        const int gq = r16 & 7, alo = r16 >> 3;
        for (int j4 = 0; j4 < 8; ++j4) {            // 4 consecutive columns = the four bytes of one word
            const int j = j4 * 4;
            const int ah = j >> 4, tq = (j >> 2) & 3;
            const int a = alo | (ah << 1);
            const uint32_t v = (uint32_t)(bytes[j >> 3] >> (8 * (j & 7)));
            std::memcpy(dst + (4 * gq + tq) * 16 + a * 4, &v, 4);
        }
    }
}

// Header and the two scale sections for a layer whose tiles are produced elsewhere.
// `tail` receives off_partial - off_g bytes (the image from off_g up to the scratch sections).
bool rabit_build_meta(const uint16_t* g, const uint16_t* h, int K, int M, int N, RabitGeom* geom, RabitHeader* hdr,
                      std::vector<uint8_t>* tail) {
    RabitGeom G;
    if (!rabit_make_geom(K, M, N, &G)) return false;
    rabit_scale_meta(g, h, K, M, N, &G);
    rabit_fill_header(G, hdr);
    tail->assign((size_t)(hdr->off_partial - hdr->off_g), 0);
    uint8_t* base = tail->data() - hdr->off_g;                    // so that image offsets can be used
    uint16_t* gp = (uint16_t*)(base + hdr->off_g);
    uint16_t* hp = (uint16_t*)(base + hdr->off_h);
    for (int k = 0; k < K; ++k) {
        std::memcpy(gp + (size_t)k * G.Mp, g + (size_t)k * M, (size_t)M * 2);
        std::memcpy(hp + (size_t)k * N, h + (size_t)k * N, (size_t)N * 2);
    }
    *geom = G;
    return true;
}

extern "C" int rabit_pack_host(const uint32_t* planes, const uint16_t* g, const uint16_t* h,
                               int K, int M, int N, void* out, size_t out_bytes) {
    rabit_clear_error();
    if (!planes || !g || !h || !out) return rabit_fail(RABIT_INVALID_ARG, "rabit_pack_host: null pointer");
    RabitGeom G;
    if (!rabit_make_geom(K, M, N, &G))
        return rabit_fail(RABIT_UNSUPPORTED_SHAPE, "rabit_pack_host: unsupported shape K=%d M=%d N=%d (need 1<=K<=3, M>=1, N%%32==0)", K, M, N);
    rabit_scale_meta(g, h, K, M, N, &G);
    RabitHeader hdr;
    rabit_fill_header(G, &hdr);
    if (out_bytes < hdr.total_bytes)
        return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_pack_host: need %zu bytes, got %zu", (size_t)hdr.total_bytes, out_bytes);
    uint8_t* base = (uint8_t*)out;
    std::memset(base, 0, hdr.total_bytes);
    std::memcpy(base, &hdr, sizeof(hdr));
    std::memset(base + hdr.off_partial, 0xFF, hdr.off_flags - hdr.off_partial);   // resting state of the partial buffer

    uint8_t* bits = base + hdr.off_bits;
    const size_t plane_words = (size_t)M * (N / 32);
    int nthreads = (int)std::min<unsigned>(std::max(1u, std::thread::hardware_concurrency()), 32u);
    if ((size_t)G.n_rt * G.n_ct < 4096) nthreads = 1;
    auto work = [&](int tid) {
        for (int rt = tid; rt < G.n_rt; rt += nthreads)
            for (int k = 0; k < K; ++k)
                for (int ct = 0; ct < G.n_ct; ++ct)
                    pack_tile(G, planes + (size_t)k * plane_words, rt, ct,
                              bits + rabit_tile_pos(G, rt, k, ct) * RABIT_TILE_BYTES);
    };
    // look-up blocks: the canonical bytes (eight consecutive columns of one row), permuted
    uint8_t* lut = base + hdr.off_lut;
    const int row_bytes = N / 8;
    auto work_lut = [&](int tid) {
        for (int k = 0; k < K; ++k)
            for (int row = tid; row < M; row += nthreads) {
                const uint8_t* src = reinterpret_cast<const uint8_t*>(planes + (size_t)k * plane_words + (size_t)row * (N / 32));
                for (int cb = 0; cb < row_bytes; ++cb) lut[rabit_lut_byte_offset(G, k, row, cb)] = src[cb];
            }
    };
    if (nthreads == 1) {
        work(0);
        work_lut(0);
    } else {
        std::vector<std::thread> pool;
        for (int t = 0; t < nthreads; ++t) pool.emplace_back(work, t);
        for (auto& th : pool) th.join();
        pool.clear();
        for (int t = 0; t < nthreads; ++t) pool.emplace_back(work_lut, t);
        for (auto& th : pool) th.join();
    }
    uint16_t* gp = (uint16_t*)(base + hdr.off_g);
    uint16_t* hp = (uint16_t*)(base + hdr.off_h);
    for (int k = 0; k < K; ++k) {
        std::memcpy(gp + (size_t)k * G.Mp, g + (size_t)k * M, (size_t)M * 2);
        std::memcpy(hp + (size_t)k * N, h + (size_t)k * N, (size_t)N * 2);
    }
    return RABIT_OK;
}

extern "C" int rabit_unpack_host(const void* image, size_t image_bytes,
                                 uint32_t* planes_out, uint16_t* g_out, uint16_t* h_out) {
    rabit_clear_error();
    if (!image) return rabit_fail(RABIT_INVALID_ARG, "rabit_unpack_host: null image");
    if (image_bytes < sizeof(RabitHeader)) return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_unpack_host: image smaller than its header");
    RabitHeader hdr;
    std::memcpy(&hdr, image, sizeof(hdr));
    RabitGeom G;
    if (!rabit_geom_from_header(hdr, &G))
        return rabit_fail(RABIT_INVALID_ARG, "rabit_unpack_host: not a packed image of layout version %d", RABIT_LAYOUT_VERSION);
    if (image_bytes < hdr.total_bytes) return rabit_fail(RABIT_BUFFER_TOO_SMALL, "rabit_unpack_host: image truncated");
    const uint8_t* base = (const uint8_t*)image;
    const int K = G.K, M = G.M, N = G.N, words_per_row = N / 32;
    if (planes_out) {
        std::memset(planes_out, 0, (size_t)K * M * words_per_row * 4);
        const uint8_t* bits = base + hdr.off_bits;
        for (int rt = 0; rt < G.n_rt; ++rt)
            for (int k = 0; k < K; ++k)
                for (int ct = 0; ct < G.n_ct; ++ct) {
                    const uint8_t* tile = bits + rabit_tile_pos(G, rt, k, ct) * RABIT_TILE_BYTES;
                    for (int lane = 0; lane < 32; ++lane)
                        for (int a = 0; a < 4; ++a)
                            for (int c = 0; c < 4; ++c) {
                                const uint8_t byte = tile[lane * 16 + a * 4 + c];
                                if (!byte) continue;
                                const int gq = lane >> 2, tq = lane & 3;
                                for (int p = 0; p < 8; ++p) {
                                    if (!((byte >> p) & 1)) continue;
                                    const int row = rt * RABIT_TILE_ROWS + 16 * p + gq + 8 * (a & 1);
                                    const int col = ct * RABIT_TILE_COLS + 16 * (a >> 1) + 4 * tq + c;
                                    if (row < M)
                                        planes_out[((size_t)k * M + row) * words_per_row + col / 32] |= 1u << (col % 32);
                                }
                            }
                }
    }
    if (planes_out) {
        // the look-up blocks must describe the same signs as the tiles
        const uint8_t* lut = base + hdr.off_lut;
        for (int k = 0; k < K; ++k)
            for (int row = 0; row < M; ++row) {
                const uint8_t* want = reinterpret_cast<const uint8_t*>(planes_out + ((size_t)k * M + row) * words_per_row);
                for (int cb = 0; cb < N / 8; ++cb)
                    if (lut[rabit_lut_byte_offset(G, k, row, cb)] != want[cb])
                        return rabit_fail(RABIT_INVALID_ARG, "rabit_unpack_host: the tile section and the look-up section disagree (path %d, row %d, columns %d..%d)",
                                          k, row, 8 * cb, 8 * cb + 7);
            }
    }
    const uint16_t* gp = (const uint16_t*)(base + hdr.off_g);
    const uint16_t* hp = (const uint16_t*)(base + hdr.off_h);
    for (int k = 0; k < K; ++k) {
        if (g_out) std::memcpy(g_out + (size_t)k * M, gp + (size_t)k * G.Mp, (size_t)M * 2);
        if (h_out) std::memcpy(h_out + (size_t)k * N, hp + (size_t)k * N, (size_t)N * 2);
    }
    return RABIT_OK;
}
