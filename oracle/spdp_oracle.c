/* CPU oracle for the SPDP decode path, in plain C (full-size matrices, timed CPU baseline).
 *
 * TEST INFRASTRUCTURE ONLY.  Loaded through ctypes by oracle/c_oracle.py, which only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg may use.  Shares no code,
 * header, table or constant with the CUDA library.
 *
 * The functions restate, loop for loop, what the paper defines:
 *   - Tiled-CBC arrays (Sec. 4.1, Storage Structure): GTiles of 256 x 16 in row-major GTile
 *     order; per column tile four 64-bit bitmap words; Values in tile-column order, each
 *     column padded to a multiple of `pad` fp16 (Sec. 4.2.3: 16 bytes = 8 elements);
 *     ColInfo = (offset of the column inside the tile) << 16 | (nonzeros of the column).
 *   - DP active set (Sec. 2.2 "Dynamic Pruning"; Sec. 4.2 step (3)): magnitude of x_j against a
 *     scalar threshold.
 *   - y = W_sp . (x masked by DP) as the plain sum over the dense masked matrix (Sec. 2.2), in
 *     fp64, with the error scale S_i = sum |W_ij x_j| the parity gate uses.
 * Readings where the paper is silent are the same as in spdp_oracle.py (bit b of word w is row
 * 64w+b; offsets in fp16 elements; nonzero iff (bits & 0x7FFF) != 0; active iff
 * !(|x_j| <= thr) in fp32; zero extension of ragged edges).
 *
 * Parity pins: tests/test_oracle_c.py compares every function here with spdp_oracle.py (an
 * independent NumPy statement of the same definitions) and the fp16 widening with NumPy's for
 * all 65536 bit patterns.  Bit/word order and offset units stay "parity unpinned" against the
 * authors' own files, which do not exist here.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { TILE_M = 256, TILE_K = 16, WORDS = 4 };

/* fp16 bit pattern -> double, exactly (sign, 5-bit exponent, 10-bit fraction). */
double oracle_half_to_double(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int f = h & 0x3FF;
    double v;
    if (e == 0)        v = ldexp((double)f, -24);                 /* zero and subnormals */
    else if (e == 31)  v = f ? NAN : INFINITY;
    else               v = ldexp((double)(f + 1024), e - 25);     /* 1.f * 2^(e-15) */
    return sign ? -v : v;
}

static int64_t pad_up(int64_t n, int64_t pad) { return (n + pad - 1) / pad * pad; }

/* Dense row-major fp16 W (leading dimension ldw) -> Tiled-CBC arrays.
 * tileoffset[NGT+1], colinfo[NGT*16], bitmap[NGT*16*4] are always written.  values may be NULL
 * (sizing call); otherwise it must hold the returned number of fp16 elements.
 * Returns the length of Values in elements, or -1 if it does not fit 32 bits. */
int64_t oracle_pack(const uint16_t* W, int64_t M, int64_t K, int64_t ldw, int64_t pad,
                    uint32_t* tileoffset, uint32_t* colinfo, uint64_t* bitmap, uint16_t* values) {
    int64_t R = (M + TILE_M - 1) / TILE_M, C = (K + TILE_K - 1) / TILE_K;
    int64_t len = 0;
    for (int64_t r = 0; r < R; ++r)
        for (int64_t c = 0; c < C; ++c) {
            int64_t g = r * C + c;                 /* GTiles in row-major order */
            int64_t tile_start = len;
            if (tile_start >= ((int64_t)1 << 32)) return -1;
            tileoffset[g] = (uint32_t)tile_start;
            for (int cc = 0; cc < TILE_K; ++cc) {
                int64_t j = c * TILE_K + cc, slot = g * TILE_K + cc;
                int64_t off = len - tile_start, n = 0;
                for (int w = 0; w < WORDS; ++w) bitmap[slot * WORDS + w] = 0;
                if (j < K)
                    for (int p = 0; p < TILE_M; ++p) {
                        int64_t i = r * TILE_M + p;
                        if (i >= M) break;
                        uint16_t h = W[i * ldw + j];
                        if ((h & 0x7FFF) != 0) {
                            bitmap[slot * WORDS + p / 64] |= (uint64_t)1 << (p % 64);
                            if (values) values[len + n] = h;
                            ++n;
                        }
                    }
                int64_t padded = pad_up(n, pad);
                if (values) for (int64_t q = n; q < padded; ++q) values[len + q] = 0;
                len += padded;
                colinfo[slot] = (uint32_t)((off << 16) | n);
            }
        }
    if (len >= ((int64_t)1 << 32)) return -1;
    tileoffset[R * C] = (uint32_t)len;
    return len;
}

/* Tiled-CBC arrays -> dense row-major fp16 (every element written; absent ones are +0). */
void oracle_unpack(int64_t M, int64_t K, const uint32_t* tileoffset, const uint32_t* colinfo,
                   const uint64_t* bitmap, const uint16_t* values, uint16_t* W, int64_t ldw) {
    int64_t R = (M + TILE_M - 1) / TILE_M, C = (K + TILE_K - 1) / TILE_K;
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < K; ++j) W[i * ldw + j] = 0;
    for (int64_t r = 0; r < R; ++r)
        for (int64_t c = 0; c < C; ++c)
            for (int cc = 0; cc < TILE_K; ++cc) {
                int64_t g = r * C + c, slot = g * TILE_K + cc, j = c * TILE_K + cc;
                int64_t next = (int64_t)tileoffset[g] + (colinfo[slot] >> 16);
                for (int p = 0; p < TILE_M; ++p)
                    if ((bitmap[slot * WORDS + p / 64] >> (p % 64)) & 1) {
                        int64_t i = r * TILE_M + p;
                        if (i < M && j < K) W[i * ldw + j] = values[next];
                        ++next;
                    }
            }
}

/* DP rule -> active[j] in {0,1}; returns the number of active columns.
 * rule 0: all active.  rule 1: active iff !(|x_j| <= thr) in fp32.  rule 2: explicit bit mask,
 * bit j%32 of word j/32. */
int64_t oracle_active(const uint16_t* x, int64_t K, int rule, float thr, const uint32_t* mask,
                      uint8_t* active) {
    int64_t count = 0;
    for (int64_t j = 0; j < K; ++j) {
        int a;
        if (rule == 0) a = 1;
        else if (rule == 1) {
            float xf = (float)oracle_half_to_double(x[j]);   /* fp16 -> fp32 is exact */
            a = !(fabsf(xf) <= thr);
        } else a = (mask[j / 32] >> (j % 32)) & 1;
        active[j] = (uint8_t)a;
        count += a;
    }
    return count;
}

/* y[i] = sum_{j active} W[i][j] x[j] and S[i] = sum_{j active} |W[i][j] x[j]|, fp64, over the
 * dense masked matrix; rows are split across `threads` OpenMP threads (<= 0: all cores).
 * Returns the number of threads used. */
int oracle_spmspv(const uint16_t* W, int64_t M, int64_t K, int64_t ldw, const uint16_t* x,
                  const uint8_t* active, double* y, double* S, int threads) {
    double* xd = (double*)__builtin_malloc((size_t)(K > 0 ? K : 1) * sizeof(double));
    for (int64_t j = 0; j < K; ++j) xd[j] = oracle_half_to_double(x[j]);
    int used = 1;
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
    used = threads;
#pragma omp parallel for num_threads(threads) schedule(static)
#endif
    for (int64_t i = 0; i < M; ++i) {
        double acc = 0.0, sc = 0.0;
        const uint16_t* row = W + i * ldw;
        for (int64_t j = 0; j < K; ++j)
            if (active[j]) {
                double t = oracle_half_to_double(row[j]) * xd[j];
                acc += t;
                sc += fabs(t);
            }
        y[i] = acc;
        if (S) S[i] = sc;
    }
    __builtin_free(xd);
    return used;
}

/* Algorithmic bytes of one call (same model as active_bytes in spdp_oracle.py). */
int64_t oracle_active_bytes(int64_t M, int64_t K, int64_t pad, const uint32_t* colinfo,
                            const uint8_t* active, int64_t y_bytes_per_elem) {
    int64_t R = (M + TILE_M - 1) / TILE_M, C = (K + TILE_K - 1) / TILE_K;
    int64_t total = 0, gt_active = 0;
    for (int64_t c = 0; c < C; ++c) {
        int any = 0;
        for (int cc = 0; cc < TILE_K; ++cc) {
            int64_t j = c * TILE_K + cc;
            if (j < K && active[j]) {
                any = 1;
                for (int64_t r = 0; r < R; ++r) {
                    int64_t n = colinfo[(r * C + c) * TILE_K + cc] & 0xFFFF;
                    total += 32 + 2 * pad_up(n, pad) + 4;
                }
            }
        }
        gt_active += any ? R : 0;
    }
    return total + 4 * (gt_active + 1) + 2 * K + y_bytes_per_elem * M;
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
