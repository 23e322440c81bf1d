// spMspV on the 4-bit variant of Tiled-CBC for sm_100a (Sec. 5.1: 4-bit round-to-nearest weights in the
// order static pruning -> quantisation -> dynamic pruning; Sec. 6: Values are stored apart from the
// sparsity metadata, so they can be low-bit).  TileOffset / ColInfo / Bitmap are those of Sec. 4.1
// (offsets count codes, padded to 32 per column tile); Values are 4-bit codes, two per byte, with
// one fp16 scale per column tile: weight = (code - 8) * scale.
//
// With half a byte per stored weight a column tile is at most 128 bytes of codes.  Every warp runs
// its own three-stage pipeline over the GTiles it takes from the CTA's range: (1) lanes 0-15 apply
// the DP test to the GTile's 16 activations (Sec. 4.2 step (3)) and read ColInfo and the scales of
// the active columns, two GTiles ahead; (2) the bitmaps and codes of the active columns of the next
// GTile stream into the warp's own shared-memory buffer with 16-byte asynchronous copies (inactive
// columns are never touched); (3) the current GTile is decoded from shared memory: lane l owns rows
// 8l .. 8l+7 of a column tile (one bitmap byte), rank = set bits before that byte (Sec. 4.2.1), its
// codes are one span of at most 8 nibbles, read as two 32-bit words, funnel-shifted into one register
// and walked bit by bit.  Same work split and split-K combine as the fp16 kernel (equal contiguous
// GTile ranges, pairwise exchanges along a fixed tree).
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kQWarps = 32;
constexpr int kQThreads = kQWarps * 32;

// A GTile's active columns as fetched: codes (at most 128 bytes per column tile) and bitmaps.
struct alignas(16) QWarpBuf {
    unsigned char codes[kTileK][128];
    uint32_t bm[kTileK][8];
};
struct QSmem {
    QWarpBuf buf[kQWarps][2];
    float red[kQWarps][kTileM];
};

struct QParams {
    const uint32_t* tileoffset;
    const uint32_t* colinfo;
    const uint32_t* bitmap32;       // the bitmap as 32-bit words: 8 per column tile
    const unsigned char* codes;
    const __half* scales;
    const __half* x;
    const uint32_t* mask;
    void* y;
    float thr;
    int rule;
    int ydt;
    int M, K, R, C;
    int64_t NGT;
    int num_ctas;
    float* workspace;               // [num_ctas][256] tree nodes, all zero between calls
    int* status;
    int64_t codes_len;              // codes in the array (checked build)
};

// The walk over a lane's 8 rows (Sec. 4.2.1 with 4-bit codes): a set bit takes the next nibble of `span`;
// (code | 0x4B000000) is 2^23 + code as a float, so one subtraction turns the code into code - 8 without a
// conversion; acc[row] += (code - 8) * (scale * x).  Five instructions per row, the last two predicated.
#define SPDP_Q4_ROW(K)                                              \
    " lop3.or.b32 t|p, %9, " #K ", 0, 0xC0, 0;\n"                  \
    " lop3.b32 c, %8, 15, 0x4B000000, 0xEA;\n"                     \
    " mov.b32 w, c;\n"                                             \
    " add.f32 w, w, 0fCB000008;\n"
__device__ __forceinline__ void walk_codes(unsigned bits, unsigned span, float sx, float (&acc)[8]) {
    asm volatile(
        "{\n"
        " .reg .pred p;\n"
        " .reg .b32 t, c;\n"
        " .reg .f32 w;\n"
        SPDP_Q4_ROW(1)   " @p fma.rn.f32 %0, w, %10, %0;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(2)   " @p fma.rn.f32 %1, w, %10, %1;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(4)   " @p fma.rn.f32 %2, w, %10, %2;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(8)   " @p fma.rn.f32 %3, w, %10, %3;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(16)  " @p fma.rn.f32 %4, w, %10, %4;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(32)  " @p fma.rn.f32 %5, w, %10, %5;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(64)  " @p fma.rn.f32 %6, w, %10, %6;\n @p shr.b32 %8, %8, 4;\n"
        SPDP_Q4_ROW(128) " @p fma.rn.f32 %7, w, %10, %7;\n"
        "}"
        : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3]), "+f"(acc[4]), "+f"(acc[5]), "+f"(acc[6]), "+f"(acc[7]),
          "+r"(span)
        : "r"(bits), "f"(sx));
}

__global__ void __launch_bounds__(kQThreads, 1)
spmspv_q4_kernel(const __grid_constant__ QParams p) {
    extern __shared__ __align__(128) unsigned char q4_smem_raw[];
    QSmem& sm = *reinterpret_cast<QSmem*>(q4_smem_raw);
    float (*red)[kTileM] = sm.red;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const unsigned ngt_all = static_cast<unsigned>(p.NGT), nctas = static_cast<unsigned>(p.num_ctas);
    const unsigned g_begin = range_begin(ngt_all, nctas, blockIdx.x), g_end = range_begin(ngt_all, nctas, blockIdx.x + 1);
    const int my_word = lane >> 2, my_shift = 8 * (lane & 3);
    const int fcol = lane >> 3, fpiece = lane & 7;      // fetch role: column (of a quad) and 16-byte piece

    for (unsigned g0 = g_begin; g0 < g_end;) {
        // ---- one segment: this CTA's share of row tile r ----
        const int r = static_cast<int>(g0 / static_cast<unsigned>(p.C));
        const int c0 = static_cast<int>(g0 - static_cast<unsigned>(r) * static_cast<unsigned>(p.C));
        int ngt = p.C - c0;
        if (ngt > static_cast<int>(g_end - g0)) ngt = static_cast<int>(g_end - g0);
        float acc[8];                       // rows 8*lane .. 8*lane+7 of the row tile
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;

        // what lanes 0-15 know about "their" column of a GTile, and the GTile's start in Codes
        struct GMeta { unsigned am, ci, to; float sx; };
        auto load_meta = [&](int gi) -> GMeta {
            GMeta m = {0u, 0u, 0u, 0.f};
            if (gi >= ngt) return m;
            const int64_t g = static_cast<int64_t>(g0) + gi;
            const int j = (c0 + gi) * kTileK + (lane & 15);
            bool act = false;
            if (lane < kTileK && j < p.K) {
                const __half xj = p.x[j];
                if (p.rule == SPDP_DP_NONE) act = true;
                else if (p.rule == SPDP_DP_ABS_GT) act = !(fabsf(__half2float(xj)) <= p.thr);
                else act = (__ldg(p.mask + (j >> 5)) >> (j & 31)) & 1u;
                if (act) {
                    m.ci = __ldg(p.colinfo + g * kTileK + lane);
                    m.sx = __half2float(__ldg(p.scales + g * kTileK + lane)) * __half2float(xj);   // exact in fp32
                }
            }
            m.am = __ballot_sync(0xFFFFFFFFu, act) & 0xFFFFu;
            m.to = __ldg(p.tileoffset + g);
            return m;
        };
        // starts the copies of the active columns of GTile gi into one of the warp's two buffers
        auto fetch = [&](int gi, const GMeta& m, QWarpBuf& b) {
            if (gi < ngt) {
                const int64_t g = static_cast<int64_t>(g0) + gi;
#pragma unroll
                for (int q = 0; q < kTileK / 4; ++q) {
                    const int c = 4 * q + fcol;
                    const unsigned ci_c = __shfl_sync(0xFFFFFFFFu, m.ci, c);
                    if ((m.am >> c) & 1u) {
                        const unsigned n = ci_c & 0xFFFFu, first = m.to + (ci_c >> 16);
                        int pieces = static_cast<int>((n + 31u) >> 5);
                        if (!SPDP_CHECK(p.status, first, 32 * pieces, p.codes_len, kSiteValuesSpan) ||
                            !SPDP_CHECK(p.status, 0, pieces, 8, kSitePieces))
                            pieces = 0;                                          // checked build only: the tile is left out
                        if (fpiece < pieces)
                            cp_async16<0>(smem_u32(&b.codes[c][16 * fpiece]), p.codes + (first >> 1) + 16 * fpiece, 1);
                        if (fpiece < 2) {
                            if (pieces > 0 || n == 0u)
                                cp_async16<0>(smem_u32(&b.bm[c][4 * fpiece]),
                                              reinterpret_cast<const unsigned char*>(p.bitmap32) + (g * kTileK + c) * 32 + 16 * fpiece, 1);
                            else
                                *reinterpret_cast<uint4*>(&b.bm[c][4 * fpiece]) = make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                }
            }
            cp_async_commit();
        };

        GMeta cur = load_meta(warp);
        fetch(warp, cur, sm.buf[warp][0]);
        GMeta nxt = load_meta(warp + kQWarps);
        int k = 0;
        for (int gi = warp; gi < ngt; gi += kQWarps, ++k) {
            fetch(gi + kQWarps, nxt, sm.buf[warp][(k + 1) & 1]);        // the next GTile's copies
            const GMeta nxt2 = load_meta(gi + 2 * kQWarps);             // and the metadata of the one after it
            cp_async_wait<1>();                                         // this GTile's copies have arrived
            __syncwarp();
            const QWarpBuf& b = sm.buf[warp][k & 1];
            unsigned am = cur.am;
            while (am != 0u) {
                const int cc = __ffs(am) - 1;
                am &= am - 1u;
                const float sx_c = __shfl_sync(0xFFFFFFFFu, cur.sx, cc);
                // set bits before each of the 8 words: a scan over 8-lane segments (every segment holds the 8 words)
                const unsigned w8 = b.bm[cc][lane & 7];
                const unsigned cnt = __popc(w8);
                unsigned inc = cnt;
                scan8_level<1>(inc);
                scan8_level<2>(inc);
                scan8_level<4>(inc);
                const unsigned wd = __shfl_sync(0xFFFFFFFFu, w8, my_word);
                const unsigned before = __shfl_sync(0xFFFFFFFFu, inc - cnt, my_word);
                const unsigned bits = (wd >> my_shift) & 0xFFu;                  // my 8 rows
                if (bits != 0u) {
                    const unsigned rank = before + __popc(wd & ((1u << my_shift) - 1u));
                    // my codes: at most 8 nibbles from nibble `rank` on, inside two consecutive 32-bit words
                    const uint32_t* cw = reinterpret_cast<const uint32_t*>(&b.codes[cc][0]) + (rank >> 3);
                    unsigned span = __funnelshift_r(cw[0], cw[1], 4 * (rank & 7u));
                    walk_codes(bits, span, sx_c, acc);
                }
            }
            __syncwarp();                                               // the buffer may be refilled
            cur = nxt;
            nxt = nxt2;
        }
        cp_async_wait<0>();
        // ---- cross-warp sums in warp order, split-K combine, store ----
        *reinterpret_cast<float4*>(&red[warp][8 * lane]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        *reinterpret_cast<float4*>(&red[warp][8 * lane + 4]) = make_float4(acc[4], acc[5], acc[6], acc[7]);
        __syncthreads();
        if (t < kTileM) {
            float part = 0.f;
#pragma unroll
            for (int w = 0; w < kQWarps; ++w) part += red[w][t];
            const int64_t row = static_cast<int64_t>(r) * kTileM + t;
            if (row < p.M) {
                const int q0 = range_owner(ngt_all, nctas, static_cast<unsigned>(r) * p.C);
                const int nseg = range_owner(ngt_all, nctas, static_cast<unsigned>(r + 1) * p.C - 1u) - q0 + 1;
                if (SPDP_CHECK(p.status, q0, nseg, p.num_ctas, kSiteTreeNodes) &&
                    SPDP_CHECK(p.status, static_cast<int>(blockIdx.x) - q0, 1, nseg, kSiteTreeNodes) &&
                    tree_combine(part, reinterpret_cast<unsigned*>(p.workspace) + t, kTileM, q0, nseg,
                                 static_cast<int>(blockIdx.x) - q0))
                    store_y(p.y, p.ydt, row, part);
            }
        }
        __syncthreads();
        g0 += static_cast<unsigned>(ngt);
    }
}

}  // namespace

spdp_status configure_spmspv_q4_kernel() {
    static std::mutex mu;
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SPDP_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(spmspv_q4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(sizeof(QSmem))));
        configured[dev] = true;
    }
    return SPDP_OK;
}

spdp_status launch_spmspv_q4(const spdp_matrix* h, const __half* x, int rule, float thr, const uint32_t* mask, void* y,
                             int ydt, cudaStream_t s) {
    QParams p;
    p.tileoffset = h->tileoffset;
    p.colinfo = h->colinfo;
    p.bitmap32 = reinterpret_cast<const uint32_t*>(h->bitmap);
    p.codes = reinterpret_cast<const unsigned char*>(h->values);
    p.scales = h->scales;
    p.x = x;
    p.mask = mask;
    p.y = y;
    p.thr = thr;
    p.rule = rule;
    p.ydt = ydt;
    p.M = static_cast<int>(h->M);
    p.K = static_cast<int>(h->K);
    p.R = static_cast<int>(h->R);
    p.C = static_cast<int>(h->C);
    p.NGT = h->NGT;
    p.num_ctas = h->num_ctas;
    p.workspace = h->workspace;
    p.status = h->status_word;
    p.codes_len = h->values_len;
    spdp_status st = configure_spmspv_q4_kernel();
    if (st != SPDP_OK) return st;
    spmspv_q4_kernel<<<static_cast<unsigned>(h->num_ctas), kQThreads, sizeof(QSmem), s>>>(p);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
