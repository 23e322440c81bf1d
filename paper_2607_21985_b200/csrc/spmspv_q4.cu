// spMspV on the 4-bit variant of Tiled-CBC for sm_100a (Sec. 5.1: 4-bit round-to-nearest weights in the
// order static pruning -> quantisation -> dynamic pruning; Sec. 6: Values are stored apart from the
// sparsity metadata, so they can be low-bit).  TileOffset / ColInfo / Bitmap are those of Sec. 4.1
// (offsets count codes, padded to 32 per column tile); Values are 4-bit codes, two per byte, with
// one fp16 scale per column tile: weight = (code - 8) * scale.
//
// With half a byte per stored weight a column tile is at most 128 bytes, so nothing is staged in
// shared memory: a warp takes a GTile, its lanes 0-15 apply the DP test to the 16 activations
// (Sec. 4.2 step (3)) and read ColInfo and the scales of the active columns, and for every active
// column tile lane l owns rows 8l .. 8l+7 (one bitmap byte): rank = set bits before that byte
// (Sec. 4.2.1), its codes are one span of at most 8 nibbles, read as two 32-bit words straight from
// global memory and walked bit by bit in a register.  Same work split and split-K combine as the
// fp16 kernel (equal contiguous GTile ranges, pairwise exchanges along a fixed tree).
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kQWarps = 32;
constexpr int kQThreads = kQWarps * 32;

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

__global__ void __launch_bounds__(kQThreads, 1)
spmspv_q4_kernel(const __grid_constant__ QParams p) {
    __shared__ float red[kQWarps][kTileM];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const unsigned ngt_all = static_cast<unsigned>(p.NGT), nctas = static_cast<unsigned>(p.num_ctas);
    const unsigned g_begin = range_begin(ngt_all, nctas, blockIdx.x), g_end = range_begin(ngt_all, nctas, blockIdx.x + 1);
    const int my_word = lane >> 2, my_shift = 8 * (lane & 3);

    for (unsigned g0 = g_begin; g0 < g_end;) {
        // ---- one segment: this CTA's share of row tile r ----
        const int r = static_cast<int>(g0 / static_cast<unsigned>(p.C));
        const int c0 = static_cast<int>(g0 - static_cast<unsigned>(r) * static_cast<unsigned>(p.C));
        int ngt = p.C - c0;
        if (ngt > static_cast<int>(g_end - g0)) ngt = static_cast<int>(g_end - g0);
        float acc[8];                       // rows 8*lane .. 8*lane+7 of the row tile
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;

        for (int gi = warp; gi < ngt; gi += kQWarps) {
            const int64_t g = static_cast<int64_t>(g0) + gi;
            const int j = (c0 + gi) * kTileK + (lane & 15);
            bool act = false;
            float sx = 0.f;
            unsigned ci = 0;
            if (lane < kTileK && j < p.K) {
                const __half xj = p.x[j];
                if (p.rule == SPDP_DP_NONE) act = true;
                else if (p.rule == SPDP_DP_ABS_GT) act = !(fabsf(__half2float(xj)) <= p.thr);
                else act = (__ldg(p.mask + (j >> 5)) >> (j & 31)) & 1u;
                if (act) {
                    ci = __ldg(p.colinfo + g * kTileK + lane);
                    sx = __half2float(__ldg(p.scales + g * kTileK + lane)) * __half2float(xj);   // exact in fp32
                }
            }
            const unsigned am = __ballot_sync(0xFFFFFFFFu, act) & 0xFFFFu;
            const unsigned to = __ldg(p.tileoffset + g);
            const uint32_t* bm = p.bitmap32 + g * (kTileK * 8) + my_word;       // my word of column 0 of the GTile
            // The active columns are taken 8 at a time in three sweeps, so that the loads of a sweep are
            // all in flight together: (a) my bitmap word of each column, (b) ranks, then my two code words
            // of each column, (c) the walks.
#pragma unroll 1
            for (int h8 = 0; h8 < kTileK; h8 += 8) {
                const unsigned sub = (am >> h8) & 0xFFu;                         // warp-uniform
                if (sub == 0u) continue;
                unsigned wd[8], w0[8], w1[8], meta[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if ((sub >> i) & 1u) wd[i] = __ldg(bm + (h8 + i) * 8);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (!((sub >> i) & 1u)) continue;
                    const unsigned ci_c = __shfl_sync(0xFFFFFFFFu, ci, h8 + i);
                    // set bits before my word: a warp scan in which one lane per word (of the four that hold it) counts
                    const unsigned cnt = __popc(wd[i]);
                    unsigned inc = (lane & 3) == 0 ? cnt : 0u;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        const unsigned u = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                        if (lane >= d) inc += u;
                    }
                    const unsigned bits = (wd[i] >> my_shift) & 0xFFu;           // my 8 rows
                    const unsigned rank = inc - cnt + __popc(wd[i] & ((1u << my_shift) - 1u));
                    const unsigned first = to + (ci_c >> 16);                     // first code of the column tile
                    meta[i] = 0u;
                    if (bits != 0u &&
                        SPDP_CHECK(p.status, first, ((ci_c & 0xFFFFu) + 31u) & ~31u, p.codes_len, kSiteValuesSpan) &&
                        SPDP_CHECK(p.status, rank, 1, ci_c & 0xFFFFu, kSiteRecordIndex)) {
                        // my codes: at most 8 nibbles from nibble `rank` on, inside two consecutive 32-bit words
                        const uint32_t* cw = reinterpret_cast<const uint32_t*>(p.codes) + (first >> 3) + (rank >> 3);
                        w0[i] = __ldg(cw);
                        w1[i] = __ldg(cw + 1);
                        meta[i] = bits | ((rank & 7u) << 8);
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (!((sub >> i) & 1u)) continue;
                    const float sx_c = __shfl_sync(0xFFFFFFFFu, sx, h8 + i);
                    const unsigned bits = meta[i] & 0xFFu;
                    if (bits != 0u) {
                        unsigned span = __funnelshift_r(w0[i], w1[i], 4 * (meta[i] >> 8));
                        // code -> float without a conversion: 0x4B000000 | code is 2^23 + code as a float
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const bool on = (bits >> k) & 1u;
                            const float q = __uint_as_float((span & 15u) | 0x4B000000u) - 8388616.0f;   // code - 8
                            acc[k] = on ? fmaf(q, sx_c, acc[k]) : acc[k];
                            span = on ? span >> 4 : span;
                        }
                    }
                }
            }
        }
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
    spmspv_q4_kernel<<<static_cast<unsigned>(h->num_ctas), kQThreads, 0, s>>>(p);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
