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
            unsigned am = __ballot_sync(0xFFFFFFFFu, act) & 0xFFFFu;
            const unsigned to = __ldg(p.tileoffset + g);
            while (am != 0u) {
                const int cc = __ffs(am) - 1;
                am &= am - 1u;
                const unsigned ci_c = __shfl_sync(0xFFFFFFFFu, ci, cc);
                const float sx_c = __shfl_sync(0xFFFFFFFFu, sx, cc);
                const unsigned n = ci_c & 0xFFFFu;
                if (n == 0u) continue;
                const int64_t slot = g * kTileK + cc;
                // the 8 bitmap words of the column tile (each lane one, four times over), set bits before each
                const unsigned wd = __ldg(p.bitmap32 + slot * 8 + (lane & 7));
                const unsigned cnt = __popc(wd);
                unsigned inc = cnt;
                scan8_level<1>(inc);
                scan8_level<2>(inc);
                scan8_level<4>(inc);
                const unsigned w_mine = __shfl_sync(0xFFFFFFFFu, wd, my_word);
                const unsigned before = __shfl_sync(0xFFFFFFFFu, inc - cnt, my_word);
                const unsigned bits = (w_mine >> my_shift) & 0xFFu;                 // my 8 rows
                if (bits != 0u) {
                    const unsigned rank = before + __popc(w_mine & ((1u << my_shift) - 1u));
                    const unsigned first = to + (ci_c >> 16);                        // first code of the column tile
                    if (SPDP_CHECK(p.status, first, (n + 31u) & ~31u, p.codes_len, kSiteValuesSpan) &&
                        SPDP_CHECK(p.status, rank, 1, n, kSiteRecordIndex)) {
                        // my codes: at most 8 nibbles from nibble `rank` on, inside two consecutive 32-bit words
                        const uint32_t* cw = reinterpret_cast<const uint32_t*>(p.codes + (first >> 1)) + (rank >> 3);
                        unsigned span = __funnelshift_r(__ldg(cw), __ldg(cw + 1), 4 * (rank & 7u));
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            if ((bits >> k) & 1u) {
                                acc[k] = fmaf(static_cast<float>(static_cast<int>(span & 15u) - 8), sx_c, acc[k]);
                                span >>= 4;
                            }
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
