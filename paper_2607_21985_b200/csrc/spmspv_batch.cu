// Small-batch SPDP decode for sm_100a: Y[b] = W_sp * x_b for up to 8 tokens in one pass over the
// Tiled-CBC matrix (the paper names batched DP decode as future work, Sec. 6; the format, the DP
// test and the selective fetch are those of Sec. 4.1-4.2).  Every token keeps its own active set;
// a column tile is fetched once if any token keeps its column, and a token that skips the column
// enters the product with x = 0 for it.
//
// Same skeleton as the single-vector kernel (persistent CTA per contiguous GTile range, active
// list from ColInfo + x, per-warp asynchronous copy ring, split-K combine along a fixed tree), with
// two differences.  The decode does not multiply: a lane rebuilds the fragment of the dense
// 16 x 8 block (16 rows x 8 active column tiles) that the warp-level tensor-core instruction
// mma.m16n8k8 expects in its registers, straight from the compact values, and the instruction
// multiplies it with the 8 x 8 block of activations (8 column tiles x 8 tokens), accumulating in
// fp32.  With N = 8 tokens the contraction is tiny; what it buys is that the expansion work is
// shared by all tokens.  And a batch never spans two row tiles, because a lane already holds
// 256 x 8 / 32 = 64 accumulators.
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kBT = 8;                       // tokens per call (the N of the tensor-core instruction)
constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kDepth = 2;                    // K-blocks a warp keeps in flight
constexpr int kBlockTiles = 8;               // active column tiles per K-block (the K of the instruction)
constexpr int kSlotBytes = 2 * kTileM + 16;   // 16 bytes more than a full column tile: the four tiles whose values the
                                             // lanes of one load read (every second slot) start 8 banks apart
constexpr int kStageBytes = kBlockTiles * kSlotBytes;
constexpr int kChunkCols = 2048;             // columns listed per batch
constexpr int kChunkGT = kChunkCols / kTileK;
constexpr uint32_t kNullRec = 0xFFFFFFFFu;
constexpr int kRecPad = kBlockTiles * (kDepth * kWarps + 1);    // null records behind the last real one
constexpr int kRedPlane = 72;                // floats per (warp, token) plane of the reduction buffer: 64 rows + 8,
                                             // so that the four token pairs of a lane hit different banks
constexpr int kNodeStride = kBT * kTileM;    // workspace words per CTA: [token][row of the row tile]

struct Params {
    const uint32_t* tileoffset;
    const uint32_t* colinfo;
    const uint64_t* bitmap;
    const __half* values;
    const __half* x;            // [batch][ldx]
    int64_t ldx;
    const uint32_t* mask;       // [batch][mask_stride] words, or null
    int64_t mask_stride;
    void* y;                    // [batch][ldy]
    int64_t ldy;
    float thr;
    int rule;
    int ydt;
    int batch;
    int M, K, R, C;
    int64_t NGT;
    int num_ctas;
    float* workspace;           // [num_ctas][kBT][256] tree nodes, all zero between calls
    int* status;
    int64_t values_len;         // elements of Values (the checked build holds every fetch against it)
};

struct __align__(128) Smem {
    union {
        unsigned char ring[kWarps][kDepth][kStageBytes];    // values of the column tiles in flight, per warp
        float red[kWarps][kBT][kRedPlane];                  // cross-warp reduction of 64 rows x 8 tokens
        struct {                                            // list phase
            float keep_clear_of_red[kWarps][kBT][kRedPlane];
            alignas(16) uint32_t colinfo[kChunkCols];
            alignas(16) unsigned short x[kBT][kChunkCols];
            uint32_t tileoff[kChunkGT];
        } stage;
    };
    struct alignas(16) WarpTab {
        uint32_t bm[kDepth][kBlockTiles * 8];               // bitmap words of a K-block: [tile][word]
        uint32_t vo[kDepth][kBlockTiles * 8];               // shared-memory address of each word's first value
    } tab[kWarps];
    alignas(16) uint2 rec[kChunkCols + kRecPad];            // as in the single-vector kernel
    alignas(16) unsigned short xact[kChunkCols + kRecPad][kBT];   // activations of a record's column, 0 where the
                                                                  // token skips it
    uint32_t warp_total[kWarps];
};
static_assert(sizeof(Smem) <= 227 * 1024, "shared memory of one CTA");
static_assert(offsetof(Smem, rec) % 16 == 0 && offsetof(Smem, xact) % 16 == 0 && offsetof(Smem, tab) % 16 == 0, "aligned tables");
static_assert(kChunkCols / 4 <= kThreads, "one list pass, 4 columns per thread");
static_assert(kRecPad <= kThreads, "one thread per trailing null record");
static_assert(sizeof(float) * kWarps * kBT * kRedPlane + 4 * (kChunkCols + kChunkGT) + 2 * kBT * kChunkCols <=
                  size_t(kWarps) * kDepth * kStageBytes, "staging must fit in the ring behind red");

__device__ __forceinline__ unsigned lds_u16(uint32_t addr) {
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
// Rebuilds this lane's part of two fragments from one 32-bit bitmap word of two column tiles (Sec. 4.2.1):
// WA / WB are the word of tile A / B, FA / FB the shared-memory address of the word's first value,
// bit k = my row inside the k-th 8-row slice of the word, below k = the bits before it.  A set bit
// takes the value at rank = set bits before it; a clear bit gives 0.  Output k packs (tile A, tile B)
// for bit k, which is what the tensor-core fragment wants (two adjacent K indices per register).
// (Ranking 2 or 4 adjacent rows with one popcount needs fewer instructions but spreads the 32
// simultaneous loads over more banks; measured 134 and 140 us against 125 us on the largest layer.)
#define SPDP_PICK(V, W, F, BELOW, BIT)                      \
    " and.b32 t, " W ", " BELOW ";\n"                      \
    " popc.b32 t, t;\n"                                    \
    " shl.b32 t, t, 1;\n"                                  \
    " add.u32 t, t, " F ";\n"                              \
    " and.b32 s, " W ", " BIT ";\n"                        \
    " setp.ne.u32 p, s, 0;\n"                              \
    " mov.b16 " V ", 0;\n"                                 \
    " @p ld.shared.u16 " V ", [t];\n"
__device__ __forceinline__ void rebuild_word(unsigned (&a)[4], unsigned WA, unsigned FA, unsigned WB, unsigned FB,
                                             const unsigned (&below)[4], const unsigned (&bit)[4]) {
    asm volatile(
        "{\n"
        " .reg .pred p;\n"
        " .reg .b16 v0, v1, v2, v3, u0, u1, u2, u3;\n"
        " .reg .b32 t, s;\n"
        SPDP_PICK("v0", "%4", "%5", "%8", "%12")
        SPDP_PICK("u0", "%6", "%7", "%8", "%12")
        SPDP_PICK("v1", "%4", "%5", "%9", "%13")
        SPDP_PICK("u1", "%6", "%7", "%9", "%13")
        SPDP_PICK("v2", "%4", "%5", "%10", "%14")
        SPDP_PICK("u2", "%6", "%7", "%10", "%14")
        SPDP_PICK("v3", "%4", "%5", "%11", "%15")
        SPDP_PICK("u3", "%6", "%7", "%11", "%15")
        " mov.b32 %0, {v0, u0};\n"
        " mov.b32 %1, {v1, u1};\n"
        " mov.b32 %2, {v2, u2};\n"
        " mov.b32 %3, {v3, u3};\n"
        "}"
        : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
        : "r"(WA), "r"(FA), "r"(WB), "r"(FB), "r"(below[0]), "r"(below[1]), "r"(below[2]), "r"(below[3]),
          "r"(bit[0]), "r"(bit[1]), "r"(bit[2]), "r"(bit[3]));
}
// The DP test of Sec. 4.2 step (3) on a pair of fp16 activations: 0xFFFF in each half whose column is
// kept, i.e. NOT(|x| <= thr).  thr2 holds, twice, the largest fp16 value that does not exceed thr:
// for an fp16 x that is the same test as the fp32 comparison, and "greater than or unordered" keeps
// NaN activations and makes a NaN threshold keep everything, as the fp32 form does.
__device__ __forceinline__ unsigned abs_gt_keep(unsigned x2, unsigned thr2) {
    unsigned r;
    asm("{\n .reg .b32 a;\n and.b32 a, %1, 0x7FFF7FFF;\n set.gtu.u32.f16x2 %0, a, %2;\n}" : "=r"(r) : "r"(x2), "r"(thr2));
    return r;
}
__device__ __forceinline__ unsigned threshold_pair(float thr) {
    unsigned short h;
    asm("cvt.rm.f16.f32 %0, %1;" : "=h"(h) : "f"(thr));
    return static_cast<unsigned>(h) * 0x00010001u;
}
// D += A (16 rows x 8 column tiles, fp16) * B (8 column tiles x 8 tokens, fp16), fp32 accumulate.
__device__ __forceinline__ void mma_16x8x8(float (&c)[4], unsigned a01, unsigned a23, unsigned b01) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a01), "r"(a23), "r"(b01));
}

__global__ void __launch_bounds__(kThreads, 1)
spmspv_batch_kernel(const Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const unsigned ngt_all = static_cast<unsigned>(p.NGT), nctas = static_cast<unsigned>(p.num_ctas);
    const unsigned g_begin = range_begin(ngt_all, nctas, blockIdx.x), g_end = range_begin(ngt_all, nctas, blockIdx.x + 1);

    // copy / scan role: lane (lgrp, lane7) = (tile of the 4-tile unit, 16-byte piece and bitmap word)
    const int lane7 = lane & 7, lgrp = lane >> 3;
    // decode role: lane (gid, tig) rebuilds rows gid, gid + 8 of every 16-row block for tiles 2*tig, 2*tig + 1
    const int gid = lane >> 2, tig = lane & 3;
    unsigned bitk[4], belowk[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        bitk[k] = pinned(1u << (gid + 8 * k));
        belowk[k] = pinned(bitk[k] - 1u);
    }
    const uint32_t ring_w = smem_u32(&sm.ring[warp][0][0]);
    const uint32_t bm_w = smem_u32(&sm.tab[warp].bm[0][0]);
    constexpr uint32_t kVoFromBm = kDepth * kBlockTiles * 8 * 4;
    constexpr uint32_t kTabStage = kBlockTiles * 8 * 4;
    const uint32_t rec_addr = smem_u32(&sm.rec[0]);
    const uint32_t x_addr = smem_u32(&sm.xact[0][0]);
    const unsigned char* const val_src = reinterpret_cast<const unsigned char*>(p.values) + 16 * lane7;
    const unsigned char* const bm_src = reinterpret_cast<const unsigned char*>(p.bitmap) + 4 * lane7;

    const unsigned thr2 = threshold_pair(p.thr);

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited_for_stream = false;

    float acc[16][4];               // [16-row block][fragment element]: rows 16*rb + gid (+8), tokens 2*tig (+1)
#pragma unroll
    for (int rb = 0; rb < 16; ++rb)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[rb][e] = 0.f;

    for (unsigned g0 = g_begin; g0 < g_end;) {
        // ---- the batch: GTiles [g0, g0 + ngt) of row tile r ----
        const int r = static_cast<int>(g0 / static_cast<unsigned>(p.C));
        const int c0 = static_cast<int>(g0 - static_cast<unsigned>(r) * static_cast<unsigned>(p.C));
        int ngt = p.C - c0;
        if (ngt > static_cast<int>(g_end - g0)) ngt = static_cast<int>(g_end - g0);
        if (ngt > kChunkGT) ngt = kChunkGT;
        const unsigned gA = g0;
        g0 += ngt;
        const bool done = (c0 + ngt == p.C) || (g0 == g_end);       // the CTA's share of row tile r ends here
        const int j0 = c0 * kTileK;
        const int n = min((c0 + ngt) * kTileK, p.K) - j0;           // columns of the batch

        // ---- (1) stage ColInfo / TileOffset and every token's slice of x ----
        {
            const uint32_t ci_stage = smem_u32(&sm.stage.colinfo[0]);
            const uint32_t to_stage = smem_u32(&sm.stage.tileoff[0]);
            const uint4* ci = reinterpret_cast<const uint4*>(p.colinfo + static_cast<size_t>(gA) * kTileK);
            for (int i = t; i < ngt * (kTileK / 4); i += kThreads) cp_async16<0>(ci_stage + 16 * i, ci + i, 1);
            for (int i = t; i < ngt; i += kThreads) cp_async4(to_stage + 4 * i, p.tileoffset + gA + i);
            if (!waited_for_stream) {
                asm volatile("griddepcontrol.wait;" ::: "memory");      // x, y and the workspace from here on
                waited_for_stream = true;
            }
            const bool aligned = ((reinterpret_cast<uintptr_t>(p.x) | static_cast<uintptr_t>(2 * p.ldx)) & 15u) == 0;
            for (int b = 0; b < p.batch; ++b) {
                const __half* xb = p.x + b * p.ldx + j0;
                const uint32_t x_stage = smem_u32(&sm.stage.x[b][0]);
                if (aligned) {
                    for (int i = t; 8 * i < n; i += kThreads)
                        cp_async16_partial(x_stage + 16 * i, xb + 8 * i, 2 * min(8, n - 8 * i));
                } else {
                    for (int v = t; v < n; v += kThreads) sm.stage.x[b][v] = __half_as_ushort(xb[v]);
                }
            }
            cp_async_commit();
        }
        cp_async_wait<0>();
        __syncthreads();

        // ---- (2) active list of the union of the tokens' active sets ----
        // A thread takes 4 consecutive columns: per token the DP test on two fp16 pairs gives a keep
        // mask (0xFFFF per kept half), which zeroes the activations the token skips; the union of the
        // tokens' bits decides which column tiles get a record.
        const int v0 = t * 4;
        unsigned m = 0;
        unsigned xs[kBT][2];                 // my 4 columns' activations per token (fp16 pairs), skipped ones zeroed
        {
            const int lim = n - v0;                                         // positions of mine that hold a column
            const unsigned valid0 = lim >= 2 ? 0xFFFFFFFFu : (lim == 1 ? 0x0000FFFFu : 0u);
            const unsigned valid1 = lim >= 4 ? 0xFFFFFFFFu : (lim == 3 ? 0x0000FFFFu : 0u);
#pragma unroll
            for (int b = 0; b < kBT; ++b) {
                xs[b][0] = xs[b][1] = 0u;
                if (b < p.batch && lim > 0) {
                    const uint2 xv = *reinterpret_cast<const uint2*>(&sm.stage.x[b][v0]);
                    unsigned k0 = 0xFFFFFFFFu, k1 = 0xFFFFFFFFu;
                    if (p.rule == SPDP_DP_ABS_GT) {
                        k0 = abs_gt_keep(xv.x, thr2);
                        k1 = abs_gt_keep(xv.y, thr2);
                    } else if (p.rule == SPDP_DP_MASK) {
                        const int j = j0 + v0;                              // a multiple of 4
                        const unsigned bits = __ldg(p.mask + b * p.mask_stride + (j >> 5)) >> (j & 31);
                        k0 = ((bits & 1u) ? 0x0000FFFFu : 0u) | ((bits & 2u) ? 0xFFFF0000u : 0u);
                        k1 = ((bits & 4u) ? 0x0000FFFFu : 0u) | ((bits & 8u) ? 0xFFFF0000u : 0u);
                    }
                    k0 &= valid0;
                    k1 &= valid1;
                    xs[b][0] = xv.x & k0;
                    xs[b][1] = xv.y & k1;
                    m |= (k0 & 1u) | ((k0 >> 30) & 2u) | ((k1 & 1u) << 2) | ((k1 >> 28) & 8u);
                }
            }
        }
        const unsigned cnt = __popc(m);
        unsigned inc = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned u = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += u;
        }
        if (lane == 31) sm.warp_total[warp] = inc;
        __syncthreads();
        int nact;
        {
            const unsigned tl = (lane < kWarps) ? sm.warp_total[lane] : 0u;
            const unsigned base = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? tl : 0u);
            nact = static_cast<int>(__reduce_add_sync(0xFFFFFFFFu, tl));
            if (m != 0u) {
                const unsigned slot0 = gA * kTileK + v0;                    // column slot of position v0
                int item = static_cast<int>(base + inc - cnt);
                const unsigned to = sm.stage.tileoff[v0 >> 4];
                const uint4 cv = *reinterpret_cast<const uint4*>(&sm.stage.colinfo[v0]);
                const unsigned ci[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if ((m >> k) & 1u) {
                        const unsigned start = to + (ci[k] >> 16), pieces = ((ci[k] & 0xFFFFu) + 7u) >> 3;
                        const bool rec_ok = SPDP_CHECK(p.status, item, 1, kChunkCols, kSiteRecordIndex) &&
                                            SPDP_CHECK(p.status, start, 8u * pieces, p.values_len, kSiteValuesSpan) &&
                                            SPDP_CHECK(p.status, 0, pieces, 32, kSitePieces) &&
                                            SPDP_CHECK(p.status, slot0 + k, 1, p.NGT * kTileK, kSiteBitmapSlot);
                        if (!SPDP_CHECK(p.status, item, 1, kChunkCols, kSiteRecordIndex)) {
                            ++item;
                            continue;
                        }
                        sm.rec[item] = rec_ok ? make_uint2(start, ((slot0 + k) << 6) | pieces) : make_uint2(0u, kNullRec);
                        uint4 xr;
                        unsigned* xo = reinterpret_cast<unsigned*>(&xr);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {                       // tokens 2q, 2q + 1
                            const unsigned lo = (k & 1) ? (xs[2 * q][k >> 1] >> 16) : (xs[2 * q][k >> 1] & 0xFFFFu);
                            const unsigned hi = (k & 1) ? (xs[2 * q + 1][k >> 1] >> 16) : (xs[2 * q + 1][k >> 1] & 0xFFFFu);
                            xo[q] = lo | (hi << 16);
                        }
                        *reinterpret_cast<uint4*>(&sm.xact[item][0]) = xr;
                        ++item;
                    }
                }
            }
            if (t < kRecPad) {                                              // null records with zero activations
                sm.rec[nact + t] = make_uint2(0u, kNullRec);
                *reinterpret_cast<uint4*>(&sm.xact[nact + t][0]) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        __syncthreads();       // the records are complete; the staging area becomes the ring again
        const int nblocks = (nact + kBlockTiles - 1) / kBlockTiles;

        // ---- (3) per-warp copy / rebuild / multiply pipeline over K-blocks warp, warp + kWarps, ... ----
        auto fetch_block = [&](int kb, int stage) {
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const int tile = 4 * s + lgrp;
                const uint2 rc = lds_v2(rec_addr + 8u * (kb * kBlockTiles + tile));
                const uint32_t bdst = bm_w + stage * kTabStage + 4u * (tile * 8 + lane7);
                if (rc.y != kNullRec) {
                    const int rem = static_cast<int>(rc.y & 63u) - lane7;
                    const unsigned char* src = offset_wide<2>(val_src, rc.x);
                    const uint32_t dst = ring_w + stage * kStageBytes + tile * kSlotBytes + 16 * lane7;
                    cp_async16<0>(dst, src, rem);
                    cp_async16<128>(dst, src, rem);
                    cp_async16<256>(dst, src, rem);
                    cp_async16<384>(dst, src, rem);
                    cp_async4(bdst, offset_wide<32>(bm_src, rc.y >> 6));
                } else {
                    sts_u32(bdst, 0u);
                }
            }
            cp_async_commit();
        };
#pragma unroll
        for (int dd = 0; dd < kDepth; ++dd) fetch_block(warp + dd * kWarps, dd);     // null records past the end

        int stage = 0;
        for (int kb = warp; kb < nblocks; kb += kWarps) {
            cp_async_wait<kDepth - 1>();
            __syncwarp();
            const uint32_t tabs = bm_w + stage * kTabStage;
#pragma unroll
            for (int s = 0; s < 2; ++s) {       // scan role: address of my word's first value inside the warp's ring
                const int tile = 4 * s + lgrp;
                const uint32_t own = tabs + 4u * (tile * 8 + lane7);
                const unsigned c = __popc(lds_u32(own));
                unsigned ic = c;
                scan8_level<1>(ic);
                scan8_level<2>(ic);
                scan8_level<4>(ic);
                sts_u32<kVoFromBm>(own, ring_w + stage * kStageBytes + tile * kSlotBytes + 2u * (ic - c));
            }
            __syncwarp();
            // decode role: tiles tA = 2*tig and tB = tA + 1 of the K-block; the tokens' activations for them
            const uint32_t tA = tabs + 4u * (2 * tig * 8);
            const uint32_t xa = x_addr + 2u * ((kb * kBlockTiles + 2 * tig) * kBT + gid);
            const unsigned b01 = lds_u16(xa) | (lds_u16(xa + 2 * kBT) << 16);       // token gid: (tile tA, tile tB)
#pragma unroll
            for (int h = 0; h < 2; ++h) {                                            // words 4h .. 4h + 3
                const uint4 wA = lds_v4<0>(tA + 16 * h), fA = lds_v4<kVoFromBm>(tA + 16 * h);
                const uint4 wB = lds_v4<32>(tA + 16 * h), fB = lds_v4<kVoFromBm + 32>(tA + 16 * h);
                const unsigned WA[4] = {wA.x, wA.y, wA.z, wA.w}, FA[4] = {fA.x, fA.y, fA.z, fA.w};
                const unsigned WB[4] = {wB.x, wB.y, wB.z, wB.w}, FB[4] = {fB.x, fB.y, fB.z, fB.w};
                unsigned a[4][4];                                                    // [word][bit gid + 8k]: (tile tA, tile tB)
#pragma unroll
                for (int w = 0; w < 4; ++w) rebuild_word(a[w], WA[w], FA[w], WB[w], FB[w], belowk, bitk);
#pragma unroll
                for (int w = 0; w < 4; ++w) {                                        // rows 32 * (4h + w) ..
                    mma_16x8x8(acc[2 * (4 * h + w)], a[w][0], a[w][1], b01);
                    mma_16x8x8(acc[2 * (4 * h + w) + 1], a[w][2], a[w][3], b01);
                }
            }
            __syncwarp();                  // everyone is done with this ring position
            fetch_block(kb + kDepth * kWarps, stage);
            stage ^= 1;
        }
        cp_async_wait<0>();
        __syncthreads();       // all pipelines drained: the ring is idle

        // ---- (4) the CTA's share of row tile r is complete: reduce across warps, combine, store ----
        if (done) {
            const int q0 = range_owner(ngt_all, nctas, static_cast<unsigned>(r) * p.C);
            const int nseg = range_owner(ngt_all, nctas, static_cast<unsigned>(r + 1) * p.C - 1u) - q0 + 1;
            const int tok = t >> 6, rr = t & 63;                // my output in every 64-row chunk
            float part[4];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {                    // 64 rows at a time through the idle ring
#pragma unroll
                for (int rbl = 0; rbl < 4; ++rbl) {
                    float (&c)[4] = acc[4 * ch + rbl];
                    sm.red[warp][2 * tig][16 * rbl + gid] = c[0];
                    sm.red[warp][2 * tig + 1][16 * rbl + gid] = c[1];
                    sm.red[warp][2 * tig][16 * rbl + gid + 8] = c[2];
                    sm.red[warp][2 * tig + 1][16 * rbl + gid + 8] = c[3];
                    c[0] = c[1] = c[2] = c[3] = 0.f;
                }
                __syncthreads();
                float sum = 0.f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) sum += sm.red[w][tok][rr];
                part[ch] = sum;
                __syncthreads();
            }
            // The four outputs walk the same tree (same segments); their exchanges at a level are
            // issued together, so the walk costs one round trip per level, not four.
            if (tok < p.batch && SPDP_CHECK(p.status, q0, nseg, p.num_ctas, kSiteTreeNodes) &&
                SPDP_CHECK(p.status, static_cast<int>(blockIdx.x) - q0, 1, nseg, kSiteTreeNodes)) {
                unsigned* nodes = reinterpret_cast<unsigned*>(p.workspace) + tok * kTileM + rr;
                const int64_t row0 = static_cast<int64_t>(r) * kTileM + rr;
                bool alive[4];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) alive[ch] = row0 + 64 * ch < p.M;
                int idx = static_cast<int>(blockIdx.x) - q0;
                for (int nn = nseg, level = 0; nn > 1; nn = (nn + 1) >> 1, ++level, idx >>= 1) {
                    const int right = idx | 1;
                    if (right >= nn) continue;                  // no neighbour at this level
                    unsigned* node = nodes + static_cast<int64_t>(q0 + (right << level)) * kNodeStride;
                    unsigned old[4];
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
                        if (alive[ch]) old[ch] = atomicExch(node + 64 * ch, canonical_bits(part[ch]) ^ kNodeKey);
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        if (!alive[ch]) continue;
                        if (old[ch] == 0u) {
                            alive[ch] = false;                  // first at the node: the neighbour carries the sum on
                        } else {
                            node[64 * ch] = 0u;                 // second: empty the node for the next call
                            part[ch] += __uint_as_float(old[ch] ^ kNodeKey);
                        }
                    }
                }
#pragma unroll
                for (int ch = 0; ch < 4; ++ch)
                    if (alive[ch]) store_y(p.y, p.ydt, tok * p.ldy + row0 + 64 * ch, part[ch]);
            }
        }
    }
}

}  // namespace

int64_t batch_workspace_bytes(int num_ctas) { return static_cast<int64_t>(num_ctas) * kNodeStride * sizeof(float); }

spdp_status configure_spmspv_batch_kernel() {
    static std::mutex mu;
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SPDP_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(spmspv_batch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(sizeof(Smem))));
        configured[dev] = true;
    }
    return SPDP_OK;
}

spdp_status launch_spmspv_batch(const spdp_matrix* h, const __half* x, int64_t ldx, int batch, int rule, float thr,
                                const uint32_t* mask, int64_t mask_stride, void* y, int64_t ldy, int ydt,
                                cudaStream_t s) {
    spdp_status st = configure_spmspv_batch_kernel();
    if (st != SPDP_OK) return st;
    Params p;
    p.tileoffset = h->tileoffset;
    p.colinfo = h->colinfo;
    p.bitmap = h->bitmap;
    p.values = h->values;
    p.x = x;
    p.ldx = ldx;
    p.mask = mask;
    p.mask_stride = mask_stride;
    p.y = y;
    p.ldy = ldy;
    p.thr = thr;
    p.rule = rule;
    p.ydt = ydt;
    p.batch = batch;
    p.M = static_cast<int>(h->M);
    p.K = static_cast<int>(h->K);
    p.R = static_cast<int>(h->R);
    p.C = static_cast<int>(h->C);
    p.NGT = h->NGT;
    p.num_ctas = h->num_ctas;
    p.workspace = h->workspace_batch;
    p.status = h->status_word;
    p.values_len = h->values_len;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(h->num_ctas));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = sizeof(Smem);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    SPDP_CUDA_TRY(cudaLaunchKernelEx(&cfg, spmspv_batch_kernel, p));
    return SPDP_OK;
}

}  // namespace spdp
