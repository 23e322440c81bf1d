// SPDP spMspV for sm_100a (Sec. 4.2, Alg. 1): y = W_sp * x over the columns that pass the
// dynamic-pruning test, W_sp in Tiled-CBC.
//
// Work split (Sec. 4.2.3 "tile-based scheme combined with Split-K"): the NGT GTiles, in their
// row-major storage order, are cut into num_ctas equal contiguous ranges, one per CTA.  A range
// touches one or more row tiles; each (CTA, row tile) piece is a "segment" that yields 256
// fp32 partial sums.  A row tile fed by one segment is written to y directly; otherwise the
// segments' partials are added pairwise along a fixed binary tree through the handle's
// workspace (the paper's ReductionWorkspace): whoever reaches a tree node first leaves its sum
// there with one atomic exchange, the second takes it, adds, and moves up; the thread that
// completes the root stores y.  No CTA ever waits for another, and the shape of the tree, hence
// the rounding of the result, does not depend on who arrives when.
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

#ifndef SPDP_FMA_MODE
#define SPDP_FMA_MODE 0      // 0: mixed-precision fma.rn.f32.f16, 1: cvt + fp32 fma
#endif
#ifndef SPDP_WARPS
#define SPDP_WARPS 24
#endif
#ifndef SPDP_CTAS_PER_SM
#define SPDP_CTAS_PER_SM 1
#endif
#ifndef SPDP_CHUNK_COLS
#define SPDP_CHUNK_COLS 8192
#endif
#ifndef SPDP_DEPTH
#define SPDP_DEPTH 2
#endif
constexpr int kWarps = SPDP_WARPS;         // warps per CTA; every warp fetches and decodes its own column tiles
constexpr int kDepth = SPDP_DEPTH;         // groups a warp keeps in flight
constexpr int kGroup = 4;                  // active column tiles per group (one fetch / decode unit of a warp)
constexpr int kSlotBytes = 2 * kTileM + 32;  // a column tile's values (at most 256 fp16) + 32 bytes so that the
                                             // four tiles of a group start 8 banks apart
constexpr int kStageBytes = kGroup * kSlotBytes;
constexpr int kThreads = kWarps * 32;
constexpr int kChunkCols = SPDP_CHUNK_COLS; // columns handled between two pipeline drains
constexpr int kCtasPerSm = SPDP_CTAS_PER_SM;
constexpr uint32_t kNullRec = 0xFFFFFFFFu;
constexpr int kListPasses = (kChunkCols / 8 + kThreads - 1) / kThreads;     // 8-position units a thread lists per batch
constexpr int kChunkGT = kChunkCols / kTileK;
constexpr int kRecPad = kGroup * (kDepth * kWarps + 1);   // null records behind the last real one

struct Params {
    const uint32_t* tileoffset;
    const uint32_t* colinfo;
    const uint64_t* bitmap;
    const __half* values;
    const __half* x;
    const uint32_t* mask;
    void* y;
    float thr;
    int rule;
    int ydt;
    int M, K, R, C;
    int64_t NGT;            // R * C GTiles, cut into num_ctas equal contiguous ranges
    int num_ctas;
    float* workspace;       // [num_ctas][256] tree nodes of the split-K combine, all zero between calls
    int* status;
    int64_t values_len;     // elements of Values (the checked build holds every fetch against it)
};

struct __align__(128) Smem {
    union {
        unsigned char ring[kWarps][kDepth][kStageBytes];    // values of the column tiles in flight, per warp
        float red[kWarps][kTileM];                          // cross-warp row reduction (after the pipelines drained)
        struct {                                            // list phase: the chunk's ColInfo / TileOffset words,
            float keep_clear_of_red[kWarps][kTileM];        // placed behind red[], which may still be read
            alignas(16) uint32_t colinfo[kChunkCols];
            alignas(16) unsigned short x[kChunkCols];       // and the activations of the listed columns
            uint32_t tileoff[kChunkGT];
        } stage;
    };
    // Bitmap words of a group in decode order: word w of the group's it-th tile sits at
    // [(w & 1) * 16 + it * 4 + (w >> 1)], so the lanes that decode the even (odd) words read 16 consecutive words.
    struct alignas(16) WarpTab {
        uint32_t bm[kDepth][32];
        uint32_t vo[kDepth][32];                        // same order: shared-memory address of each word's first value
    } tab[kWarps];
    // Active list of the chunk, one record per active column tile (filled once per chunk):
    alignas(16) uint2 rec[kChunkCols + kRecPad];        // .x = start of its values in Values (elements),
                                                        // .y = (column slot in Bitmap/ColInfo) << 6 | 16-byte pieces
                                                        //      of values; kNullRec pads a piece to whole groups and
                                                        //      follows the last record for kRecPad entries, so a warp
                                                        //      can fetch kDepth groups ahead without a range test
    alignas(16) unsigned short xact[kChunkCols + kGroup];   // its activation x_j (fp16 bits)
    float red_first[kWarps][kTileM];                    // row reduction of a batch's first piece (flushed mid-stream)
    uint32_t warp_total[kListPasses][kWarps][2];        // list phase: records listed by each warp per pass (all, piece A)
};
static_assert(offsetof(Smem, rec) % 16 == 0 && offsetof(Smem, xact) % 16 == 0 && offsetof(Smem, tab) % 16 == 0, "16-byte shared loads need aligned tables");
static_assert(sizeof(float) * kWarps * kTileM <= size_t(kWarps) * kDepth * kStageBytes, "red must fit in the ring");
static_assert(sizeof(uint32_t) * (kChunkCols + kChunkGT) + 2 * kChunkCols + sizeof(float) * kWarps * kTileM <=
                  size_t(kWarps) * kDepth * kStageBytes,
              "staging must fit in the ring behind red");
static_assert(sizeof(Smem) <= (227 * 1024) / kCtasPerSm - 1024 * (kCtasPerSm - 1), "shared memory of one CTA");
static_assert(kRecPad <= kThreads, "one thread per trailing null record");
static_assert(kWarps >= 16, "two groups of 256 threads finish two row tiles side by side");

// DP test of Sec. 4.2 step (3): magnitude against the threshold; NOT(|x| <= thr) keeps NaN.
__device__ __forceinline__ bool column_active(int rule, float thr, const uint32_t* mask, int j, __half xj) {
    if (rule == SPDP_DP_NONE) return true;
    if (rule == SPDP_DP_ABS_GT) return !(fabsf(__half2float(xj)) <= thr);
    return (mask[j >> 5] >> (j & 31)) & 1u;
}

// One decode step (Sec. 4.2.1): the 2 consecutive rows this lane owns inside the 32-bit bitmap
// word W.  `first` is the shared-memory address of the word's first value, `below` masks the bits
// of lower rows, m0 and m1 are the lane's two bits.  rank = set bits before the position; a set
// bit takes the next value and adds value * x to its row's fp32 accumulator.  fma.rn.f32.f16
// multiplies two fp16 exactly and accumulates in fp32.  x32 holds two activations; kUpper picks one.
#if SPDP_FMA_MODE == 0
#define SPDP_FMA2(X)                                  \
    " @p0 fma.rn.f32.f16 %0, v0, " X ", %0;\n"        \
    " @p1 fma.rn.f32.f16 %1, v1, " X ", %1;\n"
#else
#define SPDP_FMA2(X)                                  \
    " .reg .f32 f0, f1, fx;\n"                        \
    " cvt.f32.f16 fx, " X ";\n"                       \
    " @p0 cvt.f32.f16 f0, v0;\n @p1 cvt.f32.f16 f1, v1;\n" \
    " @p0 fma.rn.f32 %0, f0, fx, %0;\n"               \
    " @p1 fma.rn.f32 %1, f1, fx, %1;\n"
#endif
#define SPDP_DECODE_BODY(X)                           \
    "{\n"                                             \
    " .reg .pred p0, p1;\n"                           \
    " .reg .b16 v0, v1, xl, xu;\n"                    \
    " .reg .b32 t, a;\n"                              \
    " and.b32 t, %2, %4;\n"                           \
    " popc.b32 t, t;\n"                               \
    " shl.b32 t, t, 1;\n"                             \
    " add.u32 a, %3, t;\n"                            \
    " lop3.or.b32 t|p0, %2, %5, 0, 0xC0, 0;\n"        \
    " lop3.or.b32 t|p1, %2, %6, 0, 0xC0, 0;\n"        \
    " mov.b32 {xl, xu}, %7;\n"                        \
    " @p0 ld.shared.u16 v0, [a];\n @p0 add.u32 a, a, 2;\n" \
    " @p1 ld.shared.u16 v1, [a];\n"                   \
    SPDP_FMA2(X)                                      \
    "}"
template <bool kUpper>
__device__ __forceinline__ void decode_step(unsigned W, uint32_t first, unsigned below, unsigned m0, unsigned m1,
                                            unsigned x32, float& a0, float& a1) {
    if (kUpper)
        asm volatile(SPDP_DECODE_BODY("xu")
                     : "+f"(a0), "+f"(a1) : "r"(W), "r"(first), "r"(below), "r"(m0), "r"(m1), "r"(x32));
    else
        asm volatile(SPDP_DECODE_BODY("xl")
                     : "+f"(a0), "+f"(a1) : "r"(W), "r"(first), "r"(below), "r"(m0), "r"(m1), "r"(x32));
}
__device__ __forceinline__ unsigned range_begin(const Params& p, unsigned c) {
    return dev::range_begin(static_cast<unsigned>(p.NGT), static_cast<unsigned>(p.num_ctas), c);
}
__device__ __forceinline__ int range_owner(const Params& p, unsigned g) {
    return dev::range_owner(static_cast<unsigned>(p.NGT), static_cast<unsigned>(p.num_ctas), g);
}

// Adds the kWarps per-warp partial sums of one row tile in warp order and finishes the row (tt =
// row inside the tile; the rows are independent, nothing here synchronises threads).  A row tile
// fed by one segment is stored directly; otherwise the segments' sums meet along the fixed tree of
// tree_combine and the thread that completes the root stores y.
__device__ __forceinline__ void finish_row_tile(const Params& p, int r, const float (*red)[kTileM], int tt) {
    float part = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) part += red[w][tt];
    const int64_t row = static_cast<int64_t>(r) * kTileM + tt;
    if (row >= p.M) return;
    const int q0 = range_owner(p, static_cast<unsigned>(r) * p.C);                 // first and last CTA feeding row tile r
    const int nseg = range_owner(p, static_cast<unsigned>(r + 1) * p.C - 1u) - q0 + 1;
    if (!SPDP_CHECK(p.status, q0, nseg, p.num_ctas, kSiteTreeNodes) ||
        !SPDP_CHECK(p.status, static_cast<int>(blockIdx.x) - q0, 1, nseg, kSiteTreeNodes) ||
        !SPDP_CHECK(p.status, row, 1, p.M, kSiteOutputRow))
        return;
    if (tree_combine(part, reinterpret_cast<unsigned*>(p.workspace) + tt, kTileM, q0, nseg,
                     static_cast<int>(blockIdx.x) - q0))
        store_y(p.y, p.ydt, row, part);
}

// One persistent CTA per GTile range; every warp runs its own fetch -> decode pipeline.
// The range is cut into pieces (part of one row tile, at most kChunkGT GTiles).  A batch is one
// piece, or the last piece of a row tile together with the first piece of the next row tile, so
// that the usual CTA range (the tail of one row tile and the head of the next) is one batch.
// Per batch:
//   (1) all warps: the pieces' ColInfo / TileOffset words and the active-column list from x
//       (a thread tests 8 columns, warp scans + prefix sums place them), one record per active
//       column tile -- Sec. 4.2 steps (1)-(3);
//   (2) each warp takes groups of kGroup active column tiles round-robin.  It keeps kDepth
//       groups in flight: the padded values of a column tile arrive with 16-byte asynchronous
//       copies (lane = one 16-byte piece of one of the group's tiles), its 8 bitmap words with
//       4-byte ones; inactive columns are never touched.  Decode (Sec. 4.2.1): lane owns 2
//       consecutive rows of every second bitmap word, rank = set bits before them, values read from
//       shared memory, fp32 accumulation in registers.  Where the first piece's groups end the
//       warp parks its sums in shared memory and starts the second piece from zero;
//   (3) batch end: cross-warp row reduction, split-K combine and store of every row tile that
//       the batch completed (two groups of 256 threads work side by side).
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
spmspv_kernel(const Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const unsigned g_begin = range_begin(p, blockIdx.x), g_end = range_begin(p, blockIdx.x + 1);

    const int lane7 = lane & 7;
    const int lgrp = lane >> 3;
    // fetch role: lane (lgrp, lane7) moves 16-byte pieces lane7, lane7+8, ... and bitmap word lane7 of the
    // group's lgrp-th tile.  scan role: the same (tile, word).  decode role: lanes 0-15 take the even
    // words of every tile, lanes 16-31 the odd ones; a lane owns rows 2*l15, 2*l15+1 of its words, so
    // the 32 simultaneous value loads of a step fall inside 64 rows = at most 128 contiguous bytes
    // (one shared-memory wavefront, whatever the density).
    const int l15 = lane & 15, lhalf = lane >> 4;
    const unsigned bit0 = pinned(1u << (2 * l15));      // my first row inside a 32-bit bitmap word
    const unsigned bit1 = pinned(bit0 << 1);
    const unsigned lt_mask = pinned(bit0 - 1u);
    const int tpos = (lane7 & 1) * 16 + lgrp * 4 + (lane7 >> 1);        // where (tile lgrp, word lane7) sits
    const uint32_t val_dst = pinned(smem_u32(&sm.ring[warp][0][lgrp * kSlotBytes + 16 * lane7]));
    const uint32_t bm_own = pinned(smem_u32(&sm.tab[warp].bm[0][tpos]));
    const uint32_t bm_dec = pinned(smem_u32(&sm.tab[warp].bm[0][lhalf * 16]));
    constexpr int kVoFromBm = kDepth * 128;             // vo[d][i] sits this many bytes behind bm[d][i]
    const uint32_t ring_slot = pinned(smem_u32(&sm.ring[warp][0][lgrp * kSlotBytes]));  // scan role: my tile's slot in stage 0
    // fetch role: my 16-byte piece of a column tile's values / my bitmap word, before the tile's offset is added
    const unsigned char* const val_src = pinned(reinterpret_cast<const unsigned char*>(p.values) + 16 * lane7);
    const unsigned char* const bm_src = pinned(reinterpret_cast<const unsigned char*>(p.bitmap) + 4 * lane7);
    const uint32_t rec_addr = smem_u32(&sm.rec[0]);
    const uint32_t x_addr = smem_u32(&sm.xact[0]);

    // Let a dependent launch (the next call) begin as soon as SMs free up.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited_for_stream = false;  // x, y, workspace and counters may belong to the previous kernel until we wait

    float acc[8];                   // acc[2s + k] = row 64*s + 2*lane + k of the current row tile
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;

    for (unsigned g0 = g_begin; g0 < g_end;) {
        // ---- the batch: piece A = [gA, gA + ngtA) of row tile rA, optionally piece B of row tile rA + 1 ----
        const int rA = static_cast<int>(g0 / static_cast<unsigned>(p.C));
        const int cA = static_cast<int>(g0 - static_cast<unsigned>(rA) * static_cast<unsigned>(p.C));
        int ngtA = p.C - cA;
        if (ngtA > static_cast<int>(g_end - g0)) ngtA = static_cast<int>(g_end - g0);
        if (ngtA > kChunkGT) ngtA = kChunkGT;
        const unsigned gA = g0;
        g0 += ngtA;
        const bool doneA = (cA + ngtA == p.C) || (g0 == g_end);     // piece A ends its row tile's share of this CTA
        const int jA0 = cA * kTileK;
        const int nA = min((cA + ngtA) * kTileK, p.K) - jA0;         // columns of piece A
        const int vB0 = (ngtA * kTileK + 31) & ~31;                  // piece B starts at this list position
        int ngtB = 0, nB = 0;
        bool doneB = false;
        if (doneA && g0 < g_end && cA + ngtA == p.C) {
            ngtB = p.C;
            if (ngtB > static_cast<int>(g_end - g0)) ngtB = static_cast<int>(g_end - g0);
            if (ngtB > (kChunkCols - vB0) / kTileK) ngtB = (kChunkCols - vB0) / kTileK;
            nB = min(ngtB * kTileK, p.K);
            doneB = (ngtB == p.C) || (g0 + ngtB == g_end);
        }
        const unsigned gB = g0;
        g0 += ngtB;
        const int rB = rA + 1;
        const int nlist = (ngtB > 0) ? vB0 + nB : nA;               // list positions (A, padding, B)

        // ---- (1) active-column list of the batch (ballots + prefix sums) and its records ----
        // One memory round trip: the pieces' ColInfo and TileOffset words and their slice of x stream
        // into the idle ring with asynchronous copies.  ColInfo of skipped columns is read too
        // (4 bytes per column tile); their bitmaps and values never are.
        {
            const uint32_t ci_stage = smem_u32(&sm.stage.colinfo[0]);
            const uint32_t to_stage = smem_u32(&sm.stage.tileoff[0]);
            const uint32_t x_stage = smem_u32(&sm.stage.x[0]);
            const uint4* ciA = reinterpret_cast<const uint4*>(p.colinfo + static_cast<size_t>(gA) * kTileK);
            const uint4* ciB = reinterpret_cast<const uint4*>(p.colinfo + static_cast<size_t>(gB) * kTileK);
            for (int i = t; i < ngtA * (kTileK / 4); i += kThreads) cp_async16<0>(ci_stage + 16 * i, ciA + i, 1);
            for (int i = t; i < ngtB * (kTileK / 4); i += kThreads) cp_async16<0>(ci_stage + 4 * vB0 + 16 * i, ciB + i, 1);
            for (int i = t; i < ngtA; i += kThreads) cp_async4(to_stage + 4 * i, p.tileoffset + gA + i);
            for (int i = t; i < ngtB; i += kThreads) cp_async4(to_stage + (vB0 >> 2) + 4 * i, p.tileoffset + gB + i);
            if (!waited_for_stream) {
                // everything above reads only the packed matrix; from here on the previous kernel's results count
                asm volatile("griddepcontrol.wait;" ::: "memory");
                waited_for_stream = true;
            }
            if ((reinterpret_cast<uintptr_t>(p.x) & 15u) == 0) {
                // list position v holds x[jA0 + v] (piece A) or x[v - vB0] (piece B); 8 activations per copy
                for (int i = t; 8 * i < nA; i += kThreads)
                    cp_async16_partial(x_stage + 16 * i, p.x + jA0 + 8 * i, 2 * min(8, nA - 8 * i));
                for (int i = t; 8 * i < nB; i += kThreads)
                    cp_async16_partial(x_stage + 2 * vB0 + 16 * i, p.x + 8 * i, 2 * min(8, nB - 8 * i));
            } else {
                for (int v = t; v < nA; v += kThreads) sm.stage.x[v] = __half_as_ushort(p.x[jA0 + v]);
                for (int v = t; v < nB; v += kThreads) sm.stage.x[vB0 + v] = __half_as_ushort(p.x[v]);
            }
            cp_async_commit();
        }
        cp_async_wait<0>();
        __syncthreads();
        // A thread lists 8 consecutive positions per pass (unit (pass * kThreads + t)): the DP test on its
        // 8 activations gives an 8-bit mask, a warp scan of the counts its place among the warp's
        // records; the warps' totals meet in shared memory, every thread derives its first record index
        // from them, and the records are written in list order.  Piece B starts on a whole group of
        // kGroup records: the padding is inserted in front of its first record.
        unsigned m8[kListPasses], below[kListPasses];
#pragma unroll
        for (int k = 0; k < kListPasses; ++k) {
            const int v0 = (k * kThreads + t) * 8;                       // first list position of my unit
            unsigned m = 0;
            if (v0 < nlist) {
                const int lim = ((v0 < vB0) ? nA : nlist) - v0;          // positions of the unit that hold a column
                if (p.rule == SPDP_DP_ABS_GT) {
                    const uint4 xv = *reinterpret_cast<const uint4*>(&sm.stage.x[v0]);
                    const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float lo = __half2float(__ushort_as_half(static_cast<unsigned short>(xw[i] & 0xFFFFu)));
                        const float hi = __half2float(__ushort_as_half(static_cast<unsigned short>(xw[i] >> 16)));
                        m |= (!(fabsf(lo) <= p.thr) ? 1u : 0u) << (2 * i);
                        m |= (!(fabsf(hi) <= p.thr) ? 1u : 0u) << (2 * i + 1);
                    }
                } else if (p.rule == SPDP_DP_MASK) {
                    // units of the padding between the two pieces hold no column: they must not touch
                    // the mask (their word can lie one past its end)
                    if (lim > 0) {
                        const int j0 = (v0 < vB0) ? jA0 + v0 : v0 - vB0; // a multiple of 8
                        m = (__ldg(p.mask + (j0 >> 5)) >> (j0 & 31)) & 0xFFu;
                    }
                } else {
                    m = 0xFFu;
                }
                m &= (lim >= 8) ? 0xFFu : (lim > 0 ? (1u << lim) - 1u : 0u);
            }
            m8[k] = m;
            const unsigned c = __popc(m);
            unsigned inc = c;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned u = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc += u;
            }
            below[k] = inc - c;
            const unsigned totA = __reduce_add_sync(0xFFFFFFFFu, (v0 < vB0) ? c : 0u);
            if (lane == 31) {
                sm.warp_total[k][warp][0] = inc;
                sm.warp_total[k][warp][1] = totA;
            }
        }
        __syncthreads();
        int nact, nactA_pad;
        {
            unsigned base[kListPasses], total = 0, realA = 0;
#pragma unroll
            for (int k = 0; k < kListPasses; ++k) {
                const unsigned tl = (lane < kWarps) ? sm.warp_total[k][lane][0] : 0u;
                const unsigned tla = (lane < kWarps) ? sm.warp_total[k][lane][1] : 0u;
                base[k] = total + __reduce_add_sync(0xFFFFFFFFu, lane < warp ? tl : 0u);   // before my warp's unit run
                total += __reduce_add_sync(0xFFFFFFFFu, tl);
                realA += __reduce_add_sync(0xFFFFFFFFu, tla);                             // records of piece A
            }
            const unsigned pad = (ngtB > 0) ? (kGroup - realA % kGroup) % kGroup : 0u;
            total += pad;
            nact = static_cast<int>(total);
            nactA_pad = (ngtB > 0) ? static_cast<int>(realA + pad) : ((nact + kGroup - 1) / kGroup) * kGroup;
            const unsigned slotA0 = gA * kTileK - jA0, slotB0 = gB * kTileK;                 // column slot of column 0
#pragma unroll
            for (int k = 0; k < kListPasses; ++k) {
                const unsigned m = m8[k];
                if (m != 0u) {
                    const int v0 = (k * kThreads + t) * 8;
                    const bool inB = v0 >= vB0;
                    const unsigned slot0 = inB ? slotB0 + (v0 - vB0) : slotA0 + jA0 + v0;   // column slot of position v0
                    int item = static_cast<int>(base[k] + (inB ? pad : 0u) + below[k]);
                    const unsigned to = sm.stage.tileoff[v0 >> 4];
                    const uint4 xv = *reinterpret_cast<const uint4*>(&sm.stage.x[v0]);
                    const uint4 c0 = *reinterpret_cast<const uint4*>(&sm.stage.colinfo[v0]);
                    const uint4 c1 = *reinterpret_cast<const uint4*>(&sm.stage.colinfo[v0 + 4]);
                    const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w};
                    const unsigned ci[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};   // ColInfo: offset << 16 | nnz
#pragma unroll
                    for (int b = 0; b < 8; ++b) {
                        if ((m >> b) & 1u) {
                            const unsigned start = to + (ci[b] >> 16), pieces = ((ci[b] & 0xFFFFu) + 7u) >> 3;
                            const bool ok = SPDP_CHECK(p.status, item, 1, kChunkCols, kSiteRecordIndex);
                            if (ok && SPDP_CHECK(p.status, start, 8u * pieces, p.values_len, kSiteValuesSpan) &&
                                SPDP_CHECK(p.status, 0, pieces, 32, kSitePieces) &&
                                SPDP_CHECK(p.status, slot0 + b, 1, p.NGT * kTileK, kSiteBitmapSlot)) {
                                sm.rec[item] = make_uint2(start, ((slot0 + b) << 6) | pieces);
                                sm.xact[item] = static_cast<unsigned short>((b & 1) ? (xw[b >> 1] >> 16) : (xw[b >> 1] & 0xFFFFu));
                            } else if (ok) {
                                sm.rec[item] = make_uint2(0u, kNullRec);       // checked build only: the tile is left out
                            }
                            ++item;
                        }
                    }
                }
            }
            // null records: the padding in front of piece B and behind the last record
            if (warp == 0 && lane < static_cast<int>(pad)) sm.rec[realA + lane] = make_uint2(0u, kNullRec);
            if (t < kRecPad) sm.rec[nact + t] = make_uint2(0u, kNullRec);
        }
        __syncthreads();       // the records are complete; the staging area becomes the ring again
        const int ngroups = (nact + kGroup - 1) / kGroup;

        // ---- (2) per-warp fetch / decode pipeline over groups warp, warp + kWarps, ... ----
        const int groupsA = nactA_pad / kGroup;                 // groups [0, groupsA) belong to piece A
        // Carried from group to group: lq = the group being decoded, (dv, db) = its ring position as
        // byte offsets into the values ring / the bitmap table, rec_nxt = my record of the next group to fetch.
        int lq = warp;
        uint32_t dv = 0, db = 0;
        uint32_t rec_nxt = rec_addr + 8u * (warp * kGroup + lgrp);
        // start the copies of group glq (my record at rec_a) into ring position (dv_f, db_f)
        auto fetch_group = [&](uint32_t rec_a, uint32_t dv_f, uint32_t db_f) {
            const uint2 rc = lds_v2(rec_a);
            const uint32_t bdst = bm_own + db_f;
            if (rc.y != kNullRec) {
                const int rem = static_cast<int>(rc.y & 63u) - lane7;                  // my 16-byte pieces left
                const unsigned char* src = offset_wide<2>(val_src, rc.x);
                const uint32_t dst = val_dst + dv_f;
                cp_async16<0>(dst, src, rem);
                cp_async16<128>(dst, src, rem);
                cp_async16<256>(dst, src, rem);
                cp_async16<384>(dst, src, rem);
                cp_async4(bdst, offset_wide<32>(bm_src, rc.y >> 6));
            } else {
                sts_u32(bdst, 0u);
            }
            cp_async_commit();
        };
#pragma unroll
        for (int dd = 0; dd < kDepth; ++dd) {
            fetch_group(rec_nxt, dd * kStageBytes, dd * 128);
            rec_nxt += 8u * kGroup * kWarps;
        }
        // one group: wait for its copies, scan, decode, refill its ring position with the group kDepth ahead
        auto one_group = [&]() {
            cp_async_wait<kDepth - 1>();
            __syncwarp();
            {   // scan role: address of my word's first value inside the warp's ring
                const uint32_t own = bm_own + db;
                const unsigned cnt = __popc(lds_u32(own));
                unsigned inc = cnt;
                scan8_level<1>(inc);
                scan8_level<2>(inc);
                scan8_level<4>(inc);
                sts_u32<kVoFromBm>(own, ring_slot + dv + 2u * (inc - cnt));
            }
            __syncwarp();
            // decode role: my 16 words (tile it, word 2s + lhalf at index 4*it + s), their value addresses, the 4 x
            const uint32_t bmd = bm_dec + db;
            const uint2 xs = lds_v2(x_addr + 8u * lq);
#pragma unroll 1
            for (int pr = 0; pr < 2; ++pr) {                                     // two column tiles per pass
                const uint32_t ah = bmd + 32 * pr;
                const unsigned x2 = pr ? xs.y : xs.x;                            // their two activations
                {
                    const uint4 w = lds_v4<0>(ah);
                    const uint4 a = lds_v4<kVoFromBm>(ah);
                    decode_step<false>(w.x, a.x, lt_mask, bit0, bit1, x2, acc[0], acc[1]);
                    decode_step<false>(w.y, a.y, lt_mask, bit0, bit1, x2, acc[2], acc[3]);
                    decode_step<false>(w.z, a.z, lt_mask, bit0, bit1, x2, acc[4], acc[5]);
                    decode_step<false>(w.w, a.w, lt_mask, bit0, bit1, x2, acc[6], acc[7]);
                }
                {
                    const uint4 w = lds_v4<16>(ah);
                    const uint4 a = lds_v4<kVoFromBm + 16>(ah);
                    decode_step<true>(w.x, a.x, lt_mask, bit0, bit1, x2, acc[0], acc[1]);
                    decode_step<true>(w.y, a.y, lt_mask, bit0, bit1, x2, acc[2], acc[3]);
                    decode_step<true>(w.z, a.z, lt_mask, bit0, bit1, x2, acc[4], acc[5]);
                    decode_step<true>(w.w, a.w, lt_mask, bit0, bit1, x2, acc[6], acc[7]);
                }
            }
            __syncwarp();                  // everyone is done with this ring position
            fetch_group(rec_nxt, dv, db);  // refill it with the group kDepth ahead (null records past the end)
            rec_nxt += 8u * kGroup * kWarps;
            lq += kWarps;
            if (kDepth == 2) {
                dv ^= kStageBytes;
                db ^= 128u;
            } else {
                dv = (dv == (kDepth - 1) * kStageBytes) ? 0u : dv + kStageBytes;
                db = (db == (kDepth - 1) * 128u) ? 0u : db + 128u;
            }
        };
        auto park_first = [&]() {      // my share of the first piece is complete: park it, restart from zero
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                *reinterpret_cast<float2*>(&sm.red_first[warp][64 * q + 2 * lane]) = make_float2(acc[2 * q], acc[2 * q + 1]);
                acc[2 * q] = 0.f;
                acc[2 * q + 1] = 0.f;
            }
        };
        int park_at = (ngtB > 0) ? groupsA : 0x7FFFFFFF;      // the first group of piece B (none: never)
        while (lq < ngroups) {
            if (lq >= park_at) {
                park_at = 0x7FFFFFFF;
                park_first();
            }
            one_group();
        }
        if (ngtB > 0 && park_at != 0x7FFFFFFF) park_first();
        cp_async_wait<0>();
        __syncthreads();       // all pipelines drained: the ring is idle

        // ---- (3) finish the row tiles this batch completed ----
        const bool two = (ngtB > 0);
        const bool done_last = two ? doneB : doneA;             // does the batch's last piece end its row tile here?
        if (done_last) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {                       // red[] reuses the idle ring
                *reinterpret_cast<float2*>(&sm.red[warp][64 * q + 2 * lane]) = make_float2(acc[2 * q], acc[2 * q + 1]);
                acc[2 * q] = 0.f;
                acc[2 * q + 1] = 0.f;
            }
        }
        __syncthreads();
        // Threads 0..255 take the batch's last row tile, threads 256..511 the first one of a two-piece
        // batch; the other warps go straight on to the next batch's list phase.  Neither red[] nor
        // red_first[] is written again before these threads have passed the next __syncthreads.
        if (t < kTileM) {
            if (done_last) finish_row_tile(p, two ? rB : rA, sm.red, t);
        } else if (t < 2 * kTileM) {
            if (two) finish_row_tile(p, rA, sm.red_first, t - kTileM);
        }
    }
}

// Launch helper shared by the entry points.  The launch carries the programmatic-stream-serialization
// attribute: the CTAs of this kernel may start while the previous kernel in the stream is still
// draining, stage the matrix metadata of their range (which no kernel in the stream writes), and
// only then wait for the previous kernel (griddepcontrol.wait) before they touch x, y or the
// workspace.  Back-to-back calls overlap one call's tail with the next call's prologue.
spdp_status launch_kernel(const Params& p, int num_ctas, cudaStream_t s) {
    spdp_status st = configure_spmspv_kernel();        // a flag test after the first call on a device
    if (st != SPDP_OK) return st;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(num_ctas));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = sizeof(Smem);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    SPDP_CUDA_TRY(cudaLaunchKernelEx(&cfg, spmspv_kernel, p));
    return SPDP_OK;
}

__global__ void active_columns_kernel(const __half* __restrict__ x, int K, int rule, float thr,
                                      const uint32_t* __restrict__ mask, uint32_t* __restrict__ bits,
                                      int* __restrict__ count) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    bool a = false;
    if (j < K) a = column_active(rule, thr, mask, j, x[j]);
    const unsigned m = __ballot_sync(0xFFFFFFFFu, a);
    if ((threadIdx.x & 31) == 0 && (j >> 5) < ((K + 31) >> 5)) {
        bits[j >> 5] = m;
        if (count != nullptr && m != 0) atomicAdd(count, __popc(m));
    }
}


// ---- allocation-free variant: scratch in a file-scope device array --------------------------
// What spdp_spmspv keeps in handle-owned allocations (the device status word and the workspace of
// split-K tree nodes, one row of 256 per CTA) lives here instead, so the entry point below never
// allocates.  One copy per device that loads the library, held until exit.
constexpr int kNoAllocMaxCtas = 512;

struct NoAllocScratch {
    int status;
    alignas(16) float workspace[kNoAllocMaxCtas * kTileM];
};

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

// Empties what a call expects to find empty (the array keeps whatever an aborted call left).
__global__ void noalloc_setup_kernel(NoAllocScratch* sc, int words) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < words; i += gridDim.x * blockDim.x) sc->workspace[i] = 0.f;
    if (blockIdx.x == 0 && threadIdx.x == 0) sc->status = 0;
}

}  // namespace

int default_ctas_per_sm() { return kCtasPerSm; }

// Opts the kernel in to its large dynamic shared memory, once per device (handle creation calls
// this, so spdp_spmspv itself only launches).
spdp_status configure_spmspv_kernel() {
    static std::mutex mu;
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SPDP_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(spmspv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(sizeof(Smem))));
        configured[dev] = true;
    }
    return SPDP_OK;
}

spdp_status launch_spmspv(const spdp_matrix* h, const __half* x, int rule, float thr,
                          const uint32_t* mask, void* y, int ydt, cudaStream_t s) {
    Params p;
    p.tileoffset = h->tileoffset;
    p.colinfo = h->colinfo;
    p.bitmap = h->bitmap;
    p.values = h->values;
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
    p.values_len = h->values_len;
    return launch_kernel(p, h->num_ctas, s);
}

spdp_status launch_spmspv_noalloc(const uint32_t* tileoffset, const uint32_t* colinfo, const uint64_t* bitmap,
                                  const __half* values, int64_t M, int64_t K, const __half* x, int rule,
                                  float thr, const uint32_t* mask, void* y, int ydt, cudaStream_t s) {
    constexpr int kMaxDevices = 64;
    static NoAllocScratch* scratch_of[kMaxDevices] = {};
    static int sm_count_of[kMaxDevices] = {};
    static std::mutex mu;
    const int64_t R = (M + kTileM - 1) / kTileM, C = (K + kTileK - 1) / kTileK, NGT = R * C;
    if (NGT * kTileK >= (int64_t(1) << 26)) return SPDP_ERR_UNSUPPORTED_SHAPE;
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SPDP_ERR_UNSUPPORTED_SHAPE;
    NoAllocScratch* sc = nullptr;
    int sms = 0;
    {
        // Once per device, with that device current: the array's name is only a host-side stand-in,
        // so ask the runtime for the device address and hand THAT to the kernels.
        std::lock_guard<std::mutex> lock(mu);
        if (scratch_of[dev] == nullptr) {
            void* ptr = nullptr;
            SPDP_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
            SPDP_CUDA_TRY(cudaDeviceGetAttribute(&sm_count_of[dev], cudaDevAttrMultiProcessorCount, dev));
            scratch_of[dev] = static_cast<NoAllocScratch*>(ptr);
        }
        sc = scratch_of[dev];
        sms = sm_count_of[dev];
    }
    int P = sms * kCtasPerSm < kNoAllocMaxCtas ? sms * kCtasPerSm : kNoAllocMaxCtas;
    if (P > NGT) P = static_cast<int>(NGT);
    noalloc_setup_kernel<<<(P * kTileM + 1023) / 1024, 256, 0, s>>>(sc, P * kTileM);
    SPDP_CUDA_TRY(cudaGetLastError());
    Params p;
    p.tileoffset = tileoffset;
    p.colinfo = colinfo;
    p.bitmap = bitmap;
    p.values = values;
    p.x = x;
    p.mask = mask;
    p.y = y;
    p.thr = thr;
    p.rule = rule;
    p.ydt = ydt;
    p.M = static_cast<int>(M);
    p.K = static_cast<int>(K);
    p.R = static_cast<int>(R);
    p.C = static_cast<int>(C);
    p.NGT = NGT;
    p.num_ctas = P;
    p.workspace = sc->workspace;            // addresses inside the device array (no host dereference)
    p.status = &sc->status;
    p.values_len = int64_t(1) << 40;        // the caller owns Values; its length is not known here
    return launch_kernel(p, P, s);
}

spdp_status launch_active_columns(const spdp_matrix* h, const __half* x, int rule, float thr,
                                  const uint32_t* mask, uint32_t* bits, int* count, cudaStream_t s) {
    const int K = static_cast<int>(h->K);
    if (count != nullptr) SPDP_CUDA_TRY(cudaMemsetAsync(count, 0, sizeof(int), s));
    const int threads = 256;
    const int blocks = (((K + 31) / 32) * 32 + threads - 1) / threads;
    active_columns_kernel<<<blocks, threads, 0, s>>>(x, K, rule, thr, mask, bits, count);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
