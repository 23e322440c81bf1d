// spMspV on the 4-bit variant of Tiled-CBC for sm_100a (Sec. 5.1: 4-bit round-to-nearest weights in the
// order static pruning -> quantisation -> dynamic pruning; Sec. 6: Values are stored apart from the
// sparsity metadata, so they can be low-bit).  TileOffset / ColInfo / Bitmap are those of Sec. 4.1
// (offsets count codes, padded to 32 per column tile); Values are 4-bit codes, two per byte, with
// one fp16 scale per column tile: weight = (code - 8) * scale.
//
// The kernel has the structure of the fp16 kernel (Sec. 4.2, Alg. 1): one persistent CTA per GTile range,
// a list phase that turns the range's activations into one record per active column tile, then every
// warp runs its own fetch -> decode pipeline over groups of 4 active column tiles, two groups in flight;
// row tiles fed by several CTAs are combined along the fixed tree of the handle's workspace.  What differs:
//   * a column tile is at most 128 bytes of codes, so a lane copies one 16-byte piece per group;
//   * the list phase also reads the active columns' scales and keeps scale * x (exact in fp32) per record;
//   * decode (Sec. 4.2.1): lane l owns rows 8l .. 8l+7 of a column tile (one bitmap byte); rank = set bits
//     before that byte; its codes are one span of at most 8 nibbles, read as two 32-bit words,
//     funnel-shifted into one register and walked bit by bit (five instructions per row).
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

#ifndef SPDP_Q4_WARPS
#define SPDP_Q4_WARPS 24
#endif
#ifndef SPDP_Q4_CTAS_PER_SM
#define SPDP_Q4_CTAS_PER_SM 1
#endif
#ifndef SPDP_Q4_CHUNK_COLS
#define SPDP_Q4_CHUNK_COLS 8192
#endif
#ifndef SPDP_Q4_DEPTH
#define SPDP_Q4_DEPTH 2
#endif
constexpr int kWarps = SPDP_Q4_WARPS;         // warps per CTA; every warp fetches and decodes its own column tiles
constexpr int kDepth = SPDP_Q4_DEPTH;         // groups a warp keeps in flight
constexpr int kGroup = 4;                  // active column tiles per group (one fetch / decode unit of a warp)
constexpr int kSlotPad = 16;                 // bytes in front of a slot's codes: the decode reads the two 32-bit words that
                                             // END at a lane's last code, the first of which may lie before the codes
constexpr int kSlotBytes = kSlotPad + kTileM / 2;   // + a column tile's codes (at most 256 nibbles); the four tiles of a
                                                    // group start 4 banks apart
constexpr int kStageBytes = kGroup * kSlotBytes;
constexpr int kThreads = kWarps * 32;
constexpr int kChunkCols = SPDP_Q4_CHUNK_COLS; // columns handled between two pipeline drains
constexpr int kCtasPerSm = SPDP_Q4_CTAS_PER_SM;
constexpr uint32_t kNullRec = 0xFFFFFFFFu;
constexpr int kListPasses = (kChunkCols / 8 + kThreads - 1) / kThreads;     // 8-position units a thread lists per batch
constexpr int kChunkGT = kChunkCols / kTileK;
constexpr int kRecPad = kGroup * (kDepth * kWarps + 1);   // null records behind the last real one

struct Params {
    const uint32_t* tileoffset;
    const uint32_t* colinfo;
    const uint64_t* bitmap;
    const unsigned char* codes;
    const __half* scales;
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
    int64_t values_len;     // codes in the array (the checked build holds every fetch against it)
};

struct __align__(128) Smem {
    union {
        unsigned char ring[kWarps][kDepth][kStageBytes];    // values of the column tiles in flight, per warp
        float red[kWarps][kTileM];                          // cross-warp row reduction (after the pipelines drained)
        struct {                                            // list phase: the chunk's ColInfo / TileOffset words,
            float keep_clear_of_red[kWarps][kTileM];        // placed behind red[], which may still be read
            alignas(16) uint32_t colinfo[kChunkCols];
            alignas(16) unsigned short x[kChunkCols];       // the activations of the listed columns
            alignas(16) unsigned short scale[kChunkCols];   // and their column tiles' scales
            uint32_t tileoff[kChunkGT];
        } stage;
    };
    // Bitmap words of a group: word w of the group's it-th tile sits at [it * 8 + w].
    struct alignas(16) WarpTab {
        uint32_t bm[kDepth][32];
        uint32_t vo[kDepth][32];                        // same order: codes of the column tile before each word
    } tab[kWarps];
    // Active list of the chunk, one record per active column tile (filled once per chunk):
    alignas(16) uint2 rec[kChunkCols + kRecPad];        // .x = start of its values in Values (elements),
                                                        // .y = (column slot in Bitmap/ColInfo) << 6 | 16-byte pieces
                                                        //      of values; kNullRec pads a piece to whole groups and
                                                        //      follows the last record for kRecPad entries, so a warp
                                                        //      can fetch kDepth groups ahead without a range test
    alignas(16) float xact[kChunkCols + kGroup];        // its scale * x_j (the product of two fp16 is exact in fp32)
    float red_first[kWarps][kTileM];                    // row reduction of a batch's first piece (flushed mid-stream)
    uint32_t warp_total[kListPasses][kWarps][2];        // list phase: records listed by each warp per pass (all, piece A)
};
static_assert(offsetof(Smem, rec) % 16 == 0 && offsetof(Smem, xact) % 16 == 0 && offsetof(Smem, tab) % 16 == 0, "16-byte shared loads need aligned tables");
static_assert(sizeof(Smem) <= (227 * 1024) / kCtasPerSm - 1024 * (kCtasPerSm - 1), "shared memory of one CTA");
static_assert(kRecPad <= kThreads, "one thread per trailing null record");
static_assert(kWarps >= 16, "two groups of 256 threads finish two row tiles side by side");

// The walk over a lane's 8 rows (Sec. 4.2.1 with 4-bit codes), from the last row to the first: `span` holds the
// lane's codes with the LAST one in the top nibble; a set bit takes the top nibble and shifts the span left.
// mad.hi(span, 16, 2^23-as-float bits) = (span >> 28) | 0x4B000000 = 2^23 + code as a float, so one subtraction
// turns the code into code - 8 without a conversion; acc[row] += (code - 8) * (scale * x).  Five instructions per
// row, the last two predicated; only the bit test uses the integer pipe (the multiply-high, the subtraction, the
// FMA and the shift-as-multiply go to the FMA pipe).
#define SPDP_Q4_ROW(K)                                              \
    " lop3.or.b32 t|p, %9, " #K ", 0, 0xC0, 0;\n"                  \
    " mad.hi.u32 c, %8, 16, 0x4B000000;\n"                         \
    " add.f32 w, c, 0fCB000008;\n"
__device__ __forceinline__ void walk_codes(unsigned bits, unsigned span, float sx, float (&acc)[8]) {
    asm volatile(
        "{\n"
        " .reg .pred p;\n"
        " .reg .b32 t, c;\n"
        " .reg .f32 w;\n"
        SPDP_Q4_ROW(128) " @p fma.rn.f32 %7, w, %10, %7;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(64)  " @p fma.rn.f32 %6, w, %10, %6;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(32)  " @p fma.rn.f32 %5, w, %10, %5;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(16)  " @p fma.rn.f32 %4, w, %10, %4;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(8)   " @p fma.rn.f32 %3, w, %10, %3;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(4)   " @p fma.rn.f32 %2, w, %10, %2;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(2)   " @p fma.rn.f32 %1, w, %10, %1;\n @p mul.lo.u32 %8, %8, 16;\n"
        SPDP_Q4_ROW(1)   " @p fma.rn.f32 %0, w, %10, %0;\n"
        "}"
        : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3]), "+f"(acc[4]), "+f"(acc[5]), "+f"(acc[6]), "+f"(acc[7]),
          "+r"(span)
        : "r"(bits), "f"(sx));
}
#undef SPDP_Q4_ROW
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
spmspv_q4_kernel(const Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const unsigned g_begin = range_begin(p, blockIdx.x), g_end = range_begin(p, blockIdx.x + 1);

    const int lane7 = lane & 7;
    const int lgrp = lane >> 3;
    // fetch role: lane (lgrp, lane7) moves 16-byte piece lane7 and bitmap word lane7 of the group's lgrp-th tile.
    // scan role: the same (tile, word).  decode role: lane l owns rows 8l .. 8l+7 of every tile of the group: byte
    // l % 4 of bitmap word l / 4.
    const int tpos = lgrp * 8 + lane7;                                  // where (tile lgrp, word lane7) sits
    const unsigned bsh = pinned(8u * (lane & 3));
    const unsigned bbelow = pinned((1u << (8 * (lane & 3))) - 1u);      // the bits of my word below my byte
    const uint32_t val_dst = pinned(smem_u32(&sm.ring[warp][0][lgrp * kSlotBytes + kSlotPad + 16 * lane7]));
    const uint32_t bm_own = pinned(smem_u32(&sm.tab[warp].bm[0][tpos]));
    const uint32_t bm_dec = pinned(smem_u32(&sm.tab[warp].bm[0][lane >> 2]));
    constexpr int kVoFromBm = kDepth * 128;             // vo[d][i] sits this many bytes behind bm[d][i]
    const uint32_t ring_warp = pinned(smem_u32(&sm.ring[warp][0][0]));
    // fetch role: my 16-byte piece of a column tile's codes / my bitmap word, before the tile's offset is added
    const unsigned char* const val_src = pinned(p.codes + 16 * lane7);
    const unsigned char* const bm_src = pinned(reinterpret_cast<const unsigned char*>(p.bitmap) + 4 * lane7);
    const uint32_t rec_addr = smem_u32(&sm.rec[0]);
    const uint32_t x_addr = smem_u32(&sm.xact[0]);

    // Let a dependent launch (the next call) begin as soon as SMs free up.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited_for_stream = false;  // x, y, workspace and counters may belong to the previous kernel until we wait

    float acc[8];                   // acc[k] = row 8*lane + k of the current row tile
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
            const uint32_t sc_stage = smem_u32(&sm.stage.scale[0]);                         // 16 scales = 32 bytes per GTile
            const uint4* scA = reinterpret_cast<const uint4*>(p.scales + static_cast<size_t>(gA) * kTileK);
            const uint4* scB = reinterpret_cast<const uint4*>(p.scales + static_cast<size_t>(gB) * kTileK);
            for (int i = t; i < ngtA * 2; i += kThreads) cp_async16<0>(sc_stage + 16 * i, scA + i, 1);
            for (int i = t; i < ngtB * 2; i += kThreads) cp_async16<0>(sc_stage + 2 * vB0 + 16 * i, scB + i, 1);
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
                    const uint4 sv = *reinterpret_cast<const uint4*>(&sm.stage.scale[v0]);
                    const uint4 c0 = *reinterpret_cast<const uint4*>(&sm.stage.colinfo[v0]);
                    const uint4 c1 = *reinterpret_cast<const uint4*>(&sm.stage.colinfo[v0 + 4]);
                    const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w};
                    const unsigned sw[4] = {sv.x, sv.y, sv.z, sv.w};
                    const unsigned ci[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};   // ColInfo: offset << 16 | nnz
#pragma unroll
                    for (int b = 0; b < 8; ++b) {
                        if ((m >> b) & 1u) {
                            // codes of the column tile: start (in codes, a multiple of 32), 16-byte pieces of 32 codes
                            const unsigned start = to + (ci[b] >> 16), pieces = ((ci[b] & 0xFFFFu) + 31u) >> 5;
                            const bool ok = SPDP_CHECK(p.status, item, 1, kChunkCols, kSiteRecordIndex);
                            if (ok && SPDP_CHECK(p.status, start, 32u * pieces, p.values_len, kSiteValuesSpan) &&
                                SPDP_CHECK(p.status, 0, pieces, 8, kSitePieces) &&
                                SPDP_CHECK(p.status, slot0 + b, 1, p.NGT * kTileK, kSiteBitmapSlot)) {
                                const unsigned short xb = static_cast<unsigned short>((b & 1) ? (xw[b >> 1] >> 16) : (xw[b >> 1] & 0xFFFFu));
                                const unsigned short sb = static_cast<unsigned short>((b & 1) ? (sw[b >> 1] >> 16) : (sw[b >> 1] & 0xFFFFu));
                                sm.rec[item] = make_uint2(start, ((slot0 + b) << 6) | pieces);
                                sm.xact[item] = __half2float(__ushort_as_half(sb)) * __half2float(__ushort_as_half(xb));
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
                const int rem = static_cast<int>(rc.y & 63u) - lane7;                  // > 0: the tile has my piece
                cp_async16<0>(val_dst + dv_f, offset_wide<1>(val_src, rc.x >> 1), rem);
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
            {   // scan role: codes of my tile before my word
                const uint32_t own = bm_own + db;
                const unsigned cnt = __popc(lds_u32(own));
                unsigned inc = cnt;
                scan8_level<1>(inc);
                scan8_level<2>(inc);
                scan8_level<4>(inc);
                sts_u32<kVoFromBm>(own, inc - cnt);
            }
            __syncwarp();
            // decode role: per tile of the group my word, the codes before it, and scale * x of the column
            const uint32_t bmd = bm_dec + db;
            const uint4 sx4 = lds_v4<0>(x_addr + 16u * lq);
            const float sx[4] = {__uint_as_float(sx4.x), __uint_as_float(sx4.y), __uint_as_float(sx4.z), __uint_as_float(sx4.w)};
#pragma unroll
            for (int it = 0; it < kGroup; ++it) {
                const unsigned W = lds_u32(bmd + 32 * it);
                const unsigned rank = lds_u32(bmd + 32 * it + kVoFromBm) + __popc(W & bbelow);   // codes before my byte
                const unsigned bits = (W >> bsh) & 0xFFu;
                // my codes: the at most 8 nibbles that end before nibble `rend`, inside the two consecutive 32-bit words
                // that end with the word of nibble `rend` (the word before the codes is padding); last code on top
                const unsigned rend = rank + __popc(bits);
                const uint32_t cw = ring_warp + dv + it * kSlotBytes + (kSlotPad - 4) + 4u * (rend >> 3);
                const unsigned span = __funnelshift_r(lds_u32(cw), lds_u32(cw + 4), 4u * (rend & 7u));
                walk_codes(bits, span, sx[it], acc);
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
                *reinterpret_cast<float2*>(&sm.red_first[warp][8 * lane + 2 * q]) = make_float2(acc[2 * q], acc[2 * q + 1]);
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
                *reinterpret_cast<float2*>(&sm.red[warp][8 * lane + 2 * q]) = make_float2(acc[2 * q], acc[2 * q + 1]);
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

}  // namespace

// Opts the kernel in to its large dynamic shared memory, once per device (handle creation calls this).
spdp_status configure_spmspv_q4_kernel() {
    static std::mutex mu;
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SPDP_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(spmspv_q4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(sizeof(Smem))));
        configured[dev] = true;
    }
    return SPDP_OK;
}

// The launch carries the programmatic-stream-serialization attribute, as the fp16 kernel's does: the CTAs may
// start while the previous kernel in the stream drains, stage the matrix metadata of their range, and wait
// for the previous kernel (griddepcontrol.wait) before they touch x, y or the workspace.
spdp_status launch_spmspv_q4(const spdp_matrix* h, const __half* x, int rule, float thr, const uint32_t* mask, void* y,
                             int ydt, cudaStream_t s) {
    Params p;
    p.tileoffset = h->tileoffset;
    p.colinfo = h->colinfo;
    p.bitmap = h->bitmap;
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
    p.values_len = h->values_len;
    spdp_status st = configure_spmspv_q4_kernel();
    if (st != SPDP_OK) return st;
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
    SPDP_CUDA_TRY(cudaLaunchKernelEx(&cfg, spmspv_q4_kernel, p));
    return SPDP_OK;
}

}  // namespace spdp
