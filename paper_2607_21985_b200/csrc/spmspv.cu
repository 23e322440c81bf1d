// SPDP spMspV for sm_100a (Sec. 4.2, Alg. 1): y = W_sp * x over the columns that pass the
// dynamic-pruning test, W_sp in Tiled-CBC.
//
// Work split (Sec. 4.2.3 "tile-based scheme combined with Split-K"): the NGT GTiles, in their
// row-major storage order, are cut into num_ctas equal contiguous ranges, one per CTA.  A range
// touches one or more row tiles; each (CTA, row tile) piece is a "segment" that yields 256
// fp32 partial sums.  A row tile fed by one segment is written to y directly; otherwise the
// partials go to the handle's workspace (the paper's ReductionWorkspace) and the CTA that
// arrives last at the row tile's counter adds them in segment order -- no CTA ever waits for
// another, and the order of the additions is fixed.  Only the first and the last segment of a
// CTA can share their row tile with another CTA, so a CTA owns two workspace slots: slot 0 for
// the row tile its range starts in, slot 1 for any later one.
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"

namespace spdp {
namespace {

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
constexpr int kListPasses = (kChunkCols / 32 + kWarps - 1) / kWarps;   // 32-column groups a warp scans per chunk
constexpr int kChunkGT = kChunkCols / kTileK;

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
    const uint32_t* cta_begin;
    const int32_t* row_first_cta;
    const int32_t* row_nseg;
    float* workspace;
    unsigned* row_counter;
    int* status;
};

struct __align__(128) Smem {
    union {
        unsigned char ring[kWarps][kDepth][kStageBytes];    // values of the column tiles in flight, per warp
        float red[kWarps][kTileM];                          // cross-warp row reduction (after the pipelines drained)
        struct {                                            // list phase: the chunk's ColInfo / TileOffset words,
            float keep_clear_of_red[kWarps][kTileM];        // placed behind red[], which may still be read
            alignas(16) uint32_t colinfo[kChunkCols];
            uint32_t tileoff[kChunkGT];
        } stage;
    };
    // Bitmap words of a group in decode order: word w of the group's it-th tile sits at
    // [(w & 3) * 8 + it * 2 + (w >> 2)], so the lanes that decode words (w & 3) == g read 8 consecutive words.
    alignas(16) uint32_t bmring[kWarps][kDepth][32];
    alignas(16) uint32_t vaddr[kWarps][32];             // same order: shared address of each word's first value
    // Active list of the chunk, one record per active column tile (filled once per chunk):
    alignas(16) uint2 rec[kChunkCols + kGroup];         // .x = start of its values in Values (elements),
                                                        // .y = (column in chunk) << 6 | 16-byte pieces of values
    alignas(16) unsigned short xact[kChunkCols + kGroup];   // its activation x_j (fp16 bits)
    uint32_t group_mask[kChunkCols / 32];
    uint32_t group_base[kChunkCols / 32 + 1];
    int is_last;
};
static_assert(offsetof(Smem, rec) % 16 == 0 && offsetof(Smem, xact) % 16 == 0 && offsetof(Smem, vaddr) % 16 == 0 &&
              offsetof(Smem, bmring) % 16 == 0, "16-byte shared loads need aligned tables");
static_assert(sizeof(float) * kWarps * kTileM <= size_t(kWarps) * kDepth * kStageBytes, "red must fit in the ring");
static_assert(sizeof(uint32_t) * (kChunkCols + kChunkGT) + sizeof(float) * kWarps * kTileM <= size_t(kWarps) * kDepth * kStageBytes,
              "staging must fit in the ring behind red");
static_assert(sizeof(Smem) <= (227 * 1024) / kCtasPerSm - 1024 * (kCtasPerSm - 1), "shared memory of one CTA");

// DP test of Sec. 4.2 step (3): magnitude against the threshold; NOT(|x| <= thr) keeps NaN.
__device__ __forceinline__ bool column_active(int rule, float thr, const uint32_t* mask, int j, __half xj) {
    if (rule == SPDP_DP_NONE) return true;
    if (rule == SPDP_DP_ABS_GT) return !(fabsf(__half2float(xj)) <= thr);
    return (mask[j >> 5] >> (j & 31)) & 1u;
}

__device__ __forceinline__ void store_y(void* y, int ydt, int64_t i, float v) {
    if (ydt == SPDP_Y_F32) static_cast<float*>(y)[i] = v;
    else static_cast<__half*>(y)[i] = __float2half_rn(v);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// Asynchronous global -> shared copies (Sec. 4.2.3: 128-bit per thread); `on` = false copies nothing.
template <int kOff>
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int rem) {
    asm volatile("{\n .reg .pred p;\n setp.gt.s32 p, %2, %3;\n @p cp.async.cg.shared.global [%0+%4], [%1+%4], 16;\n}"
                 ::"r"(dst), "l"(src), "r"(rem), "n"(kOff / 16), "n"(kOff) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One decode step (Sec. 4.2.1): the 4 consecutive rows this lane owns inside the 32-bit bitmap
// word W.  `first` is the shared-memory address of the word's first value, `below` masks the bits
// of lower nibbles, m0..m3 are the lane's four bits.  rank = set bits before the position; a set
// bit takes the next value and adds value * x to its row's fp32 accumulator.  fma.rn.f32.f16
// multiplies two fp16 exactly and accumulates in fp32.
__device__ __forceinline__ void decode_step(unsigned W, uint32_t first, unsigned below, unsigned m0, unsigned m1,
                                            unsigned m2, unsigned m3, unsigned x32, float& a0, float& a1,
                                            float& a2, float& a3) {
    asm volatile(
        "{\n"
        " .reg .pred p0, p1, p2, p3;\n"
        " .reg .b16 v0, v1, v2, v3, xl, xu;\n"
        " .reg .b32 t, a;\n"
        " and.b32 t, %4, %6;\n"
        " popc.b32 t, t;\n"
        " shl.b32 t, t, 1;\n"
        " add.u32 a, %5, t;\n"
        " lop3.or.b32 t|p0, %4, %7, 0, 0xC0, 0;\n"
        " lop3.or.b32 t|p1, %4, %8, 0, 0xC0, 0;\n"
        " lop3.or.b32 t|p2, %4, %9, 0, 0xC0, 0;\n"
        " lop3.or.b32 t|p3, %4, %10, 0, 0xC0, 0;\n"
        " mov.b32 {xl, xu}, %11;\n"
        " @p0 ld.shared.u16 v0, [a];\n @p0 add.u32 a, a, 2;\n"
        " @p1 ld.shared.u16 v1, [a];\n @p1 add.u32 a, a, 2;\n"
        " @p2 ld.shared.u16 v2, [a];\n @p2 add.u32 a, a, 2;\n"
        " @p3 ld.shared.u16 v3, [a];\n"
#if SPDP_FMA_MODE == 0
        " @p0 fma.rn.f32.f16 %0, v0, xl, %0;\n"
        " @p1 fma.rn.f32.f16 %1, v1, xl, %1;\n"
        " @p2 fma.rn.f32.f16 %2, v2, xl, %2;\n"
        " @p3 fma.rn.f32.f16 %3, v3, xl, %3;\n"
#else
        " .reg .f32 f0, f1, f2, f3, fx;\n"
        " cvt.f32.f16 fx, xl;\n"
        " @p0 cvt.f32.f16 f0, v0;\n @p1 cvt.f32.f16 f1, v1;\n @p2 cvt.f32.f16 f2, v2;\n @p3 cvt.f32.f16 f3, v3;\n"
        " @p0 fma.rn.f32 %0, f0, fx, %0;\n"
        " @p1 fma.rn.f32 %1, f1, fx, %1;\n"
        " @p2 fma.rn.f32 %2, f2, fx, %2;\n"
        " @p3 fma.rn.f32 %3, f3, fx, %3;\n"
#endif
        "}"
        : "+f"(a0), "+f"(a1), "+f"(a2), "+f"(a3)
        : "r"(W), "r"(first), "r"(below), "r"(m0), "r"(m1), "r"(m2), "r"(m3), "r"(x32));
}
__device__ __forceinline__ unsigned lds_u32(uint32_t addr) {
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, unsigned v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// One persistent CTA per GTile range; every warp runs its own fetch -> decode pipeline.
// Per chunk of the range:
//   (1) all warps: ColInfo / TileOffset of the chunk to shared memory and the active-column list
//       from x (ballots + prefix sums) -- Sec. 4.2 steps (1)-(3);
//   (2) each warp takes groups of kGroup active column tiles round-robin.  It keeps kDepth
//       groups in flight: the padded values of a column tile arrive with 16-byte asynchronous
//       copies (lane = one 16-byte piece of one of the group's tiles), its 8 bitmap words with
//       4-byte ones; inactive columns are never touched.  Decode (Sec. 4.2.1): lane owns 4
//       consecutive rows of a half column tile, rank = set bits before them, values read from
//       shared memory, fp32 accumulation in registers;
//   (3) segment end: cross-warp row reduction, split-K combine, store.
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
spmspv_kernel(const Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int64_t g_begin = p.cta_begin[blockIdx.x], g_end = p.cta_begin[blockIdx.x + 1];
    const int r_first = static_cast<int>(g_begin / p.C);

    const int lane7 = lane & 7;
    const int lgrp = lane >> 3;
    const unsigned bit0 = 1u << (4 * lane7);        // first bit of my nibble inside a 32-bit bitmap word
    const unsigned lt_mask = bit0 - 1u;
    // fetch role: lane (lgrp, lane7) moves 16-byte pieces lane7, lane7+8, ... and bitmap word lane7 of the
    // group's lgrp-th tile.  scan role: the same (tile, word).  decode role: nibble lane7 of words w with
    // (w & 3) == lgrp of every tile of the group.
    const int tpos = (lane7 & 3) * 8 + lgrp * 2 + (lane7 >> 2);         // where (tile lgrp, word lane7) sits
    const uint32_t val_dst = smem_u32(&sm.ring[warp][0][lgrp * kSlotBytes + 16 * lane7]);
    const uint32_t bm_own = smem_u32(&sm.bmring[warp][0][tpos]);
    const uint32_t bm_dec = smem_u32(&sm.bmring[warp][0][lgrp * 8]);
    const uint32_t va_own = smem_u32(&sm.vaddr[warp][tpos]);
    const uint32_t va_dec = smem_u32(&sm.vaddr[warp][lgrp * 8]);
    const uint32_t slot_own = smem_u32(&sm.ring[warp][0][lgrp * kSlotBytes]);      // scan role: my tile's slot
    const uint32_t rec_addr = smem_u32(&sm.rec[0]);
    const uint32_t x_addr = smem_u32(&sm.xact[0]);
    const unsigned char* bm8 = reinterpret_cast<const unsigned char*>(p.bitmap);
    const unsigned char* val_src = reinterpret_cast<const unsigned char*>(p.values) + 16 * lane7;   // fetch role

    for (int64_t g0 = g_begin; g0 < g_end;) {
        const int r = static_cast<int>(g0 / p.C);
        const int c_lo = static_cast<int>(g0 - static_cast<int64_t>(r) * p.C);
        const int64_t c_end = c_lo + (g_end - g0);
        const int c_hi = static_cast<int>(c_end < p.C ? c_end : p.C);
        g0 += c_hi - c_lo;

        float acc[8];                   // rows 4*lane+k (k<4) and 128+4*lane+(k-4) of the row tile
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;

        const int64_t row_slot0 = static_cast<int64_t>(r) * p.C * kTileK;       // column slot of column 0
        for (int cg = c_lo; cg < c_hi; cg += kChunkGT) {
            const int ngt = min(kChunkGT, c_hi - cg);
            const int j0 = cg * kTileK, j_hi = min((cg + ngt) * kTileK, p.K);
            const int ncols = j_hi - j0;
            const int ngroups32 = (ncols + 31) >> 5;
            const int64_t gt0 = static_cast<int64_t>(r) * p.C + cg;

            // ---- (1) active-column list of the chunk (ballots + prefix sums) and its records ----
            // One memory round trip: the chunk's ColInfo and TileOffset words stream into the idle
            // ring with asynchronous copies while x is read and tested.  ColInfo of skipped columns
            // is read too (4 bytes per column tile); their bitmaps and values never are.
            {
                const uint32_t ci_stage = smem_u32(&sm.stage.colinfo[0]);
                const uint32_t to_stage = smem_u32(&sm.stage.tileoff[0]);
                const uint4* ci_src = reinterpret_cast<const uint4*>(p.colinfo + gt0 * kTileK);
                for (int i = t; i < ngt * (kTileK / 4); i += kThreads) cp_async16<0>(ci_stage + 16 * i, ci_src + i, 1);
                for (int i = t; i < ngt; i += kThreads) cp_async4(to_stage + 4 * i, p.tileoffset + gt0 + i);
                cp_async_commit();
            }
            unsigned xb[kListPasses], act[kListPasses];
#pragma unroll
            for (int u = 0; u < kListPasses; ++u) {
                const int j = j0 + (warp + u * kWarps) * 32 + lane;
                xb[u] = 0u;
                act[u] = 0u;
                if (j < j_hi) {
                    xb[u] = __half_as_ushort(p.x[j]);
                    if (p.rule == SPDP_DP_MASK) act[u] = __ldg(p.mask + (j >> 5));
                }
            }
#pragma unroll
            for (int u = 0; u < kListPasses; ++u) {
                const int q = warp + u * kWarps;
                const int j = j0 + q * 32 + lane;
                bool a = false;
                if (j < j_hi) {
                    if (p.rule == SPDP_DP_NONE) a = true;
                    else if (p.rule == SPDP_DP_ABS_GT)
                        a = !(fabsf(__half2float(__ushort_as_half(static_cast<unsigned short>(xb[u])))) <= p.thr);
                    else a = (act[u] >> (j & 31)) & 1u;
                }
                act[u] = __ballot_sync(0xFFFFFFFFu, a);
                if (lane == 0 && q < ngroups32) sm.group_mask[q] = act[u];
            }
            cp_async_wait<0>();
            __syncthreads();
            if (warp == 0) {
                unsigned run = 0;
                for (int q0 = 0; q0 < ngroups32; q0 += 32) {
                    const int q = q0 + lane;
                    unsigned c = (q < ngroups32) ? __popc(sm.group_mask[q]) : 0u;
                    unsigned inc = c;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        unsigned v = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                        if (lane >= d) inc += v;
                    }
                    if (q < ngroups32) sm.group_base[q] = run + inc - c;
                    run += __shfl_sync(0xFFFFFFFFu, inc, 31);
                }
                if (lane == 0) sm.group_base[ngroups32] = run;
            }
            __syncthreads();
#pragma unroll
            for (int u = 0; u < kListPasses; ++u) {
                const int q = warp + u * kWarps;
                if ((act[u] >> lane) & 1u) {
                    const int jj = q * 32 + lane;
                    const int item = static_cast<int>(sm.group_base[q] + __popc(act[u] & ((1u << lane) - 1u)));
                    const uint32_t ci = sm.stage.colinfo[jj];                           // ColInfo: offset << 16 | nnz
                    sm.rec[item] = make_uint2(sm.stage.tileoff[jj >> 4] + (ci >> 16),
                                              (static_cast<unsigned>(jj) << 6) | (((ci & 0xFFFFu) + 7u) >> 3));
                    sm.xact[item] = static_cast<unsigned short>(xb[u]);
                }
            }
            __syncthreads();       // the records are complete; the staging area becomes the ring again
            const int nact = static_cast<int>(sm.group_base[ngroups32]);
            const int ngroups = (nact + kGroup - 1) / kGroup;

            // ---- (2) per-warp fetch / decode pipeline over groups warp, warp + kWarps, ... ----
            const unsigned char* bm_chunk = bm8 + (row_slot0 + j0) * 32 + lane7 * 4;
            // fetch(i): start the copies of my i-th group into ring position i % kDepth
            auto fetch = [&](int i) {
                const int lq = warp + i * kWarps;
                if (lq < ngroups) {
                    const int d = i % kDepth;
                    const int item = lq * kGroup + lgrp;
                    const uint32_t bdst = bm_own + d * 128;
                    if (item < nact) {
                        const uint2 rc = lds_v2(rec_addr + 8u * item);
                        const int rem = static_cast<int>(rc.y & 63u) - lane7;                  // my 16-byte pieces left
                        const unsigned char* src = val_src + 2 * static_cast<uint64_t>(rc.x);
                        const uint32_t dst = val_dst + d * kStageBytes;
                        cp_async16<0>(dst, src, rem);
                        cp_async16<128>(dst, src, rem);
                        cp_async16<256>(dst, src, rem);
                        cp_async16<384>(dst, src, rem);
                        cp_async4(bdst, bm_chunk + static_cast<size_t>(rc.y >> 6) * 32);
                    } else {
                        sts_u32(bdst, 0u);
                    }
                }
                cp_async_commit();
            };
#pragma unroll
            for (int d = 0; d < kDepth; ++d) fetch(d);

            int d = 0;
            for (int i = 0, lq = warp; lq < ngroups; ++i, lq += kWarps) {
                cp_async_wait<kDepth - 1>();
                __syncwarp();
                // scan role: shared address of my word's first value
                {
                    const unsigned cnt = __popc(lds_u32(bm_own + d * 128));
                    unsigned inc = cnt;
#pragma unroll
                    for (int dd = 1; dd < 8; dd <<= 1) {
                        unsigned v = __shfl_up_sync(0xFFFFFFFFu, inc, dd, 8);
                        if (lane7 >= dd) inc += v;
                    }
                    sts_u32(va_own, slot_own + d * kStageBytes + 2u * (inc - cnt));
                }
                __syncwarp();
                // decode role: my 8 words (tile it, word 4h + lgrp at index 2*it + h), their value addresses, the 4 x
                const unsigned m1 = bit0 << 1, m2 = bit0 << 2, m3 = bit0 << 3;
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    const uint4 w = lds_v4(bm_dec + d * 128 + 16 * half);
                    const uint4 a = lds_v4(va_dec + 16 * half);
                    const unsigned xs = lds_u32(x_addr + 8u * lq + 4 * half);        // two activations
                    decode_step(w.x, a.x, lt_mask, bit0, m1, m2, m3, xs, acc[0], acc[1], acc[2], acc[3]);
                    decode_step(w.y, a.y, lt_mask, bit0, m1, m2, m3, xs, acc[4], acc[5], acc[6], acc[7]);
                    decode_step(w.z, a.z, lt_mask, bit0, m1, m2, m3, xs >> 16, acc[0], acc[1], acc[2], acc[3]);
                    decode_step(w.w, a.w, lt_mask, bit0, m1, m2, m3, xs >> 16, acc[4], acc[5], acc[6], acc[7]);
                }
                __syncwarp();                  // everyone is done with ring position d
                fetch(i + kDepth);
                d = (d + 1 == kDepth) ? 0 : d + 1;
            }
            cp_async_wait<0>();
            __syncthreads();       // the chunk's shared tables are rebuilt next; the ring is idle
        }

        // ---- (3) row reduction across the warps (fixed order); red[] reuses the idle ring ----
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            sm.red[warp][4 * lane + k] = acc[k];
            sm.red[warp][128 + 4 * lane + k] = acc[4 + k];
        }
        __syncthreads();
        // The first 256 threads (one per row) finish the segment; the other warps go straight on to
        // the next segment's list phase, whose global loads overlap the combine.  The ring is not
        // written again before the next __syncthreads, which these 256 threads join afterwards.
        if (t < kTileM) {
            float part = 0.f;
            const int64_t row = static_cast<int64_t>(r) * kTileM + t;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) part += sm.red[w][t];
            // ---- split-K combine ----
            const int nseg = p.row_nseg[r];
            if (nseg == 1) {
                if (row < p.M) store_y(p.y, p.ydt, row, part);
            } else {
                float* mine = p.workspace + (static_cast<int64_t>(blockIdx.x) * 2 + (r != r_first)) * kTileM;
                __stcg(mine + t, part);
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (t == 0) {
                    const unsigned old = atomicAdd(p.row_counter + r, 1u);
                    sm.is_last = (old == static_cast<unsigned>(nseg - 1));
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (sm.is_last) {
                    __threadfence();
                    if (row < p.M) {
                        const int q0 = p.row_first_cta[r];
                        float sum = 0.f;
                        for (int s = 0; s < nseg; ++s) {
                            const int q = q0 + s;
                            const int slot = (r != static_cast<int>(p.cta_begin[q] / p.C));
                            sum += __ldcg(p.workspace + (static_cast<int64_t>(q) * 2 + slot) * kTileM + t);
                        }
                        store_y(p.y, p.ydt, row, sum);
                    }
                    if (t == 0) p.row_counter[r] = 0;       // ready for the next call on this handle
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");   // is_last is rewritten by the next segment
            }
        }
    }
}

// Launch helper shared by the entry points: opts in to the large dynamic shared memory once per
// device, then launches P CTAs.
spdp_status launch_kernel(const Params& p, int num_ctas, cudaStream_t s) {
    constexpr size_t kSmemBytes = sizeof(Smem);
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(spmspv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(kSmemBytes)));
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    spmspv_kernel<<<num_ctas, kThreads, kSmemBytes, s>>>(p);
    SPDP_CUDA_TRY(cudaGetLastError());
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
// Everything spdp_spmspv keeps in handle-owned allocations (the CTA ranges, the per-row-tile
// tables, the arrival counters, the split-K partial sums) lives here instead, so the entry point
// below never allocates.  One copy per device that loads the library, held until exit.
constexpr int kNoAllocMaxCtas = 512;
constexpr int kNoAllocMaxRowTiles = 4096;          // M <= 1,048,576

struct NoAllocScratch {
    uint32_t cta_begin[kNoAllocMaxCtas + 1];
    int32_t row_first_cta[kNoAllocMaxRowTiles];
    int32_t row_nseg[kNoAllocMaxRowTiles];
    unsigned row_counter[kNoAllocMaxRowTiles];
    int status;
    float workspace[kNoAllocMaxCtas * 2 * kTileM];
};

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

// Fills the partition tables for P CTAs and zeroes what a call expects to start at zero (the
// array keeps whatever the previous call left).
__global__ void noalloc_setup_kernel(NoAllocScratch* sc, int64_t NGT, int64_t C, int R, int P) {
    for (int p = threadIdx.x; p <= P; p += blockDim.x)
        sc->cta_begin[p] = static_cast<uint32_t>((static_cast<unsigned long long>(NGT) * p) / P);
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        // the CTA whose range holds GTile s is ceil((s+1)*P/NGT) - 1
        const unsigned long long s0 = static_cast<unsigned long long>(r) * C, s1 = s0 + C - 1;
        const int first = static_cast<int>(((s0 + 1) * P + NGT - 1) / NGT) - 1;
        const int last = static_cast<int>(((s1 + 1) * P + NGT - 1) / NGT) - 1;
        sc->row_first_cta[r] = first;
        sc->row_nseg[r] = last - first + 1;
        sc->row_counter[r] = 0;
    }
    if (threadIdx.x == 0) sc->status = 0;
}

}  // namespace

int default_ctas_per_sm() { return kCtasPerSm; }

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
    p.cta_begin = h->cta_begin;
    p.row_first_cta = h->row_first_cta;
    p.row_nseg = h->row_nseg;
    p.workspace = h->workspace;
    p.row_counter = h->row_counter;
    p.status = h->status_word;
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
    if (R > kNoAllocMaxRowTiles || NGT >= (int64_t(1) << 31) / kTileK) return SPDP_ERR_UNSUPPORTED_SHAPE;
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
    noalloc_setup_kernel<<<1, 256, 0, s>>>(sc, NGT, C, static_cast<int>(R), P);
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
    p.cta_begin = sc->cta_begin;            // addresses inside the device array (no host dereference)
    p.row_first_cta = sc->row_first_cta;
    p.row_nseg = sc->row_nseg;
    p.workspace = sc->workspace;
    p.row_counter = sc->row_counter;
    p.status = &sc->status;
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
