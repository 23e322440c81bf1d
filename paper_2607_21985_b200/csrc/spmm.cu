// SPDP-SpMM for sm_100a (Sec. 4.3): Y[n] = W_sp * X[n] for N tokens on the Tiled-CBC matrix, static
// pruning only.  The paper's prefill kernel decodes a GTile with the same bitmap rule as the decode
// kernel, passes the decoded tile through shared memory to reach the tensor cores' operand layout
// (its "layout alignment" stage: TILE_K_PAD stride, ldmatrix.x4, mma.m16n8k16), and accumulates
// there.  On Blackwell the tensor cores read both operands straight from shared memory
// (tcgen05.mma) and accumulate in tensor memory, so the layout-alignment stage becomes the decode
// itself: W is given to the tensor cores M-major (rows contiguous), which is how a column tile
// lies in Tiled-CBC, so a lane that owns 8 consecutive rows of a column (one bitmap byte: its
// values are one contiguous run, rank = set bits before the byte, Sec. 4.2.1) writes exactly one
// 16-byte piece of the operand tile per column.  No registers hold accumulators, no ldmatrix pass.
//
// K is walked in blocks of kKB columns = 4 GTiles.  Warp roles (both kernels below):
//   * copy warp, one thread: everything that moves data.  The 4 GTiles of a K-block are consecutive in
//     storage order, so their Values are ONE contiguous span (TileOffset[g] .. TileOffset[g+4]), their
//     Bitmap words another, their ColInfo words a third: three bulk copies (cp.async.bulk) per K-block
//     bring the block as stored.  An X tile (kKB columns x tokens, 128-byte swizzle, zero beyond K
//     and N) is one tiled bulk-tensor copy.  All copies complete on shared-memory barriers.
//   * tensor-core warp, one thread: when a block's decoded tile and X tile are there it issues the
//     block's tcgen05.mma (K = 16 each) and commits them to the stage's barrier.
//   * 16 decode warps: warp w decodes columns w, w+16, w+32, w+48 of the block into the operand tile
//     and arrives on the stage's barriers.  They issue no copies and meet no CTA-wide barrier in the loop.
// Every wait is bounded; every copy writes only the shared memory of the CTA that issued it.
//
// Two kernels share this structure:
//   one::spmm_kernel   one CTA = one row tile (256 rows = two M = 128 accumulators) x 256 tokens.
//   pair::spmm_kernel  two CTAs on neighbouring SMs (a cluster of 2) = one row tile x 512 tokens:
//                      tcgen05.mma.cta_group::2 multiplies M = 256 (128 rows from each CTA's shared memory)
//                      by N = 256 (128 tokens from each CTA's shared memory) and leaves 128 rows x 256 fp32
//                      columns in each CTA's tensor memory; two such accumulators fill the 512 columns.  Each
//                      CTA decodes only ITS 128 rows of every column tile: half the decode per token.
// The launch picks the one with fewer rounds of CTAs x cost per K-block (small N: the first).
#include <cuda.h>

#include <algorithm>
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kWarps = 16;             // decode warps
constexpr int kKB = 64;                // columns per K-block: 4 GTiles, 4 tensor-core steps of K = 16 per accumulator
constexpr int kGTB = kKB / kTileK;     // GTiles per K-block
constexpr int kNI = 256;               // the N of the tensor-core instruction
constexpr int kTmemCols = 512;         // both kernels use all of tensor memory: two accumulators of 128 rows x kNI columns
// A (decoded W), M-major without swizzle: 16-byte piece = 8 consecutive rows of one column; the 8
// columns of a k-group are 16 bytes apart (a core matrix of 128 bytes), the 16 row chunks of a
// 128-row tile 144 bytes apart (128 + 16: the 16-byte pieces that the lanes of a quarter warp store for
// one column then fall into different banks), the k-groups 16 * 144 bytes apart.
constexpr int kAChunkStride = 144;                 // stride byte offset: next 8 rows
constexpr int kAKGroupStride = 16 * kAChunkStride; // leading byte offset: next 8 columns
constexpr int kATileBytes = (kKB / 8) * kAKGroupStride;    // 128 rows x kKB columns
// B (X tile), K-major with the 128-byte swizzle: a token's kKB columns are one 128-byte row, written by
// one tiled bulk-tensor copy per K-block; 8 tokens form a 1024-byte swizzle atom (the stride byte offset),
// and a tensor-core step of K = 16 starts 32 bytes further into the row.
constexpr int kBRowBytes = 2 * kKB;
constexpr int kBAtomBytes = 8 * kBRowBytes;
#ifndef SPDP_SPMM_WAIT_TRIES
#define SPDP_SPMM_WAIT_TRIES (1 << 22)
#endif
constexpr int kWaitTries = SPDP_SPMM_WAIT_TRIES;
constexpr int kCompValues = kKB * kTileM;          // the most values a K-block stores
static_assert(kBRowBytes == 128, "one X row of a K-block is one 128-byte swizzle row");
static_assert(kKB % 16 == 0 && kKB == 4 * kWarps, "a warp decodes 4 columns of a K-block, one per quarter of its scan");

struct Params {
    const uint32_t* tileoffset;
    const uint32_t* colinfo;
    const uint64_t* bitmap;
    const __half* values;
    int64_t N;
    void* Y;                // [N][ldy]
    int64_t ldy;
    int ydt;
    int M, K, C;
    int nblocks;            // token blocks: CTA (or CTA pair) = row tile * nblocks + token block
    // CTA-pair kernel only: pair i works on tile tile0 + i / kslices, on slice i % kslices of the tile's K-blocks; with
    // kslices > 1 it leaves fp32 partial sums in partial[i][token in tile][row in tile] instead of writing Y.
    int tile0, kslices;
    float* partial;
    int* status;
    int64_t values_len;
};

struct CompStage {                              // one K-block as stored
    alignas(128) unsigned short vals[kCompValues + 16];   // the values of its 4 GTiles, contiguous
    alignas(16) uint32_t bm[kKB][8];            // bitmaps
    alignas(16) uint32_t ci[kKB];               // ColInfo words
    uint32_t to[kGTB + 1];                      // TileOffset words of the block's GTiles (+ the next one)
};
static_assert(offsetof(CompStage, bm) % 16 == 0 && offsetof(CompStage, ci) % 16 == 0 && sizeof(CompStage) % 16 == 0,
              "bulk copies need 16-byte aligned destinations");

// Shared-memory operand descriptor of tcgen05.mma: start address, leading byte offset, stride byte
// offset (all in 16-byte units), descriptor version of this architecture, layout (bits 61-63: 0 = no
// swizzle, 2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo, uint32_t layout) {
    uint64_t d = (smem_addr & 0x3FFFFu) >> 4;
    d |= static_cast<uint64_t>(lbo >> 4) << 16;
    d |= static_cast<uint64_t>(sbo >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(layout) << 61;
    return d;
}
// Instruction descriptor: fp16 x fp16 -> fp32, A M-major (bit 15), B K-major, M rows, N = kNI.
template <int kM>
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 15) | (static_cast<uint32_t>(kNI >> 3) << 17) | (static_cast<uint32_t>(kM >> 4) << 24);
// D[tmem] (+)= A * B, one CTA (M = 128) or a CTA pair (M = 256).
__device__ __forceinline__ void mma_f16_one(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, bool accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kInstrDesc<128>), "r"(accumulate ? 1u : 0u) : "memory");
}
__device__ __forceinline__ void mma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, bool accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kInstrDesc<256>), "r"(accumulate ? 1u : 0u) : "memory");
}
__device__ __forceinline__ void barrier_init(unsigned long long* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool wait_parity(unsigned long long* bar, unsigned parity) {
    const uint32_t a = smem_u32(bar);
    {   // the phase is usually complete already: a test costs less than a wait that may suspend
        unsigned done;
        asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(a), "r"(parity) : "memory");
        if (done) return true;
    }
    for (int tries = 0; tries < kWaitTries; ++tries) {
        unsigned done;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(a), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void expect_bytes(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Arrives on the barrier at the same place in the shared memory of CTA `rank` of the pair.
__device__ __forceinline__ void arrive_at(unsigned long long* bar, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(bar)), "r"(rank));
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ void pair_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Bulk copy global -> shared (16-byte aligned, a multiple of 16 bytes), completing on a shared-memory barrier.
__device__ __forceinline__ void bulk_copy(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Tiled bulk-tensor copy of the box at (column k, token n) of the X tensor map.
__device__ __forceinline__ void tensor_copy(void* dst, const CUtensorMap* map, int k, int n, unsigned long long* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(k), "r"(n), "r"(smem_u32(bar)) : "memory");
}

// TileOffset words of K-block kb of row tile r: its GTiles and the one after (Sec. 4.1); a short last block
// repeats its end.
struct Offsets { uint32_t to[kGTB + 1]; };
__device__ __forceinline__ Offsets fetch_offsets(const Params& p, int r, int nkb, int kb) {
    Offsets o;
#pragma unroll
    for (int i = 0; i <= kGTB; ++i) o.to[i] = 0u;
    if (kb < nkb) {
        const int ngt = min(kGTB, p.C - kGTB * kb);
        const uint32_t* src = p.tileoffset + static_cast<int64_t>(r) * p.C + kGTB * kb;
#pragma unroll
        for (int i = 0; i <= kGTB; ++i) o.to[i] = __ldg(src + min(i, ngt));
    }
    return o;
}
// Starts the copies of the stored K-block kb of row tile r: Values, Bitmap and ColInfo of its GTiles, three
// contiguous spans (Sec. 4.1).  Returns false (and copies no values) if TileOffset is not what the format says.
__device__ __forceinline__ bool load_comp(const Params& p, int r, int kb, const Offsets& o, CompStage& cs,
                                          unsigned long long* bar) {
    const int ngt = min(kGTB, p.C - kGTB * kb);
    const int64_t g0 = static_cast<int64_t>(r) * p.C + kGTB * kb;
    uint32_t nvals = o.to[kGTB] - o.to[0];
    bool good = true;
    if (o.to[kGTB] < o.to[0] || nvals > static_cast<uint32_t>(kCompValues) || static_cast<int64_t>(o.to[kGTB]) > p.values_len) {
        atomicCAS(p.status, 0, SPDP_ERR_OVERFLOW);
        good = false;
        nvals = 0u;
    }
#pragma unroll
    for (int i = 0; i <= kGTB; ++i) cs.to[i] = nvals ? o.to[i] : 0u;
    expect_bytes(bar, 2u * nvals + static_cast<uint32_t>(ngt) * (kTileK * 32u + kTileK * 4u));
    if (nvals) bulk_copy(&cs.vals[0], p.values + o.to[0], 2u * nvals, bar);
    bulk_copy(&cs.bm[0][0], p.bitmap + g0 * kTileK * 4, static_cast<uint32_t>(ngt) * kTileK * 32u, bar);
    bulk_copy(&cs.ci[0], p.colinfo + g0 * kTileK, static_cast<uint32_t>(ngt) * kTileK * 4u, bar);
    return good;
}

// The walk over one bitmap byte (Sec. 4.2.1): `first` = shared-memory address of the byte's first value; a set
// bit takes the next value, a clear bit leaves a zero.  Returns the 8 rows as 8 fp16.
#define SPDP_WALK_ROW(R, BIT) \
    " lop3.or.b32 t|p, %4, " #BIT ", 0, 0xC0, 0;\n @p ld.shared.u16 v" #R ", [a];\n @p add.u32 a, a, 2;\n"
__device__ __forceinline__ uint4 walk_byte(unsigned bits, uint32_t first) {
    uint4 o;
    asm("{\n .reg .pred p;\n .reg .b16 v<8>;\n .reg .b32 t, a;\n mov.u32 a, %5;\n"
        " mov.b16 v0, 0;\n mov.b16 v1, 0;\n mov.b16 v2, 0;\n mov.b16 v3, 0;\n"
        " mov.b16 v4, 0;\n mov.b16 v5, 0;\n mov.b16 v6, 0;\n mov.b16 v7, 0;\n"
        SPDP_WALK_ROW(0, 1) SPDP_WALK_ROW(1, 2) SPDP_WALK_ROW(2, 4) SPDP_WALK_ROW(3, 8)
        SPDP_WALK_ROW(4, 16) SPDP_WALK_ROW(5, 32) SPDP_WALK_ROW(6, 64)
        " lop3.or.b32 t|p, %4, 128, 0, 0xC0, 0;\n @p ld.shared.u16 v7, [a];\n"
        " mov.b32 %0, {v0, v1};\n mov.b32 %1, {v2, v3};\n mov.b32 %2, {v4, v5};\n mov.b32 %3, {v6, v7};\n}"
        : "=r"(o.x), "=r"(o.y), "=r"(o.z), "=r"(o.w) : "r"(bits), "r"(first));
    return o;
}
#undef SPDP_WALK_ROW

// One scan for the warp's 4 columns (warp, warp + 16, +32, +48) of the K-block in `cs`: lane (q, w) = (lane / 8,
// lane % 8) counts bitmap word w of column q, and an 8-lane prefix sum gives the index, inside the stage, of the
// word's first value (the column's start = its GTile's TileOffset relative to the block's first + its ColInfo
// offset, Sec. 4.1).  `ngt` = GTiles the block really has; the columns of the others are empty.
__device__ __forceinline__ void scan_columns(const Params& p, const CompStage& cs, int ngt, int warp, int lane,
                                             unsigned& w8, unsigned& base_w) {
    const int q = lane >> 3, w = lane & 7;
    const int jq = warp + kWarps * q;
    unsigned start = 0u;
    w8 = 0u;
    if ((jq >> 4) < ngt) {
        const uint32_t ciw = cs.ci[jq];
        start = cs.to[jq >> 4] - cs.to[0] + (ciw >> 16);
        w8 = cs.bm[jq][w];
        if (!SPDP_CHECK(p.status, start, ciw & 0xFFFFu, cs.to[ngt] - cs.to[0], kSiteValuesSpan)) w8 = 0u;   // checked build only
    }
    const unsigned cnt = __popc(w8);
    unsigned inc = cnt;
    scan8_level<1>(inc);
    scan8_level<2>(inc);
    scan8_level<4>(inc);
    base_w = start + inc - cnt;
}

// Epilogue of both kernels: tensor-memory lanes [lane_base, +32) x columns [c_begin, c_end) -> Y rows `row`,
// tokens n0 + column.  A thread holds one row, 16 tokens at a time, so a warp's stores of one token are 32
// consecutive rows.
__device__ __forceinline__ void store_accumulators(const Params& p, uint32_t tmem, int lane_base, int c_begin, int c_end,
                                                   int64_t row, int64_t n0) {
    for (int c0 = c_begin; c0 < c_end; c0 += 16) {
        if (n0 + c0 >= p.N) break;                                          // warp-uniform
        uint32_t v[16];
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                       "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                     : "r"(tmem + (static_cast<uint32_t>(lane_base) << 16) + c0) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (row < p.M) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int64_t n = n0 + c0 + i;
                if (n < p.N) store_y(p.Y, p.ydt, n * p.ldy + row, __uint_as_float(v[i]));
            }
        }
    }
}

// The same for a slice of K: the accumulators go, as fp32, to dst[column * 256 + row] (row = my row inside the row tile).
__device__ __forceinline__ void store_partial(float* dst, uint32_t tmem, int lane_base, int c_begin, int c_end, int row,
                                              int valid_columns) {
    for (int c0 = c_begin; c0 < c_end; c0 += 16) {
        if (c0 >= valid_columns) break;                                     // warp-uniform
        uint32_t v[16];
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                       "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                     : "r"(tmem + (static_cast<uint32_t>(lane_base) << 16) + c0) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (c0 + i < valid_columns) dst[static_cast<size_t>(c0 + i) * kTileM + row] = __uint_as_float(v[i]);
    }
}

// ===================================================================================================
namespace one {     // one CTA = one row tile x 256 tokens

constexpr int kThreads = (kWarps + 2) * 32;   // decode warps + the tensor-core warp + the copy warp
constexpr int kNT = kNI;                      // tokens per CTA
constexpr int kStages = 2;
constexpr int kBBytes = kNT * kBRowBytes;

struct __align__(1024) Smem {
    unsigned char B[kStages][kBBytes];              // X tiles (each stage starts on a 1024-byte boundary: swizzle atoms)
    unsigned char A[kStages][2][kATileBytes];       // decoded W, two 128-row tiles per stage
    CompStage comp[kStages];
    alignas(8) unsigned long long mma_done[kStages];    // the tensor cores are done with A stage s and B stage s
    alignas(8) unsigned long long a_ready[kStages];     // the decode warps have written A stage s (and read comp stage s)
    alignas(8) unsigned long long x_full[kStages];      // the X tile of B stage s has arrived
    alignas(8) unsigned long long comp_full[kStages];   // the stored K-block of comp stage s has arrived
    uint32_t tmem_base;
    int abort;
};
constexpr size_t kSmemBytes = sizeof(Smem) + 1024;      // the dynamic shared memory is aligned by hand
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
static_assert(kBBytes % 1024 == 0, "every B stage on a swizzle-atom boundary");

// Decodes the warp's 4 columns into the operand tiles at `a_stage`: per column, a lane owns the 8 rows of bitmap
// byte `lane`, fetches its word and the index of the word's first value from the scan lane, adds the set bits
// below its byte (its rank, Sec. 4.2.1) and walks the byte.
__device__ __forceinline__ void decode_block(const Params& p, const CompStage& cs, int ngt, int warp, int lane,
                                             unsigned char* a_stage) {
    unsigned w8, base_w;
    scan_columns(p, cs, ngt, warp, lane, w8, base_w);
    const int sh = 8 * (lane & 3);
    const unsigned below = (1u << sh) - 1u;
    const uint32_t vals = smem_u32(&cs.vals[0]);
    uint4 piece[4];
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        const unsigned word = __shfl_sync(0xFFFFFFFFu, w8, 8 * qq + (lane >> 2));
        const unsigned base = __shfl_sync(0xFFFFFFFFu, base_w, 8 * qq + (lane >> 2));
        const unsigned bits = (word >> sh) & 0xFFu;
        piece[qq] = walk_byte(bits, vals + 2u * (base + __popc(word & below)));
    }
    // the stores come after all four walks, so that the walks' loads are free to overlap
    unsigned char* mine = a_stage + (lane >> 4) * kATileBytes + (lane & 15) * kAChunkStride;
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        const int j = warp + kWarps * qq;
        *reinterpret_cast<uint4*>(mine + (j >> 3) * kAKGroupStride + (j & 7) * 16) = piece[qq];
    }
}

__global__ void __launch_bounds__(kThreads, 1)
spmm_kernel(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap xmap) {
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int r = static_cast<int>(blockIdx.x / static_cast<unsigned>(p.nblocks));
    const int nb = static_cast<int>(blockIdx.x - static_cast<unsigned>(r) * static_cast<unsigned>(p.nblocks));
    const int64_t n0 = static_cast<int64_t>(nb) * kNT;

    // ---- set-up: the barriers, and tensor memory ----
    if (t == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
            barrier_init(&sm.mma_done[s], 1);
            barrier_init(&sm.a_ready[s], kWarps);
            barrier_init(&sm.x_full[s], 1);
            barrier_init(&sm.comp_full[s], 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        sm.abort = 0;
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sm.tmem_base)), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm.tmem_base;
    const int nkb = (p.C + kGTB - 1) / kGTB;
    // A wait that runs out (it never should) clears `ok`: the thread then stops waiting but keeps walking the
    // same barriers as the others, the status word gets SPDP_ERR_TIMEOUT and the outputs stay unwritten.
    bool ok = true;

    if (warp == kWarps) {
        // ================= tensor-core warp: one thread issues the K-blocks' products =================
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % kStages;
                const unsigned phase = (kb / kStages) & 1;
                if (ok) ok = wait_parity(&sm.a_ready[s], phase);         // the decoded W tile is in place
                if (ok) ok = wait_parity(&sm.x_full[s], phase);          // and so is the X tile
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t ad0 = operand_desc(smem_u32(&sm.A[s][0][0]), kAKGroupStride, kAChunkStride, 0u);
                const uint64_t bd0 = operand_desc(smem_u32(&sm.B[s][0]), 16, kBAtomBytes, 2u);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int kk = 0; kk < kKB / 16; ++kk)    // the start address is the descriptor's low field, in 16-byte units
                        mma_f16_one(tmem + h * kNI, ad0 + ((h * kATileBytes + kk * 2 * kAKGroupStride) >> 4), bd0 + ((kk * 32) >> 4),
                                    kb > 0 || kk > 0);
                }
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(smem_u32(&sm.mma_done[s])) : "memory");
            }
        }
        __syncwarp();           // the other lanes wait here, not on a barrier in shared memory
    } else if (warp == kWarps + 1) {
        // ================= copy warp: one thread moves the stored K-blocks and the X tiles =================
        if (lane == 0) {
            auto load_x = [&](int kb) {
                expect_bytes(&sm.x_full[kb % kStages], kBBytes);
                tensor_copy(&sm.B[kb % kStages][0], &xmap, kb * kKB, static_cast<int>(n0), &sm.x_full[kb % kStages]);
            };
            for (int kb = 0; kb < kStages && kb < nkb; ++kb) {
                ok = load_comp(p, r, kb, fetch_offsets(p, r, nkb, kb), sm.comp[kb % kStages], &sm.comp_full[kb % kStages]) && ok;
                load_x(kb);
            }
            Offsets next = fetch_offsets(p, r, nkb, kStages);
            for (int kb = 0; kb + kStages < nkb; ++kb) {
                const int s = kb % kStages;
                const unsigned phase = (kb / kStages) & 1;
                // the stored block kb + kStages goes where block kb was decoded from, once every decode warp is done with it
                if (ok) ok = wait_parity(&sm.a_ready[s], phase);
                ok = load_comp(p, r, kb + kStages, next, sm.comp[s], &sm.comp_full[s]) && ok;
                next = fetch_offsets(p, r, nkb, kb + kStages + 1);
                // the X tile of block kb + kStages goes where block kb multiplies from, once that work is complete
                if (ok) ok = wait_parity(&sm.mma_done[s], phase);
                load_x(kb + kStages);
            }
        }
        __syncwarp();
    } else {
        // ================= decode warps =================
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % kStages;
            const unsigned phase = (kb / kStages) & 1;
            if (ok) ok = wait_parity(&sm.comp_full[s], phase);                           // the stored block has arrived
            if (kb >= kStages && ok) ok = wait_parity(&sm.mma_done[s], phase ^ 1u);     // the tensor cores are done with this A stage
            decode_block(p, sm.comp[s], min(kGTB, p.C - kGTB * kb), warp, lane, &sm.A[s][0][0]);
            // the operand tile was written through the generic proxy; the tensor cores read through the async proxy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) arrive(&sm.a_ready[s]);
        }
    }
    // the last blocks' tensor-core work
    for (int kb = (nkb > kStages ? nkb - kStages : 0); ok && kb < nkb; ++kb)
        ok = wait_parity(&sm.mma_done[kb % kStages], (kb / kStages) & 1);
    if (!ok) {
        sm.abort = 1;
        if (lane == 0) atomicCAS(p.status, 0, SPDP_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    __syncthreads();

    // ---- epilogue.  Warp w reads lanes 32*(w%4).. of accumulator (w/4)%2, token columns [(w/8)*128, +128) ----
    if (!sm.abort && warp < kWarps) {
        const int half = (warp >> 2) & 1, lane_base = 32 * (warp & 3), cbase = (warp >> 3) * (kNT / 2);
        store_accumulators(p, tmem + half * kNI, lane_base, cbase, cbase + kNT / 2,
                           static_cast<int64_t>(r) * kTileM + half * 128 + lane_base + lane, n0);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
}

}  // namespace one

// ===================================================================================================
namespace pair {    // two CTAs (a cluster of 2) = one row tile x 512 tokens

constexpr int kThreads = (kWarps + 3) * 32;   // decode warps + the tensor-core warp, the copy warp and the relay warp
constexpr int kNTiles = 2;                    // accumulators per CTA
constexpr int kNT = kNTiles * kNI;            // tokens per CTA pair
constexpr int kStages = 3;                    // operand tiles (decoded W, X) in flight
constexpr int kCStages = 2;                   // stored K-blocks in flight
constexpr int kBTileBytes = (kNI / 2) * kBRowBytes;    // this CTA's 128 tokens of one X tile
constexpr int kBBytes = kNTiles * kBTileBytes;
static_assert(kNTiles * kNI == kTmemCols, "the accumulators fill tensor memory");

struct __align__(1024) Smem {
    unsigned char B[kStages][kBBytes];              // my halves of the X tiles (each on a 1024-byte boundary: swizzle atoms)
    unsigned char A[kStages][kATileBytes];          // decoded W: my 128 rows
    CompStage comp[kCStages];
    alignas(8) unsigned long long mma_done[kStages];    // the tensor cores are done with A stage s and B stage s (both CTAs)
    alignas(8) unsigned long long a_ready[kStages];     // my decode warps have written A stage s (and read the stored block)
    alignas(8) unsigned long long ready[kStages];       // A stage s is written and my X tiles of B stage s have arrived
                                                        // (first CTA: and the second CTA says the same of its own)
    alignas(8) unsigned long long comp_full[kCStages];  // the stored K-block of comp stage s has arrived
    uint32_t tmem_base;
    int abort;
};
constexpr size_t kSmemBytes = sizeof(Smem) + 1024;      // the dynamic shared memory is aligned by hand
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
static_assert(kBTileBytes % 1024 == 0, "every X tile on a swizzle-atom boundary");

// Decodes my 128 rows (half `c` of the row tile) of the warp's 4 columns into the operand tile `a_tile`, in two
// passes: in a pass the lower half warp takes one column, the upper the next; a lane owns the 8 rows of bitmap
// byte 16 c + lane % 16, fetches its word and the index of the word's first value from the scan lane, adds the
// set bits below its byte (its rank, Sec. 4.2.1) and walks the byte.
__device__ __forceinline__ void decode_block(const Params& p, const CompStage& cs, int ngt, int c, int warp, int lane,
                                             unsigned char* a_tile) {
    unsigned w8, base_w;
    scan_columns(p, cs, ngt, warp, lane, w8, base_w);
    const int sh = 8 * (lane & 3);
    const unsigned below = (1u << sh) - 1u;
    const uint32_t vals = smem_u32(&cs.vals[0]);
    const int hw = lane >> 4, l16 = lane & 15;
    uint4 piece[2];
#pragma unroll
    for (int ps = 0; ps < 2; ++ps) {
        const int src = 8 * (2 * ps + hw) + 4 * c + (l16 >> 2);       // the scan lane of (my column, my word)
        const unsigned word = __shfl_sync(0xFFFFFFFFu, w8, src);
        const unsigned base = __shfl_sync(0xFFFFFFFFu, base_w, src);
        const unsigned bits = (word >> sh) & 0xFFu;
        piece[ps] = walk_byte(bits, vals + 2u * (base + __popc(word & below)));
    }
    // the stores come after both walks, so that the walks' loads are free to overlap
#pragma unroll
    for (int ps = 0; ps < 2; ++ps) {
        const int j = warp + kWarps * (2 * ps + hw);
        *reinterpret_cast<uint4*>(a_tile + l16 * kAChunkStride + (j >> 3) * kAKGroupStride + (j & 7) * 16) = piece[ps];
    }
}

__global__ void __launch_bounds__(kThreads, 1)
spmm_kernel(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap xmap) {
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int c = static_cast<int>(blockIdx.x & 1u);                  // my rank in the pair = my half of the row tile
    const unsigned pr = blockIdx.x >> 1;
    const unsigned tile = static_cast<unsigned>(p.tile0) + pr / static_cast<unsigned>(p.kslices);
    const int slice = static_cast<int>(pr % static_cast<unsigned>(p.kslices));
    const int r = static_cast<int>(tile / static_cast<unsigned>(p.nblocks));
    const int nb = static_cast<int>(tile - static_cast<unsigned>(r) * static_cast<unsigned>(p.nblocks));
    const int64_t n0 = static_cast<int64_t>(nb) * kNT;
    const int ntiles = (p.N - n0 > kNI) ? 2 : 1;                      // accumulators in use

    // ---- set-up: the barriers, and tensor memory (both CTAs of the pair allocate together) ----
    if (t == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
            barrier_init(&sm.mma_done[s], 1);
            barrier_init(&sm.a_ready[s], kWarps);
            // arrivals on ready[]: my decode warps, my copy thread (with the X tiles' bytes), in the first CTA the second CTA
            barrier_init(&sm.ready[s], kWarps + 1 + (c == 0 ? 1 : 0));
        }
#pragma unroll
        for (int s = 0; s < kCStages; ++s) barrier_init(&sm.comp_full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        sm.abort = 0;
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sm.tmem_base)), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    pair_sync();                       // both CTAs' barriers and tensor memory exist before either reaches into the other
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm.tmem_base;
    // my K-blocks: slice `slice` of the tile's nkb_all; kb below counts from the slice's first block kb0
    const int nkb_all = (p.C + kGTB - 1) / kGTB;
    const int kb0 = static_cast<int>(static_cast<int64_t>(nkb_all) * slice / p.kslices);
    const int nkb = static_cast<int>(static_cast<int64_t>(nkb_all) * (slice + 1) / p.kslices) - kb0;
    // A wait that runs out (it never should) clears `ok`: the thread then stops waiting but keeps walking the
    // same barriers as the others, the status word gets SPDP_ERR_TIMEOUT and the outputs stay unwritten.
    bool ok = true;

    if (warp == kWarps) {
        if (lane == 0 && c == 0) {
            // ================= tensor-core thread (first CTA): issues the K-blocks' products for the pair =================
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % kStages;
                if (ok) ok = wait_parity(&sm.ready[s], (kb / kStages) & 1);      // both CTAs' decoded W tiles and X tiles are in place
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t ad0 = operand_desc(smem_u32(&sm.A[s][0]), kAKGroupStride, kAChunkStride, 0u);
                const uint64_t bd0 = operand_desc(smem_u32(&sm.B[s][0]), 16, kBAtomBytes, 2u);
                for (int i = 0; i < ntiles; ++i) {
#pragma unroll
                    for (int kk = 0; kk < kKB / 16; ++kk)    // the start address is the descriptor's low field, in 16-byte units
                        mma_f16_pair(tmem + i * kNI, ad0 + ((kk * 2 * kAKGroupStride) >> 4), bd0 + ((i * kBTileBytes + kk * 32) >> 4),
                                     kb > 0 || kk > 0);
                }
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(smem_u32(&sm.mma_done[s])) : "memory");
            }
        } else if (lane == 0) {
            // ================= second CTA: tell the first when my tiles of a block are ready =================
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % kStages;
                if (ok) ok = wait_parity(&sm.ready[s], (kb / kStages) & 1);
                arrive_at(&sm.ready[s], 0u);
            }
        }
        __syncwarp();           // the other lanes wait here, not on a barrier in shared memory
    } else if (warp == kWarps + 1) {
        // ================= copy warp: one thread moves the stored K-blocks and my halves of the X tiles =================
        if (lane == 0) {
            // my 128 tokens of the X tiles of K-block kb: one tiled bulk-tensor copy per tile
            auto load_x = [&](int kb) {
                unsigned long long* bar = &sm.ready[kb % kStages];
                expect_bytes(bar, static_cast<uint32_t>(ntiles) * kBTileBytes);
                for (int i = 0; i < ntiles; ++i)
                    tensor_copy(&sm.B[kb % kStages][i * kBTileBytes], &xmap, (kb0 + kb) * kKB, static_cast<int>(n0) + i * kNI + c * (kNI / 2), bar);
            };
            for (int kb = 0; kb < kCStages && kb < nkb; ++kb)
                ok = load_comp(p, r, kb0 + kb, fetch_offsets(p, r, nkb_all, kb0 + kb), sm.comp[kb % kCStages], &sm.comp_full[kb % kCStages]) && ok;
            for (int kb = 0; kb < kStages && kb < nkb; ++kb) load_x(kb);
            Offsets next = fetch_offsets(p, r, nkb_all, kb0 + kCStages);
            for (int kb = 0; kb < nkb; ++kb) {
                // the stored block kb + kCStages goes where block kb was decoded from, once my decode warps are done with it
                if (kb + kCStages < nkb) {
                    if (ok) ok = wait_parity(&sm.a_ready[kb % kStages], (kb / kStages) & 1);
                    ok = load_comp(p, r, kb0 + kb + kCStages, next, sm.comp[kb % kCStages], &sm.comp_full[kb % kCStages]) && ok;
                    next = fetch_offsets(p, r, nkb_all, kb0 + kb + kCStages + 1);
                }
                // my X tiles of block kb + 1 go where block kb + 1 - kStages multiplied from, once that work is complete
                const int kx = kb + 1;
                if (kx >= kStages && kx < nkb) {
                    if (ok) ok = wait_parity(&sm.mma_done[kx % kStages], ((kx / kStages) - 1) & 1);
                    load_x(kx);
                }
            }
        }
        __syncwarp();
    } else if (warp == kWarps + 2) {
        // ================= relay warp (first CTA): the tensor cores' completion arrives on the first CTA's barrier;
        // one thread passes it on to the second CTA's =================
        if (lane == 0 && c == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % kStages;
                if (ok) ok = wait_parity(&sm.mma_done[s], (kb / kStages) & 1);
                arrive_at(&sm.mma_done[s], 1u);
            }
        }
        __syncwarp();
    } else {
        // ================= decode warps =================
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % kStages;
            const unsigned phase = (kb / kStages) & 1;
            if (ok) ok = wait_parity(&sm.comp_full[kb % kCStages], (kb / kCStages) & 1);    // the stored block has arrived
            if (kb >= kStages && ok) ok = wait_parity(&sm.mma_done[s], phase ^ 1u);         // the tensor cores are done with this A stage
            decode_block(p, sm.comp[kb % kCStages], min(kGTB, p.C - kGTB * (kb0 + kb)), c, warp, lane, &sm.A[s][0]);
            // the operand tile was written through the generic proxy; the tensor cores read through the async proxy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                arrive(&sm.a_ready[s]);
                arrive(&sm.ready[s]);
            }
        }
    }
    // the last blocks' tensor-core work
    for (int kb = (nkb > kStages ? nkb - kStages : 0); ok && kb < nkb; ++kb)
        ok = wait_parity(&sm.mma_done[kb % kStages], (kb / kStages) & 1);
    if (!ok) {
        sm.abort = 1;
        if (lane == 0) atomicCAS(p.status, 0, SPDP_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    __syncthreads();

    // ---- epilogue.  Warp w reads lanes 32*(w%4).. (my rows 32*(w%4)..), token columns [(w/4)*128, +128) of the 512 ----
    if (!sm.abort && warp < kWarps) {
        const int lane_base = 32 * (warp & 3), cbase = (warp >> 2) * (kNT / 4);
        if (p.partial == nullptr)
            store_accumulators(p, tmem, lane_base, cbase, cbase + kNT / 4,
                               static_cast<int64_t>(r) * kTileM + c * 128 + lane_base + lane, n0);
        else
            store_partial(p.partial + static_cast<size_t>(pr) * kNT * kTileM, tmem, lane_base, cbase, cbase + kNT / 4,
                          c * 128 + lane_base + lane, static_cast<int>(min(static_cast<int64_t>(kNT), p.N - n0)));
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    pair_sync();                       // neither CTA leaves, or frees tensor memory, while the other may still reach into it
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
}

// Adds the K-slices of the tiles that were cut along K, in slice order, and writes their part of Y.
__global__ void reduce_slices_kernel(const Params p, int tiles) {
    const int64_t total = static_cast<int64_t>(tiles) * kNT * kTileM;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int row_in = static_cast<int>(i % kTileM);
        const int col = static_cast<int>((i / kTileM) % kNT);
        const int tt = static_cast<int>(i / (static_cast<int64_t>(kTileM) * kNT));
        const unsigned tile = static_cast<unsigned>(p.tile0 + tt);
        const int r = static_cast<int>(tile / static_cast<unsigned>(p.nblocks));
        const int nb = static_cast<int>(tile - static_cast<unsigned>(r) * static_cast<unsigned>(p.nblocks));
        const int64_t n = static_cast<int64_t>(nb) * kNT + col, row = static_cast<int64_t>(r) * kTileM + row_in;
        if (n >= p.N || row >= p.M) continue;
        const float* src = p.partial + (static_cast<size_t>(tt) * p.kslices * kNT + col) * kTileM + row_in;
        float sum = 0.f;
        for (int sl = 0; sl < p.kslices; ++sl) sum += src[static_cast<size_t>(sl) * kNT * kTileM];
        store_y(p.Y, p.ydt, n * p.ldy + row, sum);
    }
}

}  // namespace pair

}  // namespace

spdp_status configure_spmm_kernel() {
    static std::mutex mu;
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SPDP_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(one::spmm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(one::kSmemBytes)));
        SPDP_CUDA_TRY(cudaFuncSetAttribute(pair::spmm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(pair::kSmemBytes)));
        configured[dev] = true;
    }
    return SPDP_OK;
}

namespace {
// The driver's tensor-map encoder, looked up once through the runtime (the library does not link libcuda).
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}
// X as a 2-D tensor [N][K] (row stride ldx): boxes of kKB columns x `box_tokens` tokens, 128-byte swizzle, zero fill.
spdp_status encode_x(CUtensorMap* map, const __half* X, int64_t N, int64_t K, int64_t ldx, int box_tokens) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return SPDP_ERR_CUDA;
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(N)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(ldx) * sizeof(__half)};
    const cuuint32_t box[2] = {kKB, static_cast<cuuint32_t>(box_tokens)};
    const cuuint32_t estride[2] = {1, 1};
    if (encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(X), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SPDP_ERR_INVALID_ARG;
    return SPDP_OK;
}
}  // namespace

spdp_status launch_spmm(const spdp_matrix* h, const __half* X, int64_t N, int64_t ldx, void* Y, int64_t ldy, int ydt,
                        cudaStream_t s) {
    Params p;
    p.tileoffset = h->tileoffset;
    p.colinfo = h->colinfo;
    p.bitmap = h->bitmap;
    p.values = h->values;
    p.N = N;
    p.Y = Y;
    p.ldy = ldy;
    p.ydt = ydt;
    p.M = static_cast<int>(h->M);
    p.K = static_cast<int>(h->K);
    p.C = static_cast<int>(h->C);
    p.status = h->status_word;
    p.values_len = h->values_len;
    p.tile0 = 0;
    p.kslices = 1;
    p.partial = nullptr;
    // Which kernel: rounds of CTAs over the SMs x the measured cost of a K-block (a pair's CTA decodes half as much:
    // 3 : 4).  A last round of the pair kernel that would hold at most half the pairs is cut along K instead: its
    // tiles are spread over all pairs as K-slices that leave fp32 partial sums in scratch memory, and a small
    // kernel adds the slices in order (so the result does not depend on timing).
    const int64_t sms = h->sm_count > 0 ? h->sm_count : 1;
    const int64_t slots = sms / 2 > 0 ? sms / 2 : 1;                         // pairs resident at once
    const int64_t ctas_one = h->R * ((N + one::kNT - 1) / one::kNT);
    const int64_t tiles = h->R * ((N + pair::kNT - 1) / pair::kNT);         // pair tiles
    const int64_t nkb = (h->C + kGTB - 1) / kGTB;
    const int64_t full = (tiles / slots) * slots, rest = tiles - full;
    int64_t slices = 1;
    if (full > 0 && rest > 0 && 2 * rest <= slots) slices = std::min<int64_t>(std::min<int64_t>(slots / rest, nkb), 64);
    const double cost_pair = 3.0 * (static_cast<double>(full / slots) + (rest > 0 ? 1.0 / static_cast<double>(slices) : 0.0) +
                                    (slices > 1 ? 0.1 : 0.0));
    const double cost_one = 4.0 * static_cast<double>((ctas_one + sms - 1) / sms);
    const bool use_pair = cost_pair < cost_one;
    if (std::max(ctas_one, 2 * tiles * slices) >= (int64_t(1) << 31)) return SPDP_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap xmap;
    spdp_status st = encode_x(&xmap, X, N, h->K, ldx, use_pair ? kNI / 2 : one::kNT);
    if (st != SPDP_OK) return st;
    if (!use_pair) {
        p.nblocks = static_cast<int>((N + one::kNT - 1) / one::kNT);
        one::spmm_kernel<<<static_cast<unsigned>(ctas_one), one::kThreads, one::kSmemBytes, s>>>(p, xmap);
        SPDP_CUDA_TRY(cudaGetLastError());
        return SPDP_OK;
    }
    p.nblocks = static_cast<int>((N + pair::kNT - 1) / pair::kNT);
    auto launch_pairs = [&](int64_t pairs) -> spdp_status {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs));
        cfg.blockDim = dim3(pair::kThreads);
        cfg.dynamicSmemBytes = pair::kSmemBytes;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        SPDP_CUDA_TRY(cudaLaunchKernelEx(&cfg, pair::spmm_kernel, p, xmap));
        return SPDP_OK;
    };
    if (slices == 1) return launch_pairs(tiles);
    // whole tiles first, then the last tiles cut along K, then the sum of their slices
    st = launch_pairs(full);
    if (st != SPDP_OK) return st;
    float* scratch = nullptr;
    const size_t scratch_bytes = static_cast<size_t>(rest * slices) * pair::kNT * kTileM * sizeof(float);
    SPDP_CUDA_TRY(cudaMallocAsync(reinterpret_cast<void**>(&scratch), scratch_bytes, s));     // stream-ordered, from the device's pool
    p.tile0 = static_cast<int>(full);
    p.kslices = static_cast<int>(slices);
    p.partial = scratch;
    st = launch_pairs(rest * slices);
    if (st == SPDP_OK) {
        const int64_t elems = rest * pair::kNT * kTileM;
        pair::reduce_slices_kernel<<<static_cast<unsigned>(std::min<int64_t>((elems + 255) / 256, 4096)), 256, 0, s>>>(
            p, static_cast<int>(rest));
        if (cudaGetLastError() != cudaSuccess) st = SPDP_ERR_CUDA;
    }
    cudaFreeAsync(scratch, s);
    return st;
}

}  // namespace spdp
