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
// One CTA = one row tile (256 rows = two M = 128 accumulators) x kNT tokens (all 512 columns of
// tensor memory), walking K in blocks of kKB columns = 4 GTiles.  Warp roles:
//   * copy warp, one thread: everything that moves data.  The 4 GTiles of a K-block are consecutive in
//     storage order, so their Values are ONE contiguous span (TileOffset[g] .. TileOffset[g+4]), their
//     Bitmap words another, their ColInfo words a third: three bulk copies (cp.async.bulk) per K-block
//     bring the block as stored.  The X tile (kKB columns x kNT tokens, 128-byte swizzle, zero beyond K
//     and N) is one tiled bulk-tensor copy.  All copies complete on shared-memory barriers.
//   * tensor-core warp, one thread: when a block's decoded tile and X tile are there it issues
//     2 x 4 tcgen05.mma (M 128, N kNT, K 16) and commits them to the stage's barrier.
//   * 16 decode warps: warp w decodes columns w, w+16, w+32, w+48 of the block into the operand tile
//     and arrives on the stage's barrier.  They issue no copies and meet no CTA-wide barrier in the loop.
// Two stages of everything; every wait is bounded.
#include <cuda.h>

#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kWarps = 16;             // decode warps; lane l owns rows 8l .. 8l+7 of the warp's columns
constexpr int kThreads = (kWarps + 2) * 32;   // + the tensor-core warp and the copy warp (one thread each)
constexpr int kKB = 64;                // columns per K-block: 4 GTiles, 4 tensor-core steps of K = 16 per accumulator
constexpr int kGTB = kKB / kTileK;     // GTiles per K-block
constexpr int kNT = 256;               // tokens per CTA (the N of the tensor-core instruction)
constexpr int kTmemCols = 2 * kNT;     // two accumulators of 128 rows x kNT fp32 columns
constexpr int kStages = 2;
// A (decoded W), M-major without swizzle: 16-byte piece = 8 consecutive rows of one column; the 8
// columns of a k-group are 16 bytes apart (a core matrix of 128 bytes), the 16 row chunks of a
// 128-row half 144 bytes apart (128 + 16: the 16-byte pieces that the lanes of a quarter warp store for
// one column then fall into different banks), the k-groups 16 * 144 bytes apart.
constexpr int kAChunkStride = 144;                 // stride byte offset: next 8 rows
constexpr int kAKGroupStride = 16 * kAChunkStride; // leading byte offset: next 8 columns
constexpr int kAHalfBytes = (kKB / 8) * kAKGroupStride;
// B (X tile), K-major with the 128-byte swizzle: a token's kKB columns are one 128-byte row, written by
// one tiled bulk-tensor copy per K-block; 8 tokens form a 1024-byte swizzle atom (the stride byte offset),
// and a tensor-core step of K = 16 starts 32 bytes further into the row.
constexpr int kBRowBytes = 2 * kKB;
constexpr int kBAtomBytes = 8 * kBRowBytes;
constexpr int kBBytes = kNT * kBRowBytes;
constexpr int kWaitTries = 1 << 22;
constexpr int kCompValues = kKB * kTileM;          // the most values a K-block stores
static_assert(kBRowBytes == 128, "one X row of a K-block is one 128-byte swizzle row");
static_assert(kTmemCols == 512, "the CTA owns all of tensor memory");
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
    int nblocks;            // ceil(N / kNT): CTA = row tile * nblocks + token block
    int* status;
    int64_t values_len;
};

struct CompStage {                              // one K-block as stored
    alignas(128) unsigned short vals[kCompValues + 16];   // the values of its 4 GTiles, contiguous (+ slack: the walk
                                                          // may look one value past a run)
    alignas(16) uint32_t bm[kKB][8];            // bitmaps
    alignas(16) uint32_t ci[kKB];               // ColInfo words
    uint32_t to[kGTB + 1];                      // TileOffset words of the block's GTiles (+ the next one)
};
struct __align__(1024) Smem {
    unsigned char B[kStages][kBBytes];          // X tiles (each stage starts on a 1024-byte boundary: swizzle atoms)
    unsigned char A[kStages][2][kAHalfBytes];   // decoded W, two 128-row halves per stage
    CompStage comp[kStages];
    alignas(8) unsigned long long mma_done[kStages];    // the tensor cores are done with A stage s and the B stage used with it
    alignas(8) unsigned long long a_ready[kStages];     // the kWarps decode warps have written A stage s (and read comp stage s)
    alignas(8) unsigned long long x_full[kStages];      // the X tile of B stage s has arrived
    alignas(8) unsigned long long comp_full[kStages];   // the stored K-block of comp stage s has arrived
    uint32_t tmem_base;
    int abort;
};
constexpr size_t kSmemBytes = sizeof(Smem) + 1024;      // the dynamic shared memory is aligned by hand
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
static_assert(kBBytes % 1024 == 0, "every B stage on a swizzle-atom boundary");
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
// Instruction descriptor: fp16 x fp16 -> fp32, A M-major (bit 15), B K-major, M = 128, N = kNT.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 15) | (static_cast<uint32_t>(kNT >> 3) << 17) |
                                (static_cast<uint32_t>(128 >> 4) << 24);

__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, bool accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kInstrDesc), "r"(accumulate ? 1u : 0u) : "memory");
}
__device__ __forceinline__ bool wait_parity(unsigned long long* bar, unsigned parity) {
    const uint32_t a = smem_u32(bar);
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
// Bulk copy global -> shared (16-byte aligned, a multiple of 16 bytes), completing on a shared-memory barrier.
__device__ __forceinline__ void bulk_copy(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// The walk over one bitmap byte (Sec. 4.2.1): `a` = shared-memory address of the byte's first value; a set bit
// takes the next value, a clear bit leaves a zero.  Returns the 8 rows as 8 fp16.
#define SPDP_WALK_ROW(R, BIT) \
    " lop3.or.b32 t|p, %4, " #BIT ", 0, 0xC0, 0;\n @p ld.shared.u16 v" #R ", [a];\n @p add.u32 a, a, 2;\n"
__device__ __forceinline__ uint4 walk_byte(unsigned bits, uint32_t first) {
    uint4 o;
    asm volatile(
        "{\n .reg .pred p;\n .reg .b16 v<8>;\n .reg .b32 t, a;\n mov.u32 a, %5;\n"
        " mov.b16 v0, 0;\n mov.b16 v1, 0;\n mov.b16 v2, 0;\n mov.b16 v3, 0;\n"
        " mov.b16 v4, 0;\n mov.b16 v5, 0;\n mov.b16 v6, 0;\n mov.b16 v7, 0;\n"
        SPDP_WALK_ROW(0, 1) SPDP_WALK_ROW(1, 2) SPDP_WALK_ROW(2, 4) SPDP_WALK_ROW(3, 8)
        SPDP_WALK_ROW(4, 16) SPDP_WALK_ROW(5, 32) SPDP_WALK_ROW(6, 64)
        " lop3.or.b32 t|p, %4, 128, 0, 0xC0, 0;\n @p ld.shared.u16 v7, [a];\n"
        " mov.b32 %0, {v0, v1};\n mov.b32 %1, {v2, v3};\n mov.b32 %2, {v4, v5};\n mov.b32 %3, {v6, v7};\n}"
        : "=r"(o.x), "=r"(o.y), "=r"(o.z), "=r"(o.w) : "r"(bits), "r"(first) : "memory");
    return o;
}
#undef SPDP_WALK_ROW

// Decodes the warp's 4 columns (warp, warp + 16, +32, +48) of the K-block in comp stage `cs` into the operand
// tile at `a_stage` (the lane's row chunk).  One scan serves the 4 columns: lane (q, w) = (lane / 8, lane % 8)
// counts bitmap word w of column q and an 8-lane prefix sum gives the index of the word's first value inside
// the stage (the column's start = its GTile's TileOffset relative to the block's first + its ColInfo offset,
// Sec. 4.1); then, per column, a lane fetches its word and that index from the scan lane, adds the set bits
// below its byte (its rank, Sec. 4.2.1) and walks the byte.  `ngt` = GTiles the block really has.
__device__ __forceinline__ void decode_block(const Params& p, const CompStage& cs, int ngt, int warp, int lane,
                                             unsigned char* a_stage) {
    const int q = lane >> 3, w = lane & 7;
    const int jq = warp + kWarps * q;
    unsigned w8 = 0u, start = 0u;
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
    const unsigned base_w = start + inc - cnt;
    const int sh = 8 * (lane & 3);
    const unsigned below = (1u << sh) - 1u;
    const uint32_t vals = smem_u32(&cs.vals[0]);
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        const int j = warp + kWarps * qq;
        const unsigned word = __shfl_sync(0xFFFFFFFFu, w8, 8 * qq + (lane >> 2));
        const unsigned base = __shfl_sync(0xFFFFFFFFu, base_w, 8 * qq + (lane >> 2));
        const unsigned bits = (word >> sh) & 0xFFu;
        const uint4 piece = walk_byte(bits, vals + 2u * (base + __popc(word & below)));
        *reinterpret_cast<uint4*>(a_stage + (j >> 3) * kAKGroupStride + (j & 7) * 16) = piece;
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
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.mma_done[s])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&sm.a_ready[s])), "n"(kWarps) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.x_full[s])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.comp_full[s])) : "memory");
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
                        mma_f16(tmem + h * kNT, ad0 + ((h * kAHalfBytes + kk * 2 * kAKGroupStride) >> 4), bd0 + ((kk * 32) >> 4),
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
            struct Offsets { uint32_t to[kGTB + 1]; };
            // TileOffset words of K-block kb: its GTiles and the one after (Sec. 4.1); a short last block repeats its end
            auto fetch_offsets = [&](int kb) -> Offsets {
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
            };
            // the stored K-block kb: Values, Bitmap and ColInfo of its GTiles, three contiguous spans (Sec. 4.1)
            auto load_comp = [&](int kb, const Offsets& o) {
                CompStage& cs = sm.comp[kb % kStages];
                unsigned long long* bar = &sm.comp_full[kb % kStages];
                const int ngt = min(kGTB, p.C - kGTB * kb);
                const int64_t g0 = static_cast<int64_t>(r) * p.C + kGTB * kb;
                uint32_t nvals = o.to[kGTB] - o.to[0];
                if (o.to[kGTB] < o.to[0] || nvals > static_cast<uint32_t>(kCompValues) ||
                    static_cast<int64_t>(o.to[kGTB]) > p.values_len) {       // TileOffset is not what the format says
                    atomicCAS(p.status, 0, SPDP_ERR_OVERFLOW);
                    ok = false;
                    nvals = 0u;
                }
#pragma unroll
                for (int i = 0; i <= kGTB; ++i) cs.to[i] = nvals ? o.to[i] : 0u;
                expect_bytes(bar, 2u * nvals + static_cast<uint32_t>(ngt) * (kTileK * 32u + kTileK * 4u));
                if (nvals) bulk_copy(&cs.vals[0], p.values + o.to[0], 2u * nvals, bar);
                bulk_copy(&cs.bm[0][0], p.bitmap + g0 * kTileK * 4, static_cast<uint32_t>(ngt) * kTileK * 32u, bar);
                bulk_copy(&cs.ci[0], p.colinfo + g0 * kTileK, static_cast<uint32_t>(ngt) * kTileK * 4u, bar);
            };
            // the X tile of K-block kb: one tiled bulk-tensor copy (kKB columns x kNT tokens, zero beyond K and N)
            auto load_x = [&](int kb) {
                unsigned long long* bar = &sm.x_full[kb % kStages];
                expect_bytes(bar, kBBytes);
                asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                             ::"r"(smem_u32(&sm.B[kb % kStages][0])), "l"(reinterpret_cast<uint64_t>(&xmap)),
                               "r"(kb * kKB), "r"(static_cast<int>(n0)), "r"(smem_u32(bar)) : "memory");
            };
            for (int kb = 0; kb < kStages && kb < nkb; ++kb) {
                load_comp(kb, fetch_offsets(kb));
                load_x(kb);
            }
            Offsets next = fetch_offsets(kStages);
            for (int kb = 0; kb + kStages < nkb; ++kb) {
                const int s = kb % kStages;
                const unsigned phase = (kb / kStages) & 1;
                // the stored block kb + kStages goes where block kb was decoded from, once every decode warp is done with it
                if (ok) ok = wait_parity(&sm.a_ready[s], phase);
                load_comp(kb + kStages, next);
                next = fetch_offsets(kb + kStages + 1);
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
            decode_block(p, sm.comp[s], min(kGTB, p.C - kGTB * kb), warp, lane,
                         &sm.A[s][lane >> 4][0] + (lane & 15) * kAChunkStride);
            // the operand tile was written through the generic proxy; the tensor cores read through the async proxy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&sm.a_ready[s])) : "memory");
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

    // ---- epilogue: tensor memory -> registers -> Y.  Warp w reads lanes 32*(w%4).. of accumulator (w/4)%2,
    // token columns [(w/8)*kNT/2, +kNT/2); a thread holds one row, 16 tokens at a time, so a warp's stores of
    // one token are 32 consecutive rows ----
    if (!sm.abort && warp < kWarps) {
        const int half = (warp >> 2) & 1, lane_base = 32 * (warp & 3), cbase = (warp >> 3) * (kNT / 2);
        const int64_t row = static_cast<int64_t>(r) * kTileM + half * 128 + lane_base + lane;
        for (int c0 = cbase; c0 < cbase + kNT / 2; c0 += 16) {
            if (n0 + c0 >= p.N) break;                                          // warp-uniform
            uint32_t v[16];
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                           "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                         : "r"(tmem + (static_cast<uint32_t>(lane_base) << 16) + half * kNT + c0) : "memory");
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
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
}

}  // namespace

spdp_status configure_spmm_kernel() {
    static std::mutex mu;
    static bool configured[64] = {};
    int dev = 0;
    SPDP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SPDP_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        SPDP_CUDA_TRY(cudaFuncSetAttribute(spmm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(kSmemBytes)));
        configured[dev] = true;
    }
    return SPDP_OK;
}

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
    p.nblocks = static_cast<int>((N + kNT - 1) / kNT);
    p.status = h->status_word;
    p.values_len = h->values_len;
    const int64_t ctas = h->R * p.nblocks;
    if (ctas >= (int64_t(1) << 31)) return SPDP_ERR_UNSUPPORTED_SHAPE;
    // X as a 2-D tensor [N][K] (row stride ldx): boxes of kKB columns x kNT tokens, 128-byte swizzle, zero fill
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return SPDP_ERR_CUDA;
    CUtensorMap xmap;
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(h->K), static_cast<cuuint64_t>(N)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(ldx) * sizeof(__half)};
    const cuuint32_t box[2] = {kKB, kNT};
    const cuuint32_t estride[2] = {1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(X), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SPDP_ERR_INVALID_ARG;
    spmm_kernel<<<static_cast<unsigned>(ctas), kThreads, kSmemBytes, s>>>(p, xmap);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
