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
// tensor memory), walking K in blocks of kKB columns through a software pipeline: while the
// tensor cores multiply block k, the warps decode block k+1, and the copies of the compressed
// column tiles of block k+2 and of the X tile of block k+1 are in flight.  A warp copies and decodes
// its own columns, so the compressed data needs no CTA-wide barrier; one barrier per block precedes
// the tensor-core issue.  The only waits (on the tensor cores' completion barriers) are bounded.
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kWarps = 16;             // warp w decodes columns w, w + 16 of a K-block; lane l owns rows 8l .. 8l+7
constexpr int kThreads = kWarps * 32;
constexpr int kKB = 64;                // columns per K-block: 4 GTiles, 4 tensor-core steps of K = 16 per accumulator
constexpr int kNT = 256;               // tokens per CTA (the N of the tensor-core instruction)
constexpr int kTmemCols = 2 * kNT;     // two accumulators of 128 rows x kNT fp32 columns
constexpr int kAStages = 2, kBStages = 2, kCStages = 2;
// A (decoded W), M-major without swizzle: 16-byte piece = 8 consecutive rows of one column; the 8
// columns of a k-group are 16 bytes apart (a core matrix of 128 bytes), the 16 row chunks of a
// 128-row half 144 bytes apart (128 + 16: the 16-byte pieces that the lanes of a quarter warp store for
// one column then fall into different banks), the k-groups 16 * 144 bytes apart.
constexpr int kAChunkStride = 144;                 // stride byte offset: next 8 rows
constexpr int kAKGroupStride = 16 * kAChunkStride; // leading byte offset: next 8 columns
constexpr int kAHalfBytes = (kKB / 8) * kAKGroupStride;
// B (X tile), K-major without swizzle: 16-byte piece = 8 consecutive columns of one token; the 8 tokens
// of a group are 16 bytes apart (a core matrix of 128 bytes), the k-groups 144 bytes apart (128 + 16: a warp
// copies 4 tokens x 8 k-groups per instruction, 4 whole lines of X, and its 32 pieces then spread evenly
// over the banks), the token groups kKB/8 * 144 bytes apart.
constexpr int kBCore = 144;
constexpr int kBTokenGroupStride = (kKB / 8) * kBCore;
constexpr int kBBytes = (kNT / 8) * kBTokenGroupStride;
constexpr int kWaitTries = 1 << 22;
static_assert(kTmemCols == 512, "the CTA owns all of tensor memory");
static_assert(kKB % 16 == 0 && kKB % kWarps == 0, "whole columns per warp and K-block");
constexpr int kColsPerWarp = kKB / kWarps;

struct Params {
    const uint32_t* tileoffset;
    const uint32_t* colinfo;
    const uint64_t* bitmap;
    const __half* values;
    const __half* X;        // [N][ldx]
    int64_t ldx;
    int64_t N;
    void* Y;                // [N][ldy]
    int64_t ldy;
    int ydt;
    int M, K, C;
    int nblocks;            // ceil(N / kNT): CTA = row tile * nblocks + token block
    int* status;
    int64_t values_len;
};

struct CompStage {                              // one K-block as stored: compact values, bitmaps
    alignas(16) unsigned short vals[kKB][kTileM];
    alignas(16) uint32_t bm[kKB][8];
};
struct __align__(128) Smem {
    unsigned char A[kAStages][2][kAHalfBytes];  // decoded W, two 128-row halves per stage
    unsigned char B[kBStages][kBBytes];         // X tiles
    CompStage comp[kCStages];
    alignas(8) unsigned long long mma_done[kAStages];   // the tensor cores are done with A stage s (and the B stage used with it)
    uint32_t tmem_base;
    int abort;
};
static_assert(sizeof(Smem) <= 227 * 1024, "shared memory of one CTA");

// Shared-memory operand descriptor of tcgen05.mma, no swizzle: start address, leading byte offset,
// stride byte offset (all in 16-byte units), descriptor version of this architecture.
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = (smem_addr & 0x3FFFFu) >> 4;
    d |= static_cast<uint64_t>(lbo >> 4) << 16;
    d |= static_cast<uint64_t>(sbo >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
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

// The 8 rows of one column tile that lane `lane` owns (one bitmap byte), as 8 fp16 in row order, zeros
// where the bit is clear.  The set bits before each of the 8 bitmap words come from a scan over
// 8-lane segments (every segment holds the 8 words); rank = those + the bits below the lane's byte;
// then a walk over the byte (Sec. 4.2.1).
__device__ __forceinline__ uint4 decode_chunk(const CompStage& cs, int j, int lane) {
    const unsigned w8 = cs.bm[j][lane & 7];
    const unsigned cnt = __popc(w8);
    unsigned inc = cnt;
    scan8_level<1>(inc);
    scan8_level<2>(inc);
    scan8_level<4>(inc);
    const unsigned word = __shfl_sync(0xFFFFFFFFu, w8, lane >> 2);
    const unsigned before = __shfl_sync(0xFFFFFFFFu, inc - cnt, lane >> 2);
    const int sh = 8 * (lane & 3);
    const unsigned bits = (word >> sh) & 0xFFu;
    unsigned out[4] = {0u, 0u, 0u, 0u};
    if (bits != 0u) {
        const unsigned short* v = &cs.vals[j][before + __popc(word & ((1u << sh) - 1u))];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if ((bits >> r) & 1u) {
                out[r >> 1] |= static_cast<unsigned>(*v) << (16 * (r & 1));
                ++v;
            }
        }
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

__global__ void __launch_bounds__(kThreads, 1)
spmm_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int r = static_cast<int>(blockIdx.x / static_cast<unsigned>(p.nblocks));
    const int nb = static_cast<int>(blockIdx.x - static_cast<unsigned>(r) * static_cast<unsigned>(p.nblocks));
    const int64_t n0 = static_cast<int64_t>(nb) * kNT;

    // ---- set-up: the completion barriers, and tensor memory ----
    if (t == 0) {
#pragma unroll
        for (int s = 0; s < kAStages; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.mma_done[s])) : "memory");
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
    const int nkb = (p.C * kTileK + kKB - 1) / kKB;

    // Where the column tiles this warp handles in K-block kb lie (ColInfo, TileOffset: Sec. 4.1): lane q < 4
    // looks up column warp + 16 q.  The loads are issued one iteration before their values are needed.
    struct Meta { uint32_t ci, to; };
    auto fetch_meta = [&](int kb) -> Meta {
        Meta m = {0u, 0u};
        const int col = kb * kKB + warp + kWarps * lane;
        if (lane < kColsPerWarp && kb < nkb && (col >> 4) < p.C) {
            const int64_t g = static_cast<int64_t>(r) * p.C + (col >> 4);
            m.ci = __ldg(p.colinfo + g * kTileK + (col & 15));
            m.to = __ldg(p.tileoffset + g);
        }
        return m;
    };
    // Starts the copies of this warp's column tiles of K-block kb as stored: lane l the l-th 16-byte piece
    // of the values, lanes 0-1 the bitmap.
    auto load_comp = [&](int kb, const Meta m) {
        if (kb >= nkb) return;
        CompStage& cs = sm.comp[kb % kCStages];
#pragma unroll
        for (int q = 0; q < kColsPerWarp; ++q) {
            const int j = warp + kWarps * q;
            const int col = kb * kKB + j;
            const uint32_t ci = __shfl_sync(0xFFFFFFFFu, m.ci, q), to = __shfl_sync(0xFFFFFFFFu, m.to, q);
            if ((col >> 4) < p.C) {
                const int64_t slot = (static_cast<int64_t>(r) * p.C + (col >> 4)) * kTileK + (col & 15);
                const uint32_t start = to + (ci >> 16);
                int pieces = static_cast<int>(((ci & 0xFFFFu) + 7u) >> 3);
                if (!SPDP_CHECK(p.status, start, 8 * pieces, p.values_len, kSiteValuesSpan) ||
                    !SPDP_CHECK(p.status, 0, pieces, 32, kSitePieces))
                    pieces = -1;                                                 // checked build only: the tile is left out
                if (lane < pieces)
                    cp_async16<0>(smem_u32(&cs.vals[j][8 * lane]), reinterpret_cast<const unsigned char*>(p.values) + 2ull * start + 16 * lane, 1);
                if (lane < 2) {
                    if (pieces >= 0)
                        cp_async16<0>(smem_u32(&cs.bm[j][4 * lane]), reinterpret_cast<const unsigned char*>(p.bitmap) + 32 * slot + 16 * lane, 1);
                    else
                        *reinterpret_cast<uint4*>(&cs.bm[j][4 * lane]) = make_uint4(0u, 0u, 0u, 0u);
                }
            } else if (lane < 2) {
                *reinterpret_cast<uint4*>(&cs.bm[j][4 * lane]) = make_uint4(0u, 0u, 0u, 0u);   // beyond the last GTile column
            }
        }
    };
    // Starts the copies of the X tile of K-block kb: kNT tokens x kKB/8 pieces of 16 bytes, zero beyond N and K.
    auto load_x = [&](int kb) {
        if (kb >= nkb) return;
        const uint32_t b_base = smem_u32(&sm.B[kb % kBStages][0]);
#pragma unroll
        for (int i = 0; i < kNT * (kKB / 8) / kThreads; ++i) {
            const int c = t + i * kThreads, nl = c / (kKB / 8), kc = c % (kKB / 8);   // 8 consecutive threads: one token's 128 bytes
            const int64_t n = n0 + nl;
            const int64_t k = static_cast<int64_t>(kb) * kKB + 8 * kc;
            int bytes = 0;
            if (n < p.N && k < p.K) bytes = static_cast<int>(min(static_cast<int64_t>(16), 2 * (p.K - k)));
            const __half* xs = bytes ? p.X + n * p.ldx + k : p.X;
            cp_async16_partial(b_base + (nl >> 3) * kBTokenGroupStride + kc * kBCore + (nl & 7) * 16, xs, bytes);
        }
    };

    // A wait that runs out (it never should) clears `ok`: the thread then stops waiting but keeps
    // walking the same barriers as the others, the status word gets SPDP_ERR_TIMEOUT and the outputs stay unwritten.
    bool ok = true;
    // copy groups: G(-2) = {comp(0), X(0)}, G(-1) = {comp(1)}, then G(kb) = {comp(kb+2), X(kb+1)} at the end of block kb
    load_comp(0, fetch_meta(0));
    load_x(0);
    cp_async_commit();
    load_comp(1, fetch_meta(1));
    cp_async_commit();
    Meta meta_next = fetch_meta(2);
    for (int kb = 0; kb < nkb; ++kb) {
        const int sa = kb % kAStages;
        cp_async_wait<1>();                 // my column tiles of block kb have arrived (the newest group may be in flight)
        __syncwarp();
        const CompStage& cs = sm.comp[kb % kCStages];
        // the tensor cores must be done with this A stage (block kb - kAStages)
        if (kb >= kAStages && ok) ok = wait_parity(&sm.mma_done[sa], ((kb / kAStages) - 1) & 1);
        // ---- decode: my 8 rows of my columns, one 16-byte piece each ----
        {
            unsigned char* a_stage = &sm.A[sa][lane >> 4][0] + (lane & 15) * kAChunkStride;
#pragma unroll
            for (int q = 0; q < kColsPerWarp; ++q) {
                const int j = warp + q * kWarps;
                const uint4 piece = decode_chunk(cs, j, lane);
                *reinterpret_cast<uint4*>(a_stage + (j >> 3) * kAKGroupStride + (j & 7) * 16) = piece;
            }
        }
        cp_async_wait<0>();                 // my pieces of the X tile of block kb have arrived
        // the operand tiles were written through the generic proxy; the tensor cores read through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        // ---- one thread issues the K-block's tensor-core work and commits it to the stage's barrier ----
        if (t == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_base = smem_u32(&sm.A[sa][0][0]), b_base = smem_u32(&sm.B[kb % kBStages][0]);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int kk = 0; kk < kKB / 16; ++kk) {
                    const uint64_t ad = operand_desc(a_base + h * kAHalfBytes + kk * 2 * kAKGroupStride, kAKGroupStride, kAChunkStride);
                    const uint64_t bd = operand_desc(b_base + kk * 2 * kBCore, kBCore, kBTokenGroupStride);
                    mma_f16(tmem + h * kNT, ad, bd, kb > 0 || kk > 0);
                }
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         ::"r"(smem_u32(&sm.mma_done[sa])) : "memory");
        }
        // Next copies: my column tiles of block kb+2 go where I just decoded block kb from; the X tile of
        // block kb+1 goes into the stage block kb-1 multiplied from, once that work is known to be complete.
        load_comp(kb + 2, meta_next);
        meta_next = fetch_meta(kb + 3);
        if (kb >= 1 && kb + 1 < nkb && ok) ok = wait_parity(&sm.mma_done[(kb - 1) % kAStages], ((kb - 1) / kAStages) & 1);
        load_x(kb + 1);
        cp_async_commit();
    }
    // the last blocks' tensor-core work
    for (int kb = (nkb > kAStages ? nkb - kAStages : 0); ok && kb < nkb; ++kb)
        ok = wait_parity(&sm.mma_done[kb % kAStages], (kb / kAStages) & 1);
    cp_async_wait<0>();
    if (!ok) {
        sm.abort = 1;
        if (lane == 0) atomicCAS(p.status, 0, SPDP_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    __syncthreads();

    // ---- epilogue: tensor memory -> registers -> Y.  Warp w reads lanes 32*(w%4).. of accumulator (w/4)%2,
    // token columns [(w/8)*kNT/2, +kNT/2); a thread holds one row, 16 tokens at a time, so a warp's stores of
    // one token are 32 consecutive rows ----
    if (!sm.abort) {
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
                                           static_cast<int>(sizeof(Smem))));
        configured[dev] = true;
    }
    return SPDP_OK;
}

spdp_status launch_spmm(const spdp_matrix* h, const __half* X, int64_t N, int64_t ldx, void* Y, int64_t ldy, int ydt,
                        cudaStream_t s) {
    Params p;
    p.tileoffset = h->tileoffset;
    p.colinfo = h->colinfo;
    p.bitmap = h->bitmap;
    p.values = h->values;
    p.X = X;
    p.ldx = ldx;
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
    spmm_kernel<<<static_cast<unsigned>(ctas), kThreads, sizeof(Smem), s>>>(p);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
