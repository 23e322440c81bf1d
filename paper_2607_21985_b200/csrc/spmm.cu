// SPDP-SpMM for sm_100a (Sec. 4.3): Y[n] = W_sp * X[n] for N tokens on the Tiled-CBC matrix, static
// pruning only.  The paper's prefill kernel decodes a GTile with the same bitmap rule as the decode
// kernel, passes the decoded tile through shared memory to reach the tensor cores' operand layout
// (its "layout alignment" stage: TILE_K_PAD stride, ldmatrix.x4, mma.m16n8k16), and accumulates
// there.  On Blackwell the tensor cores read both operands straight from shared memory
// (tcgen05.mma) and accumulate in tensor memory, so the layout-alignment stage becomes the decode
// itself: every thread writes the dense fp16 values of its row, 8 columns at a time, directly at
// the address the operand descriptor expects (K-major core matrices of 8 rows x 16 bytes, no
// swizzle).  No registers hold accumulators and no ldmatrix pass exists.
//
// One CTA = one row tile (256 rows = two M = 128 accumulators) x kNT tokens, walking all of K in
// blocks of 64 columns (4 GTiles): copy the 64 column tiles (compressed) and the X tile into shared
// memory, decode, issue 2 x 4 tcgen05.mma (K = 16 each), commit them to a shared-memory barrier.
// Two CTAs share an SM (each owns half of tensor memory), so one decodes while the other's
// tensor-core work runs.  The only wait (on that barrier) is bounded.
#include <cstddef>
#include <mutex>

#include "spdp_internal.h"
#include "spmspv_device.cuh"

namespace spdp {
namespace {

using namespace dev;

constexpr int kThreads = 256;          // 8 warps; warp w decodes rows 32w .. 32w+31 of the row tile (bitmap word w)
constexpr int kKB = 64;                // columns per K-block: 4 GTiles, 4 tensor-core steps of K = 16
constexpr int kNT = 128;               // tokens per CTA (the N of the tensor-core instruction)
constexpr int kTmemCols = 2 * kNT;     // two accumulators of 128 rows x kNT fp32 columns (a power of two >= 32)
constexpr int kCoreBytes = 128;        // a core matrix: 8 rows x 16 bytes, rows 16 bytes apart
constexpr int kRowGroupBytes = (kKB / 8) * kCoreBytes;   // the 8 core matrices of 8 rows, one after the other along K
constexpr int kHalfBytes = 16 * kRowGroupBytes;          // 128 rows
constexpr int kWaitTries = 1 << 22;
static_assert(kTmemCols == 256 || kTmemCols == 512 || kTmemCols == 128, "tensor memory is allocated in powers of two");

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

struct __align__(128) Smem {
    unsigned char A[2][kHalfBytes];                 // decoded W: [half][row group][k core][row in group][8 fp16]
    unsigned char B[(kNT / 8) * kRowGroupBytes];    // X tile:    [token group][k core][token in group][8 fp16]
    alignas(16) unsigned short vals[kKB][kTileM];   // the K-block's column tiles as stored (compact values)
    alignas(16) uint32_t bm[kKB][8];                // their bitmaps as 32-bit words
    unsigned short prefix[kKB][8];                  // set bits before each word inside its column tile
    uint32_t start[kKB];                            // start of each column tile's values in Values (elements)
    uint32_t pieces[kKB];                           // its 16-byte pieces
    alignas(8) unsigned long long mma_done;         // the tensor cores' completion barrier
    uint32_t tmem_base;
    int abort;
};
static_assert(sizeof(Smem) <= 110 * 1024, "two CTAs per SM");

// Shared-memory operand descriptor of tcgen05.mma for a K-major tile without swizzle: the 16-byte
// row pieces of 8 consecutive rows are contiguous (a core matrix); lbo = distance between the two
// core matrices one instruction reads along K, sbo = distance between 8-row groups.
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = (smem_addr & 0x3FFFFu) >> 4;
    d |= static_cast<uint64_t>(lbo >> 4) << 16;
    d |= static_cast<uint64_t>(sbo >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;            // descriptor version of this architecture
    return d;                                       // layout type 0 (no swizzle), base offset 0
}
// Instruction descriptor: fp16 x fp16 -> fp32, both operands K-major, M = 128, N = kNT.
constexpr uint32_t kInstrDesc = (1u << 4) | (static_cast<uint32_t>(kNT >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);

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

__global__ void __launch_bounds__(kThreads, 2)
spmm_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int r = static_cast<int>(blockIdx.x / static_cast<unsigned>(p.nblocks));
    const int nb = static_cast<int>(blockIdx.x - static_cast<unsigned>(r) * static_cast<unsigned>(p.nblocks));
    const int64_t n0 = static_cast<int64_t>(nb) * kNT;

    // ---- set-up: the completion barrier, and this CTA's half of tensor memory ----
    if (t == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.mma_done)) : "memory");
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

    const uint32_t a_base = smem_u32(&sm.A[0][0]), b_base = smem_u32(&sm.B[0]);
    const uint32_t vals_base = smem_u32(&sm.vals[0][0]), bm_base = smem_u32(&sm.bm[0][0]);
    const int nkb = (p.C + 3) / 4;
    const unsigned lt_mask = (1u << lane) - 1u;
    bool ok = true;

    for (int kb = 0; kb < nkb; ++kb) {
        // ---- (1) where the K-block's 64 column tiles are (ColInfo, TileOffset: Sec. 4.1) ----
        if (t < kKB) {
            const int gc = 4 * kb + (t >> 4);                                   // GTile column
            uint32_t start = 0, pieces = 0;
            if (gc < p.C) {
                const int64_t g = static_cast<int64_t>(r) * p.C + gc;
                const uint32_t ci = __ldg(p.colinfo + g * kTileK + (t & 15));
                start = __ldg(p.tileoffset + g) + (ci >> 16);
                pieces = ((ci & 0xFFFFu) + 7u) >> 3;
                if (!SPDP_CHECK(p.status, start, 8u * pieces, p.values_len, kSiteValuesSpan) ||
                    !SPDP_CHECK(p.status, 0, pieces, 32, kSitePieces))
                    pieces = 0;                                                 // checked build only: the tile is left out
            }
            sm.start[t] = start;
            sm.pieces[t] = pieces;
        }
        __syncthreads();
        // ---- (2) copy them, and the X tile, into shared memory (16-byte asynchronous copies) ----
        {
            const int j = t >> 2, sub = t & 3;
            const int gc = 4 * kb + (j >> 4);
            const int pieces = static_cast<int>(sm.pieces[j]);
            const unsigned char* src = reinterpret_cast<const unsigned char*>(p.values) + 2ull * sm.start[j];
            for (int pc = sub; pc < pieces; pc += 4) cp_async16<0>(vals_base + j * (2 * kTileM) + 16 * pc, src + 16 * pc, 1);
            if (sub < 2) {
                if (gc < p.C) {
                    const int64_t slot = (static_cast<int64_t>(r) * p.C + gc) * kTileK + (j & 15);
                    cp_async16<0>(bm_base + 32 * j + 16 * sub, reinterpret_cast<const unsigned char*>(p.bitmap) + 32 * slot + 16 * sub, 1);
                } else {
                    *reinterpret_cast<uint4*>(&sm.bm[j][4 * sub]) = make_uint4(0u, 0u, 0u, 0u);   // beyond the last GTile column
                }
            }
#pragma unroll
            for (int i = 0; i < kNT * 8 / kThreads; ++i) {
                const int c = t + i * kThreads, nl = c >> 3, kc = c & 7;
                const int64_t n = n0 + nl;
                const int64_t k = static_cast<int64_t>(kb) * kKB + 8 * kc;
                int bytes = 0;                                                  // tokens beyond N and columns beyond K read as 0
                if (n < p.N && k < p.K) bytes = static_cast<int>(min(static_cast<int64_t>(16), 2 * (p.K - k)));
                const __half* xs = bytes ? p.X + n * p.ldx + k : p.X;
                cp_async16_partial(b_base + (nl >> 3) * kRowGroupBytes + kc * kCoreBytes + (nl & 7) * 16, xs, bytes);
            }
            cp_async_commit();
        }
        cp_async_wait<0>();
        __syncthreads();
        // ---- (3) set bits before each 32-bit word of each column tile ----
#pragma unroll
        for (int e = t; e < kKB * 8; e += kThreads) {
            const int j = e >> 3, w = e & 7;
            unsigned pre = 0;
            for (int q = 0; q < w; ++q) pre += __popc(sm.bm[j][q]);
            sm.prefix[j][w] = static_cast<unsigned short>(pre);
        }
        __syncthreads();
        // ---- (4) decode (Sec. 4.2.1 / 4.3): my row's value in each of the 64 columns, rank = set bits
        // before my position; 8 columns make one 16-byte piece of the operand tile ----
        {
            const uint32_t a_row = a_base + (warp >> 2) * kHalfBytes + ((warp & 3) * 4 + (lane >> 3)) * kRowGroupBytes + (lane & 7) * 16;
#pragma unroll 2
            for (int kc = 0; kc < 8; ++kc) {
                unsigned out[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int j = 8 * kc + c;
                    const unsigned word = sm.bm[j][warp];
                    unsigned v = 0;
                    if ((word >> lane) & 1u) v = sm.vals[j][sm.prefix[j][warp] + __popc(word & lt_mask)];
                    out[c >> 1] |= v << (16 * (c & 1));
                }
                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                             ::"r"(a_row + kc * kCoreBytes), "r"(out[0]), "r"(out[1]), "r"(out[2]), "r"(out[3]) : "memory");
            }
        }
        // the operand tiles were written through the generic proxy; the tensor cores read through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        // ---- (5) one thread issues the K-block's tensor-core work and commits it to the barrier ----
        if (t == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int kk = 0; kk < kKB / 16; ++kk) {
                    const uint64_t ad = operand_desc(a_base + h * kHalfBytes + kk * 2 * kCoreBytes, kCoreBytes, kRowGroupBytes);
                    const uint64_t bd = operand_desc(b_base + kk * 2 * kCoreBytes, kCoreBytes, kRowGroupBytes);
                    mma_f16(tmem + h * kNT, ad, bd, kb > 0 || kk > 0);
                }
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         ::"r"(smem_u32(&sm.mma_done)) : "memory");
        }
        // ---- (6) the tiles may be overwritten once the tensor cores are done with them ----
        ok = wait_parity(&sm.mma_done, kb & 1);
        if (!ok) break;
    }
    if (!ok) {
        sm.abort = 1;
        if (lane == 0) atomicCAS(p.status, 0, SPDP_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    __syncthreads();

    // ---- epilogue: tensor memory -> registers -> Y.  Warp w reads lanes 32*(w%4).. of accumulator w/4;
    // a thread holds one row, 16 tokens at a time, so a warp's stores of one token are 32 consecutive rows ----
    if (!sm.abort) {
        const int half = warp >> 2, lane_base = 32 * (warp & 3);
        const int64_t row = static_cast<int64_t>(r) * kTileM + half * 128 + lane_base + lane;
        for (int c0 = 0; c0 < kNT; c0 += 16) {
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
