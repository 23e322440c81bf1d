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
#include <mutex>

#include "spdp_internal.h"

namespace spdp {
namespace {

constexpr int kWarps = 16;                 // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr int kChunkCols = 4096;           // columns whose active list is built at once

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

__global__ void __launch_bounds__(kThreads)
spmspv_kernel(const Params p) {
    __shared__ uint32_t ent[kChunkCols];                 // (column in chunk) << 16 | x bits
    __shared__ uint32_t group_mask[kChunkCols / 32];
    __shared__ uint32_t group_base[kChunkCols / 32 + 1];
    __shared__ float red[kWarps][kTileM];
    __shared__ int is_last;

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int64_t g_begin = p.cta_begin[blockIdx.x], g_end = p.cta_begin[blockIdx.x + 1];
    const int r_first = static_cast<int>(g_begin / p.C);

    for (int64_t g0 = g_begin; g0 < g_end;) {
        const int r = static_cast<int>(g0 / p.C);
        const int c_lo = static_cast<int>(g0 - static_cast<int64_t>(r) * p.C);
        const int64_t c_end = c_lo + (g_end - g0);
        const int c_hi = static_cast<int>(c_end < p.C ? c_end : p.C);
        g0 += c_hi - c_lo;

        float acc[8];                                   // rows 8*lane .. 8*lane+7 of the row tile
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;

        const int j_lo = c_lo * kTileK, j_hi = min(c_hi * kTileK, p.K);
        for (int j0 = j_lo; j0 < j_hi; j0 += kChunkCols) {
            const int ncols = min(kChunkCols, j_hi - j0);
            const int ngroups = (ncols + 31) >> 5;
            // ---- active-column list of the chunk, in column order (ballots + prefix sums) ----
            for (int q = warp; q < ngroups; q += kWarps) {
                const int j = j0 + q * 32 + lane;
                bool a = false;
                if (j < j_hi) a = column_active(p.rule, p.thr, p.mask, j, p.x[j]);
                const unsigned m = __ballot_sync(0xFFFFFFFFu, a);
                if (lane == 0) group_mask[q] = m;
            }
            __syncthreads();
            if (warp == 0) {
                unsigned run = 0;
                for (int q0 = 0; q0 < ngroups; q0 += 32) {
                    const int q = q0 + lane;
                    unsigned c = (q < ngroups) ? __popc(group_mask[q]) : 0u;
                    unsigned inc = c;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        unsigned v = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                        if (lane >= d) inc += v;
                    }
                    if (q < ngroups) group_base[q] = run + inc - c;
                    run += __shfl_sync(0xFFFFFFFFu, inc, 31);
                }
                if (lane == 0) group_base[ngroups] = run;
            }
            __syncthreads();
            for (int q = warp; q < ngroups; q += kWarps) {
                const unsigned m = group_mask[q];
                if ((m >> lane) & 1u) {
                    const int jj = q * 32 + lane;
                    const unsigned xb = __half_as_ushort(p.x[j0 + jj]);
                    ent[group_base[q] + __popc(m & ((1u << lane) - 1u))] = (static_cast<unsigned>(jj) << 16) | xb;
                }
            }
            __syncthreads();
            const int nact = static_cast<int>(group_base[ngroups]);

            // ---- one warp per active column tile; lane owns 8 consecutive rows (one bitmap byte) ----
            for (int i = warp; i < nact; i += kWarps) {
                const uint32_t e = ent[i];
                const int j = j0 + static_cast<int>(e >> 16);
                const float xf = __half2float(__ushort_as_half(static_cast<unsigned short>(e & 0xFFFFu)));
                const int64_t g = static_cast<int64_t>(r) * p.C + (j >> 4);
                const int64_t slot = g * kTileK + (j & 15);
                const uint32_t ci = __ldg(p.colinfo + slot);
                if ((ci & 0xFFFFu) == 0) continue;
                const uint64_t base = static_cast<uint64_t>(__ldg(p.tileoffset + g)) + (ci >> 16);
                const unsigned b = __ldg(reinterpret_cast<const unsigned char*>(p.bitmap) + slot * 32 + lane);
                const unsigned c = __popc(b);
                unsigned inc = c;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    unsigned v = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= d) inc += v;
                }
                const __half* vp = p.values + base + (inc - c);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if ((b >> k) & 1u) {
                        acc[k] = fmaf(__half2float(__ldg(vp)), xf, acc[k]);
                        ++vp;
                    }
            }
            __syncthreads();       // ent / group_* are rebuilt by the next chunk
        }

        // ---- row reduction across the warps of the CTA (fixed order) ----
#pragma unroll
        for (int k = 0; k < 8; ++k) red[warp][8 * lane + k] = acc[k];
        __syncthreads();
        float part = 0.f;
        const int64_t row = static_cast<int64_t>(r) * kTileM + t;
        if (t < kTileM) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) part += red[w][t];
        }
        // ---- split-K combine ----
        const int nseg = p.row_nseg[r];
        if (nseg == 1) {
            if (t < kTileM && row < p.M) store_y(p.y, p.ydt, row, part);
        } else {
            float* mine = p.workspace + (static_cast<int64_t>(blockIdx.x) * 2 + (r != r_first)) * kTileM;
            if (t < kTileM) __stcg(mine + t, part);
            __threadfence();
            __syncthreads();
            if (t == 0) {
                const unsigned old = atomicAdd(p.row_counter + r, 1u);
                is_last = (old == static_cast<unsigned>(nseg - 1));
            }
            __syncthreads();
            if (is_last) {
                __threadfence();
                if (t < kTileM && row < p.M) {
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
        }
        __syncthreads();           // red[] and is_last are reused by the next segment
    }
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
constexpr int kNoAllocMaxCtas = 256;
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
    spmspv_kernel<<<h->num_ctas, kThreads, 0, s>>>(p);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
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
    int P = sms < kNoAllocMaxCtas ? sms : kNoAllocMaxCtas;
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
    spmspv_kernel<<<P, kThreads, 0, s>>>(p);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
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
