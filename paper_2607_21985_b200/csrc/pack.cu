// Tiled-CBC packer and unpacker kernels (Sec. 4.1 "Storage Structure", Sec. 4.2.1 decode rule,
// Sec. 4.2.3 padding).  Offline path: three passes (count -> scan -> emit), one CTA per GTile.
#include "spdp_internal.h"

namespace spdp {
namespace {

__device__ __forceinline__ bool is_stored(unsigned short bits) { return (bits & 0x7FFFu) != 0; }

// Loads row `row` of GTile (r, c): 16 fp16 bit patterns, zero beyond the matrix edge.
__device__ __forceinline__ void load_tile_row(const unsigned short* __restrict__ W, int64_t ldw,
                                              int64_t M, int64_t K, int64_t row, int64_t col0,
                                              unsigned short (&v)[kTileK]) {
#pragma unroll
    for (int cc = 0; cc < kTileK; ++cc) v[cc] = 0;
    if (row >= M) return;
    const unsigned short* p = W + row * ldw + col0;
    if (col0 + kTileK <= K && ((reinterpret_cast<uintptr_t>(p) & 15u) == 0)) {
        uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
        uint4 b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
        unsigned w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            v[2 * q] = static_cast<unsigned short>(w[q] & 0xFFFFu);
            v[2 * q + 1] = static_cast<unsigned short>(w[q] >> 16);
        }
    } else {
#pragma unroll
        for (int cc = 0; cc < kTileK; ++cc)
            if (col0 + cc < K) v[cc] = __ldg(p + cc);
    }
}

// Pass 1: bitmap words, per-column nonzero counts, ColInfo, padded length of the GTile.
__global__ void __launch_bounds__(kTileM)
pack_count_kernel(const unsigned short* __restrict__ W, int64_t ldw, int64_t M, int64_t K, int64_t C,
                  int pad_elems, uint64_t* __restrict__ bitmap, uint32_t* __restrict__ colinfo,
                  uint32_t* __restrict__ tile_len, unsigned long long* __restrict__ nnz_total) {
    __shared__ unsigned words32[kTileK][kTileM / 32];
    __shared__ unsigned padded[kTileK];
    __shared__ unsigned count[kTileK];
    const int64_t g = blockIdx.x;
    const int64_t r = g / C, c = g % C;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    unsigned short v[kTileK];
    load_tile_row(W, ldw, M, K, r * kTileM + t, c * kTileK, v);
#pragma unroll
    for (int cc = 0; cc < kTileK; ++cc) {
        unsigned b = __ballot_sync(0xFFFFFFFFu, is_stored(v[cc]));
        if (lane == 0) words32[cc][warp] = b;
    }
    __syncthreads();
    if (t < kTileK * kWordsPerCol) {
        int cc = t >> 2, w = t & 3;
        uint64_t word = static_cast<uint64_t>(words32[cc][2 * w]) |
                        (static_cast<uint64_t>(words32[cc][2 * w + 1]) << 32);
        bitmap[(g * kTileK + cc) * kWordsPerCol + w] = word;
    }
    if (t < kTileK) {
        unsigned n = 0;
#pragma unroll
        for (int w = 0; w < kTileM / 32; ++w) n += __popc(words32[t][w]);
        count[t] = n;
        padded[t] = (n + pad_elems - 1) / pad_elems * pad_elems;
    }
    __syncthreads();
    if (t == 0) {
        unsigned off = 0, n = 0;
        for (int cc = 0; cc < kTileK; ++cc) {
            colinfo[g * kTileK + cc] = (off << 16) | count[cc];
            off += padded[cc];
            n += count[cc];
        }
        tile_len[g] = off;
        if (n) atomicAdd(nnz_total, static_cast<unsigned long long>(n));
    }
}

// Pass 2: exclusive scan of the padded GTile lengths into TileOffset (one CTA; the array has
// at most a few hundred thousand entries).  total_out receives the 64-bit total.
__global__ void __launch_bounds__(1024)
pack_scan_kernel(const uint32_t* __restrict__ tile_len, int64_t NGT, uint32_t* __restrict__ tileoffset,
                 unsigned long long* __restrict__ total_out) {
    __shared__ unsigned long long part[1024];
    const int t = threadIdx.x;
    const int64_t per = (NGT + 1023) / 1024;
    const int64_t lo = min(NGT, t * per), hi = min(NGT, lo + per);
    unsigned long long s = 0;
    for (int64_t i = lo; i < hi; ++i) s += tile_len[i];
    part[t] = s;
    __syncthreads();
    for (int d = 1; d < 1024; d <<= 1) {
        unsigned long long add = (t >= d) ? part[t - d] : 0ull;
        __syncthreads();
        part[t] += add;
        __syncthreads();
    }
    unsigned long long run = part[t] - s;
    for (int64_t i = lo; i < hi; ++i) {
        tileoffset[i] = static_cast<uint32_t>(run);
        run += tile_len[i];
    }
    if (t == 1023) {
        tileoffset[NGT] = static_cast<uint32_t>(part[1023]);
        *total_out = part[1023];
    }
}

// Pass 3: write every stored element to Values[TileOffset[g] + column offset + rank]; the
// padding halfwords keep the zero fill of the buffer.
__global__ void __launch_bounds__(kTileM)
pack_emit_kernel(const unsigned short* __restrict__ W, int64_t ldw, int64_t M, int64_t K, int64_t C,
                 const uint32_t* __restrict__ tileoffset, const uint32_t* __restrict__ colinfo,
                 unsigned short* __restrict__ values) {
    __shared__ unsigned words32[kTileK][kTileM / 32];
    const int64_t g = blockIdx.x;
    const int64_t r = g / C, c = g % C;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    unsigned short v[kTileK];
    load_tile_row(W, ldw, M, K, r * kTileM + t, c * kTileK, v);
    unsigned mine[kTileK];
#pragma unroll
    for (int cc = 0; cc < kTileK; ++cc) {
        mine[cc] = __ballot_sync(0xFFFFFFFFu, is_stored(v[cc]));
        if (lane == 0) words32[cc][warp] = mine[cc];
    }
    __syncthreads();
    const uint64_t base = tileoffset[g];
#pragma unroll
    for (int cc = 0; cc < kTileK; ++cc) {
        if (!is_stored(v[cc])) continue;
        unsigned rank = __popc(mine[cc] & ((1u << lane) - 1u));
        for (int w = 0; w < warp; ++w) rank += __popc(words32[cc][w]);
        values[base + (colinfo[g * kTileK + cc] >> 16) + rank] = v[cc];
    }
}

// Pass 3 of the 4-bit variant (Sec. 5.1, 4-bit round to nearest, after static pruning): one fp16 scale
// per column tile = max|w| / 7, code = clamp(rint(w / scale), -7, 7) + 8 in fp32 (ties to even; code 8
// where the scale underflows to 0), the column's codes in row order, two per byte, low nibble first.
__global__ void __launch_bounds__(kTileM)
pack_q4_emit_kernel(const unsigned short* __restrict__ W, int64_t ldw, int64_t M, int64_t K, int64_t C,
                    const uint32_t* __restrict__ tileoffset, const uint32_t* __restrict__ colinfo,
                    unsigned char* __restrict__ codes, unsigned short* __restrict__ scales) {
    __shared__ unsigned words32[kTileK][kTileM / 32];
    __shared__ float warp_max[kTileK][kTileM / 32];
    __shared__ unsigned char by_rank[kTileK][kTileM];
    const int64_t g = blockIdx.x;
    const int64_t r = g / C, c = g % C;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    unsigned short v[kTileK];
    load_tile_row(W, ldw, M, K, r * kTileM + t, c * kTileK, v);
    unsigned mine[kTileK];
#pragma unroll
    for (int cc = 0; cc < kTileK; ++cc) {
        mine[cc] = __ballot_sync(0xFFFFFFFFu, is_stored(v[cc]));
        float a = is_stored(v[cc]) ? fabsf(__half2float(__ushort_as_half(v[cc]))) : 0.f;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, d));
        if (lane == 0) {
            words32[cc][warp] = mine[cc];
            warp_max[cc][warp] = a;
        }
    }
    __syncthreads();
#pragma unroll
    for (int cc = 0; cc < kTileK; ++cc) {
        float mx = 0.f;
#pragma unroll
        for (int w = 0; w < kTileM / 32; ++w) mx = fmaxf(mx, warp_max[cc][w]);
        const __half s16 = __float2half_rn(__fdiv_rn(mx, 7.0f));
        if (t == 0) scales[g * kTileK + cc] = __half_as_ushort(s16);
        if (!is_stored(v[cc])) continue;
        const float sf = __half2float(s16);
        int q = 0;
        if (sf != 0.f) {
            q = static_cast<int>(rintf(__fdiv_rn(__half2float(__ushort_as_half(v[cc])), sf)));
            q = q < -7 ? -7 : (q > 7 ? 7 : q);
        }
        unsigned rank = __popc(mine[cc] & ((1u << lane) - 1u));
        for (int w = 0; w < warp; ++w) rank += __popc(words32[cc][w]);
        by_rank[cc][rank] = static_cast<unsigned char>(q + 8);
    }
    __syncthreads();
    const uint64_t base = tileoffset[g];
    if (t < kTileM / 2) {
#pragma unroll
        for (int cc = 0; cc < kTileK; ++cc) {
            const uint32_t ci = colinfo[g * kTileK + cc];
            const int n = static_cast<int>(ci & 0xFFFFu);
            if (2 * t < n) {
                const unsigned lo = by_rank[cc][2 * t], hi = (2 * t + 1 < n) ? by_rank[cc][2 * t + 1] : 0u;
                codes[((base + (ci >> 16)) >> 1) + t] = static_cast<unsigned char>(lo | (hi << 4));
            }
        }
    }
}

// Decode rule of Sec. 4.2.1: bit clear -> +0, else Values[base + set bits before the position].
__global__ void __launch_bounds__(kTileM)
unpack_kernel(const uint32_t* __restrict__ tileoffset, const uint32_t* __restrict__ colinfo,
              const uint64_t* __restrict__ bitmap, const unsigned short* __restrict__ values,
              int64_t M, int64_t K, int64_t C, unsigned short* __restrict__ W, int64_t ldw) {
    const int64_t g = blockIdx.x;
    const int64_t r = g / C, c = g % C;
    const int t = threadIdx.x;
    const int64_t row = r * kTileM + t;
    if (row >= M) return;
    const uint64_t base = tileoffset[g];
    const int w = t >> 6, b = t & 63;
    for (int cc = 0; cc < kTileK; ++cc) {
        const int64_t col = c * kTileK + cc;
        if (col >= K) break;
        const uint64_t* bm = bitmap + (g * kTileK + cc) * kWordsPerCol;
        uint64_t word = bm[w];
        unsigned short out = 0;
        if ((word >> b) & 1ull) {
            unsigned rank = __popcll(word & ((1ull << b) - 1ull));
            for (int q = 0; q < w; ++q) rank += __popcll(bm[q]);
            out = values[base + (colinfo[g * kTileK + cc] >> 16) + rank];
        }
        W[row * ldw + col] = out;
    }
}

}  // namespace

spdp_status pack_device(spdp_matrix* h, const __half* W, int64_t ldw, cudaStream_t s) {
    const int64_t NGT = h->NGT;
    uint32_t* tile_len = nullptr;
    unsigned long long* total_dev = nullptr;
    SPDP_CUDA_TRY(cudaMalloc(&h->tileoffset, (NGT + 1) * sizeof(uint32_t)));
    SPDP_CUDA_TRY(cudaMalloc(&h->colinfo, NGT * kTileK * sizeof(uint32_t)));
    SPDP_CUDA_TRY(cudaMalloc(&h->bitmap, NGT * kTileK * kWordsPerCol * sizeof(uint64_t)));
    SPDP_CUDA_TRY(cudaMalloc(&tile_len, NGT * sizeof(uint32_t)));
    cudaError_t e = cudaMalloc(&total_dev, 2 * sizeof(unsigned long long));   // [0] Values length, [1] nnz
    if (e != cudaSuccess) { cudaFree(tile_len); SPDP_CUDA_TRY(e); }
    const unsigned short* Wb = reinterpret_cast<const unsigned short*>(W);
    spdp_status st = SPDP_OK;
    unsigned long long totals[2] = {0, 0};
    do {
        e = cudaMemsetAsync(total_dev, 0, 2 * sizeof(unsigned long long), s);
        if (e != cudaSuccess) { note_cuda_error(e, "cudaMemsetAsync(totals)"); st = SPDP_ERR_CUDA; break; }
        pack_count_kernel<<<static_cast<unsigned>(NGT), kTileM, 0, s>>>(
            Wb, ldw, h->M, h->K, h->C, h->pad_elems, h->bitmap, h->colinfo, tile_len, total_dev + 1);
        pack_scan_kernel<<<1, 1024, 0, s>>>(tile_len, NGT, h->tileoffset, total_dev);
        e = cudaMemcpyAsync(totals, total_dev, sizeof(totals), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) { note_cuda_error(e, "pack count/scan"); st = SPDP_ERR_CUDA; break; }
        const unsigned long long total = totals[0];
        if (total >= (1ull << 32)) { st = SPDP_ERR_OVERFLOW; break; }
        h->values_len = static_cast<int64_t>(total);
        h->nnz = static_cast<int64_t>(totals[1]);
        const size_t vbytes = static_cast<size_t>(total) * sizeof(__half);
        e = cudaMalloc(&h->values, vbytes < 16 ? 16 : vbytes);
        if (e != cudaSuccess) { note_cuda_error(e, "cudaMalloc(values)"); st = SPDP_ERR_ALLOC; break; }
        e = cudaMemsetAsync(h->values, 0, vbytes < 16 ? 16 : vbytes, s);
        if (e != cudaSuccess) { note_cuda_error(e, "cudaMemsetAsync(values)"); st = SPDP_ERR_CUDA; break; }
        pack_emit_kernel<<<static_cast<unsigned>(NGT), kTileM, 0, s>>>(
            Wb, ldw, h->M, h->K, h->C, h->tileoffset, h->colinfo,
            reinterpret_cast<unsigned short*>(h->values));
        e = cudaStreamSynchronize(s);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { note_cuda_error(e, "pack emit"); st = SPDP_ERR_CUDA; break; }
    } while (false);
    cudaFree(tile_len);
    cudaFree(total_dev);
    return st;
}

// The 4-bit variant: same count and scan passes with a padding unit of 32 codes, then the quantising emit.
spdp_status pack_q4_device(spdp_matrix* h, const __half* W, int64_t ldw, cudaStream_t s) {
    const int64_t NGT = h->NGT;
    uint32_t* tile_len = nullptr;
    unsigned long long* total_dev = nullptr;
    SPDP_CUDA_TRY(cudaMalloc(&h->tileoffset, (NGT + 1) * sizeof(uint32_t)));
    SPDP_CUDA_TRY(cudaMalloc(&h->colinfo, NGT * kTileK * sizeof(uint32_t)));
    SPDP_CUDA_TRY(cudaMalloc(&h->bitmap, NGT * kTileK * kWordsPerCol * sizeof(uint64_t)));
    SPDP_CUDA_TRY(cudaMalloc(&h->scales, NGT * kTileK * sizeof(__half)));
    SPDP_CUDA_TRY(cudaMalloc(&tile_len, NGT * sizeof(uint32_t)));
    cudaError_t e = cudaMalloc(&total_dev, 2 * sizeof(unsigned long long));   // [0] code count, [1] nnz
    if (e != cudaSuccess) { cudaFree(tile_len); SPDP_CUDA_TRY(e); }
    const unsigned short* Wb = reinterpret_cast<const unsigned short*>(W);
    spdp_status st = SPDP_OK;
    unsigned long long totals[2] = {0, 0};
    do {
        e = cudaMemsetAsync(total_dev, 0, 2 * sizeof(unsigned long long), s);
        if (e != cudaSuccess) { note_cuda_error(e, "cudaMemsetAsync(totals)"); st = SPDP_ERR_CUDA; break; }
        pack_count_kernel<<<static_cast<unsigned>(NGT), kTileM, 0, s>>>(
            Wb, ldw, h->M, h->K, h->C, h->pad_elems, h->bitmap, h->colinfo, tile_len, total_dev + 1);
        pack_scan_kernel<<<1, 1024, 0, s>>>(tile_len, NGT, h->tileoffset, total_dev);
        e = cudaMemcpyAsync(totals, total_dev, sizeof(totals), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) { note_cuda_error(e, "pack count/scan"); st = SPDP_ERR_CUDA; break; }
        if (totals[0] >= (1ull << 32)) { st = SPDP_ERR_OVERFLOW; break; }
        h->values_len = static_cast<int64_t>(totals[0]);
        h->nnz = static_cast<int64_t>(totals[1]);
        const size_t cbytes = static_cast<size_t>(totals[0]) / 2 + 16;         // + 16: the decode reads one word past a span
        e = cudaMalloc(&h->values, cbytes);
        if (e != cudaSuccess) { note_cuda_error(e, "cudaMalloc(codes)"); st = SPDP_ERR_ALLOC; break; }
        e = cudaMemsetAsync(h->values, 0, cbytes, s);
        if (e != cudaSuccess) { note_cuda_error(e, "cudaMemsetAsync(codes)"); st = SPDP_ERR_CUDA; break; }
        pack_q4_emit_kernel<<<static_cast<unsigned>(NGT), kTileM, 0, s>>>(
            Wb, ldw, h->M, h->K, h->C, h->tileoffset, h->colinfo, reinterpret_cast<unsigned char*>(h->values),
            reinterpret_cast<unsigned short*>(h->scales));
        e = cudaStreamSynchronize(s);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { note_cuda_error(e, "pack q4 emit"); st = SPDP_ERR_CUDA; break; }
    } while (false);
    cudaFree(tile_len);
    cudaFree(total_dev);
    return st;
}

spdp_status unpack_device(const spdp_matrix* h, __half* W, int64_t ldw, cudaStream_t s) {
    unpack_kernel<<<static_cast<unsigned>(h->NGT), kTileM, 0, s>>>(
        h->tileoffset, h->colinfo, h->bitmap, reinterpret_cast<const unsigned short*>(h->values),
        h->M, h->K, h->C, reinterpret_cast<unsigned short*>(W), ldw);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
