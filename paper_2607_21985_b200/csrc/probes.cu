// Context measurements for the benchmark, not part of the method: how fast this GPU (a) reads the
// packed Values array front to back and (b) gathers exactly the bytes one spdp_spmspv call must
// fetch (the active column tiles' bitmaps and padded values, found through ColInfo / TileOffset)
// with plain loads and no decoding at all.  (b) is the ceiling of the access pattern that the
// spMspV kernel's time is held against, next to the copy-bandwidth roofline.
#include "spdp_internal.h"

namespace spdp {
namespace {

__global__ void probe_stream_read_kernel(const uint4* __restrict__ p, long long n, unsigned* __restrict__ sink) {
    unsigned acc = 0;
    long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (; i + 3 * stride < n; i += 4 * stride) {
        const uint4 a = __ldcs(p + i), b = __ldcs(p + i + stride), c = __ldcs(p + i + 2 * stride),
                    d = __ldcs(p + i + 3 * stride);
        acc ^= a.x ^ b.y ^ c.z ^ d.w;
    }
    for (; i < n; i += stride) acc ^= __ldcs(p + i).x;
    if (acc == 0x12345678u) sink[0] = acc;          // keeps the loads alive; practically never taken
}

// One warp per (row tile, 32 consecutive columns): the lanes test their column (the DP rule of
// Sec. 4.2 step (3)) and read its ColInfo word; then the warp walks the active columns four at a
// time, lane l reading the l-th 16-byte piece of a column's values and lanes 0-1 its bitmap.
__global__ void probe_gather_kernel(const uint32_t* __restrict__ tileoffset, const uint32_t* __restrict__ colinfo,
                                    const uint4* __restrict__ bitmap, const uint4* __restrict__ values,
                                    const __half* __restrict__ x, int rule, float thr,
                                    const uint32_t* __restrict__ mask, int K, int R, int C,
                                    unsigned* __restrict__ sink) {
    const int lane = threadIdx.x & 31;
    const long long nwarps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const long long wid = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int blocks_per_row = (K + 31) / 32;
    const long long total = static_cast<long long>(R) * blocks_per_row;
    const long long per = (total + nwarps - 1) / nwarps;
    const long long i0 = wid * per, i1 = (i0 + per < total) ? i0 + per : total;
    unsigned acc = 0;
    for (long long it = i0; it < i1; ++it) {
        const int r = static_cast<int>(it / blocks_per_row);
        const int j = static_cast<int>(it - static_cast<long long>(r) * blocks_per_row) * 32 + lane;
        bool act = false;
        unsigned ci = 0, base16 = 0;
        long long slot = 0;
        if (j < K) {
            if (rule == SPDP_DP_NONE) act = true;
            else if (rule == SPDP_DP_ABS_GT) act = !(fabsf(__half2float(x[j])) <= thr);
            else act = (mask[j >> 5] >> (j & 31)) & 1u;
            const long long g = static_cast<long long>(r) * C + (j >> 4);
            slot = g * kTileK + (j & 15);
            if (act) {
                ci = colinfo[slot];
                base16 = (tileoffset[g] + (ci >> 16)) >> 3;                 // 16-byte units into Values
            }
        }
        unsigned m = __ballot_sync(0xFFFFFFFFu, act);
        while (m != 0u) {
            uint4 v[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                v[u] = make_uint4(0, 0, 0, 0);
                b[u] = make_uint4(0, 0, 0, 0);
                const int src = (m != 0u) ? __ffs(m) - 1 : 0;
                const bool on = m != 0u;
                m &= m - 1u;
                const unsigned cu = __shfl_sync(0xFFFFFFFFu, ci, src);
                const unsigned bu = __shfl_sync(0xFFFFFFFFu, base16, src);
                const long long su = __shfl_sync(0xFFFFFFFFu, slot, src);
                if (on) {
                    const int pieces = ((cu & 0xFFFFu) + 7u) >> 3;
                    if (lane < pieces) v[u] = __ldcs(values + bu + lane);
                    if (lane < 2) b[u] = __ldcs(bitmap + su * 2 + lane);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w ^ b[u].x ^ b[u].w;
        }
    }
    if (acc == 0x12345678u) sink[0] = acc;
}

}  // namespace

spdp_status launch_probe_stream_read(const spdp_matrix* h, cudaStream_t s) {
    const long long n16 = h->values_len * 2 / 16;
    probe_stream_read_kernel<<<h->sm_count * 8, 256, 0, s>>>(reinterpret_cast<const uint4*>(h->values), n16,
                                                             reinterpret_cast<unsigned*>(h->status_word) + 1);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

spdp_status launch_probe_gather(const spdp_matrix* h, const __half* x, int rule, float thr, const uint32_t* mask,
                                cudaStream_t s) {
    probe_gather_kernel<<<h->sm_count * 8, 256, 0, s>>>(h->tileoffset, h->colinfo, reinterpret_cast<const uint4*>(h->bitmap),
                                                        reinterpret_cast<const uint4*>(h->values), x, rule, thr, mask,
                                                        static_cast<int>(h->K), static_cast<int>(h->R),
                                                        static_cast<int>(h->C),
                                                        reinterpret_cast<unsigned*>(h->status_word) + 1);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
