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

// Builds the list of what one call must fetch, one 8-byte item per active column tile in storage
// order: {start of its values in 16-byte units, column slot << 6 | 16-byte pieces}.  One CTA per
// row tile walks the columns in order (the DP rule of Sec. 4.2 step (3) per column, ballots and a
// running count).  Not timed.
__global__ void probe_items_kernel(const uint32_t* __restrict__ tileoffset, const uint32_t* __restrict__ colinfo,
                                   const __half* __restrict__ x, int rule, float thr,
                                   const uint32_t* __restrict__ mask, int K, int C, uint2* __restrict__ items,
                                   unsigned long long* __restrict__ count) {
    __shared__ unsigned warp_count[32];
    const int r = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    // pass 1 over the columns counts, pass 2 places: the active columns before row tile r are r * nact
    unsigned nact = 0;
    for (int pass = 0; pass < 2; ++pass) {
        unsigned running = 0;
        for (int j0 = 0; j0 < K; j0 += blockDim.x) {
            const int j = j0 + threadIdx.x;
            bool act = false;
            if (j < K) {
                if (rule == SPDP_DP_NONE) act = true;
                else if (rule == SPDP_DP_ABS_GT) act = !(fabsf(__half2float(x[j])) <= thr);
                else act = (mask[j >> 5] >> (j & 31)) & 1u;
            }
            const unsigned m = __ballot_sync(0xFFFFFFFFu, act);
            if (lane == 0) warp_count[warp] = __popc(m);
            __syncthreads();
            unsigned before = 0, all = 0;
            for (int w = 0; w < nwarps; ++w) {
                if (w < warp) before += warp_count[w];
                all += warp_count[w];
            }
            if (pass == 1 && act) {
                const long long g = static_cast<long long>(r) * C + (j >> 4);
                const long long slot = g * kTileK + (j & 15);
                const unsigned ci = colinfo[slot];
                const unsigned idx = running + before + __popc(m & ((1u << lane) - 1u));
                items[static_cast<long long>(r) * nact + idx] =
                    make_uint2((tileoffset[g] + (ci >> 16)) >> 3,
                               (static_cast<unsigned>(slot) << 6) | (((ci & 0xFFFFu) + 7u) >> 3));
            }
            running += all;
            __syncthreads();
        }
        nact = running;
    }
    if (r == 0 && threadIdx.x == 0) *count = static_cast<unsigned long long>(nact) * gridDim.x;
}

// The timed part: warps take groups of kUnroll items round-robin; lane l reads the l-th 16-byte
// piece of an item's values, lanes 0-1 its bitmap.
template <int kUnroll>
__global__ void probe_gather_kernel(const uint2* __restrict__ items, const unsigned long long* __restrict__ count,
                                    const uint4* __restrict__ values, const uint4* __restrict__ bitmap,
                                    unsigned* __restrict__ sink) {
    const int lane = threadIdx.x & 31;
    const long long n = static_cast<long long>(*count);
    const long long nwarps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const long long wid = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    unsigned acc = 0;
    for (long long i = wid * kUnroll; i < n; i += nwarps * kUnroll) {
        uint4 v[kUnroll], b[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            v[u] = make_uint4(0, 0, 0, 0);
            b[u] = make_uint4(0, 0, 0, 0);
            if (i + u < n) {
                const uint2 it = items[i + u];
                if (lane < static_cast<int>(it.y & 63u)) v[u] = __ldcs(values + it.x + lane);
                if (lane < 2) b[u] = __ldcs(bitmap + static_cast<long long>(it.y >> 6) * 2 + lane);
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w ^ b[u].x ^ b[u].w;
    }
    if (acc == 0x12345678u) sink[0] = acc;
}

}  // namespace

spdp_status launch_probe_stream_read(const spdp_matrix* h, cudaStream_t s) {
    const long long n16 = (h->q4 ? h->values_len / 2 : h->values_len * 2) / 16;      // bytes of the Values payload / 16
    probe_stream_read_kernel<<<h->sm_count * 8, 256, 0, s>>>(reinterpret_cast<const uint4*>(h->values), n16,
                                                             reinterpret_cast<unsigned*>(h->status_word) + 1);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

spdp_status launch_probe_gather(spdp_matrix* h, const __half* x, int rule, float thr, const uint32_t* mask,
                                cudaStream_t s) {
    // The item list is built on the first call and whenever the arguments change (a call with the same
    // pointers is taken to mean the same contents: this is a benchmark probe, not part of the method).
    const spdp_matrix::ProbeKey key = {x, mask, rule, thr};
    const bool same = h->probe_items != nullptr && h->probe_key.x == key.x && h->probe_key.mask == key.mask &&
                      h->probe_key.rule == key.rule && h->probe_key.thr == key.thr;
    if (!same) {
        if (h->probe_items == nullptr) {
            SPDP_CUDA_TRY(cudaMalloc(&h->probe_items, static_cast<size_t>(h->R) * h->K * sizeof(uint2) + 16));
            SPDP_CUDA_TRY(cudaMalloc(&h->probe_count, sizeof(unsigned long long)));
        }
        probe_items_kernel<<<static_cast<unsigned>(h->R), 256, 0, s>>>(h->tileoffset, h->colinfo, x, rule, thr, mask,
                                                                      static_cast<int>(h->K), static_cast<int>(h->C),
                                                                      static_cast<uint2*>(h->probe_items),
                                                                      static_cast<unsigned long long*>(h->probe_count));
        SPDP_CUDA_TRY(cudaGetLastError());
        h->probe_key = key;
    }
    probe_gather_kernel<8><<<h->sm_count * 8, 256, 0, s>>>(static_cast<const uint2*>(h->probe_items),
                                                          static_cast<const unsigned long long*>(h->probe_count),
                                                          reinterpret_cast<const uint4*>(h->values),
                                                          reinterpret_cast<const uint4*>(h->bitmap),
                                                          reinterpret_cast<unsigned*>(h->status_word) + 1);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
