// Device helpers shared by the spMspV kernels (single vector and small batch): asynchronous copies,
// shared-memory accesses with explicit state space, the work split and the split-K combine.
#pragma once

#include "spdp_hostdev.h"
#include "spdp_internal.h"

namespace spdp {
namespace dev {

#ifndef SPDP_L2HINT
#define SPDP_L2HINT ".L2::64B"   // fill granularity asked of L2 for the value / bitmap copies: a column tile is a
                                 // few hundred bytes between skipped neighbours, so whole 128-byte lines over-fetch
#endif

__device__ __forceinline__ void store_y(void* y, int ydt, int64_t i, float v) {
    if (ydt == SPDP_Y_F32) static_cast<float*>(y)[i] = v;
    else static_cast<__half*>(y)[i] = __float2half_rn(v);
}

// Makes a loop-invariant value opaque to the compiler, so that it stays in its register instead of
// being recomputed from the thread index inside the hot loop.
template <typename T>
__device__ __forceinline__ T pinned(T v) {
    if constexpr (sizeof(T) == 8) asm volatile("" : "+l"(v));
    else asm volatile("" : "+r"(v));
    return v;
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// Asynchronous global -> shared copies (Sec. 4.2.3: 128-bit per thread); `on` = false copies nothing.
template <int kOff>
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int rem) {
    asm volatile("{\n .reg .pred p;\n setp.gt.s32 p, %2, %3;\n @p cp.async.cg.shared.global" SPDP_L2HINT " [%0+%4], [%1+%4], 16;\n}"
                 ::"r"(dst), "l"(src), "r"(rem), "n"(kOff / 16), "n"(kOff) : "memory");
}
// 16-byte copy that reads only the first `bytes` (0..16) source bytes and zero-fills the rest.
__device__ __forceinline__ void cp_async16_partial(uint32_t dst, const void* src, int bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global" SPDP_L2HINT " [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One level of an inclusive prefix sum over segments of 8 lanes.
template <int kDelta>
__device__ __forceinline__ void scan8_level(unsigned& v) {
    asm volatile("{\n .reg .pred p;\n .reg .b32 u;\n shfl.sync.up.b32 u|p, %0, %1, 0x1800, 0xffffffff;\n @p add.u32 %0, %0, u;\n}"
                 : "+r"(v) : "n"(kDelta));
}
__device__ __forceinline__ unsigned lds_u32(uint32_t addr) {
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
template <int kOff>
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4+%5];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr), "n"(kOff));
    return v;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
template <int kOff = 0>
__device__ __forceinline__ void sts_u32(uint32_t addr, unsigned v) {
    asm volatile("st.shared.u32 [%0+%2], %1;" ::"r"(addr), "r"(v), "n"(kOff) : "memory");
}
// base + a * kScale with a 64-bit result (one multiply-add)
template <int kScale>
__device__ __forceinline__ const unsigned char* offset_wide(const unsigned char* base, uint32_t a) {
    const unsigned char* r;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(r) : "r"(a), "n"(kScale), "l"(base));
    return r;
}

using hostdev::range_begin;     // the work split lives in spdp_hostdev.h (shared with the host)
using hostdev::range_owner;

// Checked build (-DSPDP_CHECKED): every record the kernels derive from the packed arrays (where a
// column tile's values start, how many 16-byte pieces they are, which bitmap slot they belong to,
// where the record goes) and every split-K node they are about to touch is held against its
// array's size first.  A violation stores check_code(site) in the status word (the first one
// wins) and the access is skipped: the tile is left out, the row is not stored.  Nothing traps and
// nothing asserts; it is the stand-in for a memory checker on hosts that have none.
#ifdef SPDP_CHECKED
__device__ __forceinline__ bool checked_span(int* status, uint64_t first, uint64_t count, uint64_t limit, int site) {
    if (hostdev::span_ok(first, count, limit)) return true;
    atomicCAS(status, 0, hostdev::check_code(site));
    return false;
}
#define SPDP_CHECK(status, first, count, limit, site) \
    ::spdp::dev::checked_span((status), static_cast<uint64_t>(first), static_cast<uint64_t>(count), static_cast<uint64_t>(limit), (site))
#else
#define SPDP_CHECK(status, first, count, limit, site) true
#endif
// Sites of the checks (the number a violation reports, as check_code(site)).
constexpr int kSiteRecordIndex = 1;     // record index inside the shared-memory list
constexpr int kSiteValuesSpan = 2;      // a column tile's padded values inside Values
constexpr int kSitePieces = 3;          // at most 32 16-byte pieces per column tile
constexpr int kSiteBitmapSlot = 4;      // column slot inside Bitmap / ColInfo
constexpr int kSiteTreeNodes = 5;       // split-K segments of a row tile inside the workspace
constexpr int kSiteOutputRow = 6;       // output row inside y

// A partial sum is kept in the workspace XOR this key, so that the all-zero word means "empty".
// NaN sums are made canonical first, which keeps a stored word from ever being zero.
constexpr unsigned kNodeKey = 0xFFC0DEADu;
__device__ __forceinline__ unsigned canonical_bits(float v) { return (v != v) ? 0x7FFFFFFFu : __float_as_uint(v); }


// Split-K combine of one output element across the nseg segments (CTAs q0 .. q0 + nseg - 1) that
// feed its row tile; my_seg is the caller's segment.  Segment i is leaf i of a binary tree: at level
// l, node idx stands for segments [idx << l, (idx + 1) << l); a node without a right-hand neighbour
// moves up unchanged.  Nodes (idx, idx | 1) meet in the workspace row of the CTA that owns the right
// node's first segment -- a CTA that starts inside this row tile, and a different one for every tree
// node (`nodes` points at this element inside workspace row 0, rows are node_stride words apart).
// Whoever reaches a node first leaves its sum there with one atomic exchange and returns false;
// the second takes it, empties the node for the next call, adds, and moves up.  Returns true in the
// one thread that completes the root; `part` then holds the sum.  a + b == b + a, so the result does
// not depend on the order of arrival.
__device__ __forceinline__ bool tree_combine(float& part, unsigned* nodes, int64_t node_stride, int q0, int nseg,
                                             int my_seg) {
    int idx = my_seg;
    for (int n = nseg, level = 0; n > 1; n = (n + 1) >> 1, ++level, idx >>= 1) {
        const int right = idx | 1;
        if (right >= n) continue;                       // no neighbour at this level
        unsigned* node = nodes + static_cast<int64_t>(q0 + (right << level)) * node_stride;
        const unsigned old = atomicExch(node, canonical_bits(part) ^ kNodeKey);
        if (old == 0u) return false;                    // first at the node: the neighbour carries the sum on
        *node = 0u;                                     // second: empty the node for the next call
        part += __uint_as_float(old ^ kNodeKey);
    }
    return true;
}

}  // namespace dev
}  // namespace spdp
