// Small pure functions that both the kernels and the host use (and that a host-compiled unit test
// exercises without a GPU): the split of the GTiles over the CTAs, and the range check of the
// checked build.  No CUDA headers: with a plain C++ compiler the qualifiers vanish.
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define SPDP_HD __host__ __device__ __forceinline__
#else
#define SPDP_HD inline
#endif

namespace spdp {
namespace hostdev {

// The work split (Sec. 4.2.3, tile-based scheme with Split-K): CTA c of num_ctas owns GTiles
// [range_begin(c), range_begin(c + 1)) of the row-major GTile order.  NGT < 2^22 and
// c <= num_ctas <= 1024 keep the product below 2^32.
SPDP_HD unsigned range_begin(unsigned ngt, unsigned num_ctas, unsigned c) { return (ngt * c) / num_ctas; }

// The CTA whose range holds GTile g: ceil((g + 1) * num_ctas / NGT) - 1.  The numerator can reach
// 2^32 + 2^22 at the limits, so this one is 64-bit (it runs twice per row tile, not per GTile).
SPDP_HD int range_owner(unsigned ngt, unsigned num_ctas, unsigned g) {
    const unsigned long long num = static_cast<unsigned long long>(g + 1u) * num_ctas + ngt - 1u;
    return static_cast<int>(num / ngt) - 1;
}

// Checked build: is [first, first + count) inside [0, limit)?  A violation is encoded as
// kCheckBase - site (site = a small number naming the access in the source) for the status word;
// the caller then skips the access.  Nothing traps and nothing asserts.
constexpr int kCheckBase = -1000;
SPDP_HD bool span_ok(uint64_t first, uint64_t count, uint64_t limit) {
    return first <= limit && count <= limit - first;
}
SPDP_HD int check_code(int site) { return kCheckBase - site; }

}  // namespace hostdev
}  // namespace spdp
