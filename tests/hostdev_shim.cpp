// Host build of the helpers the kernels share with the host (csrc/spdp_hostdev.h), for
// tests/test_hostdev_helpers.py.  Compiled with g++ by the test; not part of the library.
#include "spdp_hostdev.h"

extern "C" {
unsigned shim_range_begin(unsigned ngt, unsigned p, unsigned c) { return spdp::hostdev::range_begin(ngt, p, c); }
int shim_range_owner(unsigned ngt, unsigned p, unsigned g) { return spdp::hostdev::range_owner(ngt, p, g); }
int shim_span_ok(unsigned long long first, unsigned long long count, unsigned long long limit) {
    return spdp::hostdev::span_ok(first, count, limit) ? 1 : 0;
}
int shim_check_code(int site) { return spdp::hostdev::check_code(site); }
}
