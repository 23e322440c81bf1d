// The operation in front of a dynamically pruned projection, fused with the pruning decision
// (Sec. 6: DP variants that materialise a mask feed the same column-selection interface; Sec. 4.2
// step (3): the decision is a magnitude test against a threshold calibrated offline).  For a gated
// MLP the down-projection's input is x = silu(gate) * up; this kernel writes x (fp16) and, in the
// same pass, the K-bit mask "NOT(|x_j| <= thr)" that spdp_spmspv takes with SPDP_DP_MASK, so the
// decode kernel's list phase reads one bit per column instead of testing activations again, and a
// caller with another selection rule can write the mask itself.
#include "spdp_internal.h"

namespace spdp {
namespace {

__global__ void swiglu_dp_kernel(const __half* __restrict__ gate, const __half* __restrict__ up, int64_t K, float thr,
                                 __half* __restrict__ x_out, uint32_t* __restrict__ mask_out, int* __restrict__ count) {
    const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    bool active = false;
    if (j < K) {
        const float g = __half2float(gate[j]), u = __half2float(up[j]);
        const __half x = __float2half_rn(g / (1.0f + expf(-g)) * u);        // silu(g) * u in fp32, rounded once
        x_out[j] = x;
        active = !(fabsf(__half2float(x)) <= thr);                          // the decision is taken on the stored fp16 value
    }
    const unsigned m = __ballot_sync(0xFFFFFFFFu, active);
    if ((threadIdx.x & 31) == 0 && (j >> 5) < ((K + 31) >> 5)) {
        mask_out[j >> 5] = m;
        if (count != nullptr && m != 0u) atomicAdd(count, __popc(m));
    }
}

}  // namespace

spdp_status launch_swiglu_dp(const __half* gate, const __half* up, int64_t K, float thr, __half* x_out, uint32_t* mask_out,
                             int* count, cudaStream_t s) {
    if (count != nullptr) SPDP_CUDA_TRY(cudaMemsetAsync(count, 0, sizeof(int), s));
    const int threads = 256;
    const int64_t blocks = (((K + 31) / 32) * 32 + threads - 1) / threads;
    swiglu_dp_kernel<<<static_cast<unsigned>(blocks), threads, 0, s>>>(gate, up, K, thr, x_out, mask_out, count);
    SPDP_CUDA_TRY(cudaGetLastError());
    return SPDP_OK;
}

}  // namespace spdp
