// Internal declarations shared by the translation units of libspdp (not part of the ABI).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spdp.h"

namespace spdp {

constexpr int kTileM = 256;        // rows per column tile (Sec. 4.1)
constexpr int kTileK = 16;         // column tiles per GTile (Sec. 4.2.3)
constexpr int kWordsPerCol = 4;    // 64-bit bitmap words per column tile (Sec. 4.1)
constexpr uint64_t kMagic = 0x5350445042323030ull;   // "SPDPB200"

}  // namespace spdp

// Host-side state behind an spdp_handle.
struct spdp_matrix {
    uint64_t magic;
    int device;
    int sm_count;
    int64_t M, K, R, C, NGT;
    int pad_elems;
    int64_t nnz;
    int64_t values_len;

    // Tiled-CBC arrays (device)
    uint32_t* tileoffset;   // [NGT+1]
    uint32_t* colinfo;      // [NGT*16]
    uint64_t* bitmap;       // [NGT*16*4]
    __half* values;         // [values_len] (at least 16 bytes are allocated); 4-bit variant: values_len codes, two per byte
    int q4;                 // 1: the 4-bit variant (codes + scales), pad_elems = 32
    __half* scales;         // 4-bit variant: [NGT*16] one scale per column tile; else null

    // Work partition of one spmspv launch: the kernel cuts the NGT GTiles into num_ctas equal
    // contiguous ranges, one per CTA.
    int num_ctas;           // P
    float* workspace;       // device [P*256] split-K tree nodes, one row per CTA (all zero between calls)
    float* workspace_batch; // device [P*8*256] tree nodes of the small-batch call (all zero between calls)
    int* status_word;       // device [2]: the status word, and a sink word the benchmark probes may write
    int64_t workspace_bytes;

    // Staging for the host-vector entry point
    __half* x_stage;        // device [K]
    uint32_t* mask_stage;   // device [ceil(K/32)]
    void* y_stage;          // device [M] fp32-sized

    // spdp_spmspv_host with the same pinned buffers and arguments as the call before: the three
    // operations (copy in, kernel, copy out) are kept as one instantiated graph and replayed.
    struct HostCallKey {
        const void* x;
        const void* mask;
        void* y;
        int rule, ydt, num_ctas;
        float thr;
    };
    HostCallKey host_last;          // arguments of the previous host-vector call
    bool host_last_valid;
    HostCallKey host_graph_key;     // arguments the graph below was recorded with
    cudaGraphExec_t host_graph;     // null: none
    cudaStream_t capture_stream;    // private stream used only to record that graph

    // Benchmark probe (spdp_probe_gather): the list of active column tiles it reads, built on first use.
    struct ProbeKey {
        const void* x;
        const void* mask;
        int rule;
        float thr;
    };
    void* probe_items;              // device uint2[R*K], null until the probe is first called
    void* probe_count;              // device uint64[1]
    ProbeKey probe_key;
};

namespace spdp {

// Records the message of a failed CUDA call for spdp_last_cuda_error().
void note_cuda_error(cudaError_t e, const char* what);

#define SPDP_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) {                             \
            ::spdp::note_cuda_error(e__, #expr);              \
            return (e__ == cudaErrorMemoryAllocation) ? SPDP_ERR_ALLOC : SPDP_ERR_CUDA; \
        }                                                     \
    } while (0)

inline bool valid(const spdp_matrix* h) { return h != nullptr && h->magic == kMagic; }

// pack.cu
spdp_status pack_device(spdp_matrix* h, const __half* W, int64_t ldw, cudaStream_t s);
spdp_status unpack_device(const spdp_matrix* h, __half* W, int64_t ldw, cudaStream_t s);

// spmspv.cu
int default_ctas_per_sm();   // CTAs of the spMspV kernel that share one SM
spdp_status configure_spmspv_kernel();   // per-device kernel attributes; idempotent
spdp_status launch_spmspv(const spdp_matrix* h, const __half* x, int rule, float thr,
                          const uint32_t* mask, void* y, int ydt, cudaStream_t s);
spdp_status launch_spmspv_noalloc(const uint32_t* tileoffset, const uint32_t* colinfo, const uint64_t* bitmap,
                                  const __half* values, int64_t M, int64_t K, const __half* x, int rule,
                                  float thr, const uint32_t* mask, void* y, int ydt, cudaStream_t s);
// spmspv_batch.cu
int64_t batch_workspace_bytes(int num_ctas);
spdp_status configure_spmspv_batch_kernel();   // per-device kernel attributes; idempotent
spdp_status launch_spmspv_batch(const spdp_matrix* h, const __half* x, int64_t ldx, int batch, int rule, float thr,
                                const uint32_t* mask, int64_t mask_stride, void* y, int64_t ldy, int ydt,
                                cudaStream_t s);

// spmspv_q4.cu / pack.cu: the 4-bit variant
spdp_status configure_spmspv_q4_kernel();      // per-device kernel attributes; idempotent
spdp_status pack_q4_device(spdp_matrix* h, const __half* W, int64_t ldw, cudaStream_t s);
spdp_status launch_spmspv_q4(const spdp_matrix* h, const __half* x, int rule, float thr, const uint32_t* mask, void* y,
                             int ydt, cudaStream_t s);

// producer.cu
spdp_status launch_swiglu_dp(const __half* gate, const __half* up, int64_t K, float thr, __half* x_out, uint32_t* mask_out,
                             int* count, cudaStream_t s);

// spmm.cu
spdp_status configure_spmm_kernel();            // per-device kernel attributes; idempotent
spdp_status launch_spmm(const spdp_matrix* h, const __half* X, int64_t N, int64_t ldx, void* Y, int64_t ldy, int ydt,
                        cudaStream_t s);

// probes.cu (context measurements for the benchmark)
spdp_status launch_probe_stream_read(const spdp_matrix* h, cudaStream_t s);
spdp_status launch_probe_gather(spdp_matrix* h, const __half* x, int rule, float thr, const uint32_t* mask,
                                cudaStream_t s);

spdp_status launch_active_columns(const spdp_matrix* h, const __half* x, int rule, float thr,
                                  const uint32_t* mask, uint32_t* bits, int* count, cudaStream_t s);

}  // namespace spdp
