/* libspdp -- C ABI of the B200 (sm_100a) SPDP decode path.
 *
 * y = W_sp * (x masked by dynamic pruning): W_sp is an unstructured, statically pruned fp16
 * matrix held in the Tiled-CBC format (Sec. 4.1 of the paper), x is one token's fp16
 * activation vector, and columns whose activation fails the dynamic-pruning (DP) test are
 * never fetched from device memory (Sec. 4.2).
 *
 * Conventions that hold for every call
 *  - All tensor pointers named *_dev are CALLER-OWNED DEVICE memory on the device that was
 *    current when the handle was created; pointers named *_host are host memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *  - Every call returns an spdp_status; nothing throws; out-parameters are written only on
 *    SPDP_OK unless stated.  Host-detectable errors (null pointers, bad handle, unsupported
 *    shape) are returned before any work is enqueued.
 *  - A handle owns its packed arrays, its split-K workspace and a few staging buffers.  The
 *    workspace is per handle, so at most ONE spdp_spmspv per handle may be in flight; calls on
 *    one handle must be ordered (same stream, or events).  Different handles are independent.
 *    A call that was aborted, or that overlapped another call on the same handle, can leave a partial
 *    sum in the workspace; spdp_set_num_ctas (any value, also the current one) empties it again.
 *  - Format constants: column tile 256 x 1, GTile 256 x 16, four 64-bit bitmap words per column
 *    tile (Sec. 4.1); 16-byte padding of every column's values (Sec. 4.2.3).
 */
#ifndef SPDP_H_
#define SPDP_H_

#include <stdint.h>

#if defined(__GNUC__)
#define SPDP_API __attribute__((visibility("default")))
#else
#define SPDP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spdp_matrix* spdp_handle;   /* opaque; created by pack/import, released by spdp_free */

typedef enum {
    SPDP_OK = 0,
    SPDP_ERR_INVALID_ARG = -1,       /* null pointer, bad handle, bad enum, misaligned pointer */
    SPDP_ERR_UNSUPPORTED_SHAPE = -2, /* tile shape other than 256 x 16, M or K < 1, ldw < K      */
    SPDP_ERR_ALLOC = -3,             /* device or host allocation failed                        */
    SPDP_ERR_CUDA = -4,              /* a CUDA runtime call failed (see spdp_last_cuda_error)    */
    SPDP_ERR_OVERFLOW = -5,          /* Values would need 2^32 or more elements (TileOffset is 32-bit) */
    SPDP_ERR_TIMEOUT = -6            /* a bounded device-side wait expired (spdp_spmm; see spdp_last_device_status) */
} spdp_status;

/* Dynamic-pruning rule: which columns of W are fetched for this x (Sec. 2.2 "Dynamic Pruning",
 * W_dp(x) = W (.) M(x); Sec. 4.2 step (3): a magnitude metric of the activation against a
 * threshold calibrated offline, Sec. 5.1). */
typedef enum {
    SPDP_DP_NONE = 0,    /* every column is active                                              */
    SPDP_DP_ABS_GT = 1,  /* column j active iff NOT(|x_j| <= thr), compared in fp32 on the exactly
                            widened fp16 x_j: ties are skipped, thr = 0 skips exact zeros, thr < 0
                            keeps everything, NaN and +-Inf activations are active             */
    SPDP_DP_MASK = 2     /* explicit mask: bit (j % 32) of 32-bit word (j / 32) of mask_dev (Sec. 6:
                            DP variants that materialise a mask use the same column interface)  */
} spdp_dp_rule;

typedef enum { SPDP_Y_F16 = 0, SPDP_Y_F32 = 1 } spdp_ydtype;

/* Shape, sizes and device addresses of a packed matrix (all sizes in elements unless named bytes). */
typedef struct {
    int64_t M, K;              /* logical matrix shape                                          */
    int64_t R, C, NGT;         /* row tiles ceil(M/256), GTile columns ceil(K/16), R*C          */
    int64_t pad_elems;         /* every column's values are padded to a multiple of this (8 or 1) */
    int64_t nnz;               /* stored nonzeros                                               */
    int64_t values_len;        /* = TileOffset[NGT], padding included                           */
    int64_t packed_bytes;      /* bytes of TileOffset + ColInfo + Bitmap + Values               */
    int64_t workspace_bytes;   /* split-K scratch owned by the handle                           */
    const void* tileoffset_dev;  /* uint32[NGT+1]  start of each GTile in Values (elements)      */
    const void* colinfo_dev;     /* uint32[NGT*16] (column start inside its GTile) << 16 | nnz   */
    const void* bitmap_dev;      /* uint64[NGT*16*4] bit b of word w = row 64*w+b of the column tile */
    const void* values_dev;      /* fp16[values_len] nonzeros in tile-column order, zero padded  */
    int32_t num_ctas;          /* CTAs one spdp_spmspv launches                                 */
    int32_t device;            /* CUDA device ordinal the handle lives on                       */
} spdp_info;

/* Pack a dense, statically pruned matrix into Tiled-CBC (Sec. 4.1 "Storage Structure";
 * padding rule of Sec. 4.2.3).
 *   W_dev     fp16 [M][ldw] row-major, device; an element is "pruned" iff its value is +-0
 *             (bits & 0x7FFF == 0); every other bit pattern, NaN/Inf/subnormals included, is
 *             stored verbatim.
 *   M, K      >= 1; sides that are not multiples of 256 / 16 are zero-extended logically.  The matrix
 *             may hold at most 2^26 column tiles (ceil(M/256) * ceil(K/16) * 16), else
 *             SPDP_ERR_UNSUPPORTED_SHAPE.
 *   ldw       leading dimension in elements, >= K.
 *   tile_m, tile_k  must be 256 and 16 (the format's constants), else SPDP_ERR_UNSUPPORTED_SHAPE.
 *   out       receives the handle.  The call allocates device memory, runs on `stream` and
 *             synchronises it once (packing is an offline step).  W_dev is not retained.
 * GTile (r, c) has linear index r*C + c; its 16 ColInfo words and 64 bitmap words are
 * contiguous; Values holds, per GTile and per column, the column's nonzeros in row order
 * followed by 0x0000 padding up to a multiple of 8 elements. */
SPDP_API spdp_status spdp_pack_tiled_cbc(const void* W_dev, int64_t M, int64_t K, int64_t ldw,
                                int tile_m, int tile_k, void* stream, spdp_handle* out);

/* Same as spdp_pack_tiled_cbc with the padding unit chosen: pad_elems = 8 (the format) or 1 (no
 * padding: the byte count then equals the storage formula of Sec. 4.1 exactly).  Handles packed
 * with pad_elems = 1 can be inspected, exported and unpacked; spdp_spmspv rejects them with
 * SPDP_ERR_UNSUPPORTED_SHAPE because its 16-byte loads need the padding. */
SPDP_API spdp_status spdp_pack_tiled_cbc_ex(const void* W_dev, int64_t M, int64_t K, int64_t ldw,
                                   int tile_m, int tile_k, int pad_elems, void* stream, spdp_handle* out);

/* Pack with a 4-bit Values payload (Sec. 5.1: 4-bit round-to-nearest weights, applied after static
 * pruning and before dynamic pruning; Sec. 6: Values are stored apart from the sparsity metadata, so
 * they can be low-bit).  The paper fixes no layout for it; this library's is: TileOffset, ColInfo and
 * Bitmap exactly as in Sec. 4.1, with offsets counted in CODES and every column padded to 32 codes
 * (16 bytes); Codes holds, per column tile, its n codes in row order, two per byte (even rank in the
 * low nibble), zero padded; Scales holds one fp16 per column tile (same index as ColInfo).
 *   scale = fp16(max|w| of the column tile / 7), computed in fp32;
 *   code  = clamp(rint(w / scale), -7, 7) + 8 in fp32, ties to even (8 where the scale is 0);
 *   the weight a code stands for is (code - 8) * scale.
 * Weights must be finite (codes of Inf/NaN are unspecified).  Arguments as spdp_pack_tiled_cbc.
 * The handle works with spdp_spmspv, spdp_spmspv_host, spdp_active_columns, spdp_get_info
 * (pad_elems = 32, values_len = number of codes), spdp_set_num_ctas and spdp_export_q4; the other
 * calls return SPDP_ERR_UNSUPPORTED_SHAPE for it.  spdp_spmspv on such a handle computes
 * y = sum over active columns of (code - 8) * scale * x_j with fp32 accumulation. */
SPDP_API spdp_status spdp_pack_tiled_cbc_q4(const void* W_dev, int64_t M, int64_t K, int64_t ldw, int tile_m,
                                   int tile_k, void* stream, spdp_handle* out);

/* Copy the arrays of a 4-bit handle to HOST buffers: tileoffset uint32[NGT+1], colinfo uint32[NGT*16],
 * bitmap uint64[NGT*64], codes uint8[values_len/2], scales fp16[NGT*16] (any pointer may be NULL).
 * Synchronous.  SPDP_ERR_INVALID_ARG for a handle that is not 4-bit. */
SPDP_API spdp_status spdp_export_q4(spdp_handle h, void* tileoffset_host, void* colinfo_host, void* bitmap_host,
                           void* codes_host, void* scales_host);

/* Build a handle from the four Tiled-CBC arrays in HOST memory (Sec. 4.1).  The arrays are
 * validated on the host (monotone TileOffset, ColInfo offsets equal to the prefix sums of the
 * padded counts, bitmap popcounts equal to the ColInfo counts); a mismatch returns
 * SPDP_ERR_INVALID_ARG.  The data is copied; the host arrays are not retained. */
SPDP_API spdp_status spdp_import_tiled_cbc(int64_t M, int64_t K, int pad_elems, const void* tileoffset_host,
                                  const void* colinfo_host, const void* bitmap_host,
                                  const void* values_host, int64_t values_len, spdp_handle* out);

/* y = W_sp * x over the active columns only (Sec. 4.2, Alg. 1; fp32 accumulation).
 *   x_dev     fp16 [K], device, 2-byte aligned.
 *   rule/thr  the DP rule; thr is used by SPDP_DP_ABS_GT only.
 *   mask_dev  uint32[ceil(K/32)], device; required for SPDP_DP_MASK, ignored otherwise.
 *   y_dev     [M] of ydt (fp16 rounded to nearest even from the fp32 sum, or fp32), device.
 *             Every one of the M entries is written, also when no column is active (zeros).
 * Asynchronous on `stream`; allocates nothing and never synchronises.  Launches one kernel.
 * The summation order is fixed for a given handle, so repeated calls give identical bits.
 * No CTA of the kernel ever waits for another one (the split-K combine is made of single atomic
 * exchanges), so there is nothing on the device that can time out; the handle's device status word,
 * readable with spdp_last_device_status, is reserved for device-side checks and stays 0. */
SPDP_API spdp_status spdp_spmspv(spdp_handle h, const void* x_dev, spdp_dp_rule rule, float thr,
                        const void* mask_dev, void* y_dev, spdp_ydtype ydt, void* stream);

/* Small-batch decode: Y[b] = W_sp * x_b for `batch` tokens (1..SPDP_MAX_BATCH) in one pass over
 * the packed matrix.  The paper treats one token per call and names batched DP decode as future
 * work (Sec. 6); this entry point applies its definition token by token: token b has its own
 * active set (the DP rule on x_b), a column tile is fetched once if ANY token keeps its column,
 * and a token that skips a column enters the product with 0 for it.  With finite weights that is
 * the omission of the column; a column tile that holds Inf or NaN and is fetched for another token
 * gives NaN instead (0 * Inf).  Likewise a NaN or Inf activation of a kept column reaches, through the
 * zeros of the fetched tiles, every row (0 * NaN), as in a dense product; the single-vector call
 * multiplies stored nonzeros only.
 *   x_dev        fp16 [batch][ldx], device, ldx >= K elements between tokens.
 *   mask_dev     uint32 [batch][mask_stride] words, mask_stride >= ceil(K/32); SPDP_DP_MASK only.
 *   y_dev        [batch][ldy] of ydt, ldy >= M elements between tokens; all batch*M entries are written.
 * Asynchronous on `stream`, allocates nothing; launches one kernel for 3 or more tokens and one
 * single-vector kernel per token below that (which is faster there).  The handle's workspaces allow
 * one such call in flight per handle.  Results are identical from call to call. */
#define SPDP_MAX_BATCH 8
SPDP_API spdp_status spdp_spmspv_batch(spdp_handle h, const void* x_dev, int64_t ldx, int batch, spdp_dp_rule rule,
                              float thr, const void* mask_dev, int64_t mask_stride, void* y_dev, int64_t ldy,
                              spdp_ydtype ydt, void* stream);

/* Prefill product on the same packed handle (Sec. 4.3, SPDP-SpMM): Y[n] = W_sp * X[n] for N tokens,
 * static pruning only (no dynamic pruning: every column is fetched once per block of tokens).
 * The column tiles are decoded from Tiled-CBC into dense fp16 operand tiles in shared memory (what
 * the paper's layout-alignment stage does for its tensor-core path), the contraction runs on the
 * 5th-generation tensor cores (tcgen05.mma, fp16 inputs, fp32 accumulation in tensor memory).
 *   X_dev   fp16 [N][ldx], device, one token per row, ldx >= K elements between tokens; X_dev must
 *           be 16-byte aligned and ldx a multiple of 8 (the tiles are read through a tensor map,
 *           encoded on the host at every call), else SPDP_ERR_INVALID_ARG.
 *   N       >= 1 tokens.
 *   Y_dev   [N][ldy] of ydt, device, ldy >= M elements between tokens; all N*M entries are written.
 * Asynchronous on `stream`.  Usually one kernel and no allocation.  When the last round of CTAs would
 * leave more than half of the SMs idle, the tiles of that round are cut along K instead: a second launch
 * leaves fp32 partial sums in scratch memory taken from the device's stream-ordered pool (cudaMallocAsync /
 * cudaFreeAsync on `stream`, 0.5 MB per slice) and a third adds the slices in a fixed order.  The handle's
 * workspace is never touched, so calls on one handle may overlap.  The waits inside the kernel (on
 * shared-memory barriers that the copies and the tensor cores complete) are bounded; one that runs
 * out records SPDP_ERR_TIMEOUT in the handle's status word and the CTA leaves its outputs unwritten;
 * TileOffset words that do not describe a K-block that fits shared memory record SPDP_ERR_OVERFLOW
 * the same way.  SPDP_ERR_CUDA if the driver's tensor-map encoder cannot be found. */
SPDP_API spdp_status spdp_spmm(spdp_handle h, const void* X_dev, int64_t N, int64_t ldx, void* Y_dev, int64_t ldy,
                      spdp_ydtype ydt, void* stream);

/* Same product with HOST vectors (Sec. 4.2): copies x_host (fp16 [K], ideally pinned) to a
 * staging buffer of the handle, runs spdp_spmspv, copies y back into y_host ([M] of ydt) and
 * synchronises `stream`.  mask_host is uint32[ceil(K/32)] or NULL.  When the same pinned buffers and
 * arguments come twice in a row, the three operations are recorded once as a CUDA graph (on a private
 * stream of the handle) and later calls with those arguments replay it with one launch; pageable
 * buffers, changing arguments or a stream that is being captured take the plain path. */
SPDP_API spdp_status spdp_spmspv_host(spdp_handle h, const void* x_host, spdp_dp_rule rule, float thr,
                             const void* mask_host, void* y_host, spdp_ydtype ydt, void* stream);

/* The same product for callers that must not allocate (the paper has no counterpart: this entry
 * point exists for the library's users, not for the method).  Some hosts of this code cannot
 * call cudaMalloc at all: a serving process that hands all device memory to its own arena at
 * start-up, an embedding that forbids driver allocations after initialisation, a caller that
 * already holds the four Tiled-CBC arrays in memory it manages.  For them nothing here creates a
 * handle; the caller passes the packed arrays (device pointers, laid out as spdp_info describes,
 * 16-byte column padding), x, the DP rule and y, exactly as for spdp_spmspv.
 *
 * What spdp_spmspv keeps in a handle-owned allocation (the split-K partial sums that CTAs
 * exchange) lives in ONE fixed device array inside the library, about 0.5 MB, present on every
 * GPU that loads the library until the process exits.  It bounds the launch to 512 CTAs (the
 * library never asks for more); shapes beyond the library's general limit (2^26 column tiles)
 * return SPDP_ERR_UNSUPPORTED_SHAPE.  The call enqueues a small set-up kernel (which empties the
 * part of the array this call uses, whatever an earlier call left there) and the spMspV kernel
 * on `stream`; it calls no cudaMalloc, cudaFree or allocating library routine.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current) and the SM count; make that first call outside any stream capture.
 * Every call on a device shares the one array: two calls that can overlap on the GPU (different
 * streams without ordering, or two host threads) race on it and give wrong sums; order them.
 * Results equal spdp_spmspv's for the same CTA count. */
SPDP_API spdp_status spdp_spmspv_noalloc(const void* tileoffset_dev, const void* colinfo_dev,
                                const void* bitmap_dev, const void* values_dev, int64_t M, int64_t K,
                                const void* x_dev, spdp_dp_rule rule, float thr, const void* mask_dev,
                                void* y_dev, spdp_ydtype ydt, void* stream);

/* Producer-fused dynamic pruning (Sec. 6: DP variants that materialise a mask map to the same column
 * interface; Sec. 4.2 step (3): a magnitude test against a threshold calibrated offline).  The input of
 * a gated MLP's down-projection is x = silu(gate) * up; this call computes it (fp32 arithmetic, one
 * rounding to fp16) and writes, in the same pass, the mask of the columns the following spdp_spmspv
 * should keep: bit (j % 32) of word (j / 32) is NOT(|x_j| <= thr) evaluated on the STORED fp16 x_j, i.e.
 * exactly the set SPDP_DP_ABS_GT would choose.  Pass the mask with SPDP_DP_MASK.  A caller with
 * another per-column score (say |x_j| times a column norm) gets its mask from spdp_active_columns on
 * the score vector and uses SPDP_DP_MASK in the same way.
 *   gate_dev, up_dev  fp16 [K], device.     x_dev_out  fp16 [K], device.
 *   mask_dev_out      uint32[ceil(K/32)], device (bits beyond K clear).
 *   count_dev_out     int32[1], device, or NULL: number of kept columns.
 * Asynchronous on `stream`; allocates nothing. */
SPDP_API spdp_status spdp_swiglu_dp(const void* gate_dev, const void* up_dev, int64_t K, float thr, void* x_dev_out,
                           void* mask_dev_out, void* count_dev_out, void* stream);

/* Row-tile sharding over several GPUs (the paper names multi-GPU execution as future work, Sec. 6; the
 * natural split of y = W x keeps whole 256-row tiles together, so every rank packs its own rows as
 * an independent Tiled-CBC matrix, x is replicated, and the outputs are disjoint).  This is the split
 * every rank must agree on: the ceil(M/256) row tiles are dealt out in contiguous runs, the first
 * (tiles % world) ranks get one more.  Writes rank's first row and its number of rows (0 when there
 * are fewer row tiles than ranks).  Host arithmetic only. */
SPDP_API spdp_status spdp_row_shard(int64_t M, int world, int rank, int64_t* first_row_out, int64_t* rows_out);

/* Release the handle and everything it owns.  spdp_free(NULL) is SPDP_OK. */
SPDP_API spdp_status spdp_free(spdp_handle h);

/* ---- inspection surface (the format and the active set are checked bit for bit) ---- */

SPDP_API spdp_status spdp_get_info(spdp_handle h, spdp_info* out);

/* Copy the four arrays to HOST buffers sized as in spdp_info (any pointer may be NULL to skip
 * it).  Synchronous. */
SPDP_API spdp_status spdp_export(spdp_handle h, void* tileoffset_host, void* colinfo_host,
                        void* bitmap_host, void* values_host);

/* Decode the packed matrix back to dense fp16 [M][ldw] in device memory with the rule of
 * Sec. 4.2.1 (bit clear -> +0, else Values[base + number of set bits before the position]).
 * Asynchronous on `stream`. */
SPDP_API spdp_status spdp_unpack(spdp_handle h, void* W_dev_out, int64_t ldw, void* stream);

/* The active-column set spdp_spmspv would use for this x (Sec. 4.2 step (3)):
 * bitmask_dev_out uint32[ceil(K/32)] (bit j%32 of word j/32, bits beyond K clear) and, if not
 * NULL, count_dev_out int32[1], both device.  Asynchronous on `stream`. */
SPDP_API spdp_status spdp_active_columns(spdp_handle h, const void* x_dev, spdp_dp_rule rule, float thr,
                                const void* mask_dev, void* bitmask_dev_out, void* count_dev_out,
                                void* stream);

/* Context measurements for the benchmark (the paper has no counterpart; they compute nothing).
 * spdp_probe_stream_read reads the handle's Values array front to back with plain 16-byte loads;
 * spdp_probe_gather reads exactly what one spdp_spmspv call with these arguments must fetch -- the
 * ColInfo / TileOffset words of the active columns, their bitmaps and their padded values -- with
 * plain loads and no decoding (its first call, and any call with other arguments, first builds the
 * list of those tiles in a scratch buffer it allocates; repeated calls with the same pointers reuse
 * the list, so time the repeats).  Both are asynchronous on `stream` and write nothing the caller can
 * see; the caller times them.  They give the speed of a contiguous read and
 * the ceiling of the method's access pattern on this GPU, next to which the kernel is reported. */
SPDP_API spdp_status spdp_probe_stream_read(spdp_handle h, void* stream);
SPDP_API spdp_status spdp_probe_gather(spdp_handle h, const void* x_dev, spdp_dp_rule rule, float thr,
                              const void* mask_dev, void* stream);

/* Read (and clear) the handle's device status word: 0, or an spdp_status recorded by a kernel.
 * Synchronises the device. */
SPDP_API spdp_status spdp_last_device_status(spdp_handle h, int* out);

/* Tuning knob: number of CTAs spdp_spmspv launches (0 = default, one per SM; at most 1024 and at
 * most one per GTile are used).  Takes effect on
 * the next call; re-derives the handle's split-K workspace layout (may reallocate it). */
SPDP_API spdp_status spdp_set_num_ctas(spdp_handle h, int num_ctas);

/* Text of the last CUDA runtime error seen by the library on this thread ("" if none). */
SPDP_API const char* spdp_last_cuda_error(void);

SPDP_API const char* spdp_status_string(spdp_status s);

#ifdef __cplusplus
}
#endif
#endif /* SPDP_H_ */
