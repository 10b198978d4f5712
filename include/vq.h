/*
 * vq.h — C-ABI boundary of the B200 VQ-decode linear-layer library.
 *
 * The library implements the decode-phase linear layer of GPTVQ (arXiv 2402.15319):
 * weights live in HBM vector-quantized, are expanded through small per-block
 * look-up tables and multiplied by the token activations on the fly.
 *
 * Representation (paper Sec. 2.1 and Sec. 3.1): a weight matrix W (N out-features x
 * K in-features, row-major) is split into blocks of block_rows x block_cols weights.
 * Each block is stored as the tuple
 *   (1) packed VQ indices, (2) its codebook / LUT, (3) an optional scale factor.
 * One index of `index_bits` bits selects one of k = 2^index_bits codebook entries;
 * an entry holds `vq_dim` values which are `vq_dim` ADJACENT COLUMNS of one row
 * (Sec. 4: the quantizer walks the matrix d columns at a time).  Bits per value follow the
 * paper's formula  log2(k)/d + k*d*b_c/l  (Sec. 4, the paragraph on total bits per value).
 *
 * Memory layout fixed by this library (the paper fixes no bit order or row pitch):
 *   indices : N rows; row n is a little-endian bitstream: index j (covering columns
 *             j*d .. j*d+d-1) occupies bits [j*b, (j+1)*b) where bit t of the stream is
 *             bit (t mod 8) of byte (t div 8).  Rows start at n*row_stride_bytes;
 *             row_stride_bytes = ceil(K/d*b/8) rounded up to a multiple of 16.
 *             The CALLER lays the rows out at that pitch: the buffer holds N * row_stride_bytes
 *             bytes (vq_pack_info().index_bytes), all of them readable.  The value of padding
 *             bits/bytes is ignored, but the kernels' bulk copies do read them.
 *   codebook: cb[blk][entry][t], t < d; blk = (n / block_rows)*(K / block_cols) + (k / block_cols).
 *             VQ_CB_FP16: IEEE binary16.  VQ_CB_INT8_SCALED: signed 8-bit.
 *   scale   : VQ_CB_INT8_SCALED only: one binary16 per block, w = scale * int8.
 *             (VQ_CB_INT4_G128: 4-bit entries and a scale per row and 128 columns, described at vq_cb_type.)
 *   x / X   : activations, binary16, X[batch][K] row-major.
 *   y / Y   : outputs, binary16, Y[batch][N] row-major; accumulated in fp32, rounded once.
 *
 * Conventions for every entry point:
 *   - `extern "C"`, plain pointers and sizes.  Pointers named d_* are DEVICE pointers,
 *     h_* are HOST pointers; `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - The caller owns all buffers.  Inputs are read-only.  The library allocates nothing,
 *     frees nothing, never synchronises: work is enqueued on `stream` and the call returns.
 *   - WEIGHT buffers (indices, codebooks, scales) must be complete and visible to the device
 *     BEFORE a GEMV/GEMM call is enqueued: the kernels are launched with programmatic dependent
 *     launch and start fetching weights while the previous kernel on `stream` may still be
 *     running; only activations, outputs and workspace are ordered after that kernel.  Weights
 *     produced on the device (vq_assign_indices, a copy, the caller's own kernel) therefore need
 *     a host-side stream or event synchronisation before the first call that reads them; stream
 *     order alone is not enough.
 *   - WORKSPACE (d_ws): the first vq_workspace_bytes()-defined counter region of a workspace must
 *     read as zero the first time it is used: zero-fill a workspace once after allocating it
 *     (cudaMemsetAsync on the same stream is enough).  Every call leaves the counters zero again,
 *     so the workspace can be reused by later calls of any format and batch without clearing.
 *     The rest of its contents is scratch (ignored on entry, unspecified on exit).  Calls that
 *     may overlap on the GPU (different streams) need different workspaces.
 *   - All argument checks run on the host before any launch; on error nothing is launched.
 *   - Same inputs give bit-identical outputs (no floating-point atomics).
 */
#ifndef VQ_B200_H
#define VQ_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  VQ_OK = 0,
  VQ_ERR_NULL = 1,        /* required pointer is NULL, or scale pointer presence does not match cb_type */
  VQ_ERR_FORMAT = 2,      /* vq_dim not in {1,2,4}, index_bits not in 1..8, unknown cb_type            */
  VQ_ERR_SHAPE = 3,       /* N % block_rows, K % block_cols, block_cols % vq_dim, sizes <= 0            */
  VQ_ERR_ALIGN = 4,       /* a device pointer is not 16-byte aligned                                    */
  VQ_ERR_WORKSPACE = 5,   /* workspace smaller than vq_workspace_bytes() or NULL when needed            */
  VQ_ERR_BATCH = 6,       /* batch outside 1..16                                                        */
  VQ_ERR_UNSUPPORTED = 7, /* valid format but the requested kernel variant does not cover it            */
  VQ_ERR_CUDA = 8         /* a CUDA runtime call or the launch itself reported an error                 */
} vq_status;

/* VQ_CB_INT4_G128 (paper Sec. 4.2: codebooks held as 4-bit integers, one scale per group of 128 values):
 *   d_cb    : per block 2^index_bits * vq_dim signed 4-bit integers (-8..7), two per byte, value
 *             v = entry * vq_dim + t in nibble v mod 2 (low nibble first) of byte v / 2;
 *   d_scale : binary16 [N][K/128]; w[n][k] = scale[n][k/128] * c.  K % 128 == 0.
 * vq_decode_weights decodes it with its tile kernel; the skinny GEMM runs in the tuned shared-codebook
 * kernels for 2-D formats with 5- or 6-bit indices (blocks of 32, 64 or a multiple of 128 rows and a
 * multiple of 128 columns, K a multiple of 256) and in the pair-table kernel for the block shapes that
 * one takes (see vq_impl); in both a looked-up pair is fp16(scale * c), the value vq_decode_weights
 * writes; other formats of this codebook type run in the format-generic kernel (VQ_IMPL_TUNED returns
 * VQ_ERR_UNSUPPORTED for them); vq_assign_indices does not take it. */
typedef enum {
  VQ_CB_FP16 = 0,         /* binary16 entries                                                        */
  VQ_CB_INT8_SCALED = 1,  /* signed 8-bit entries, one binary16 scale per block                       */
  VQ_CB_INT4_G128 = 2     /* signed 4-bit entries, one binary16 scale per row and group of 128 columns */
} vq_cb_type;

/* Kernel selection for the *_impl entry points.  VQ_IMPL_AUTO is what the plain entry points use.
 * Tuned kernels exist for: 4-bit indices with per-row codebooks or blocks of a few rows (2-D, and 1-D
 * with int8 codebooks); 2-D 5- and 6-bit and 4-D 8-bit indices with tall blocks (32, 64 or a multiple of
 * 128 rows; 256 for 4-D); and, through tables of fp16 PAIRS private to a warp, every other 2-D format,
 * every 1-D format of up to 4 index bits (two indices per look-up) and 4-D 8-bit indices (four weights
 * per look-up) whose blocks have 1, 2, 4, 8 (4-D: 8) or a multiple of 16 rows and whose block columns
 * and K are multiples of 64 (any codebook type) - the remaining rows of the paper's table of VQ
 * configurations (its appendix on VQ configurations). */
typedef enum {
  VQ_IMPL_AUTO = 0,     /* tuned kernel when one covers the format/shape, else the generic one   */
  VQ_IMPL_GENERIC = 1,  /* format-generic fp32-FMA kernel (any valid format)                     */
  VQ_IMPL_TUNED = 2,    /* tuned kernel only; VQ_ERR_UNSUPPORTED if none covers the format/shape */
  VQ_IMPL_STREAM = 3    /* the persistent tuned kernel only (the one AUTO picks for large per-row 4-bit
                           layers and for groups); VQ_ERR_UNSUPPORTED if it does not cover the format */
} vq_impl;

/* Caller-filled description of one VQ-compressed matrix (paper Sec. 2.1 notation in comments). */
typedef struct {
  int32_t n_rows;      /* N, out features (rows of W)                         */
  int32_t k_cols;      /* K, in features (columns of W)                       */
  int32_t vq_dim;      /* d in {1,2,4}: values per codebook entry             */
  int32_t index_bits;  /* b = log2(k) in 1..8: bits per index                 */
  int32_t block_rows;  /* rows of the block sharing one codebook              */
  int32_t block_cols;  /* columns of that block (multiple of d); l = rows*cols */
  int32_t cb_type;     /* vq_cb_type                                          */
} vq_format;

/* Library-filled sizes for a format. */
typedef struct {
  int32_t entries;                  /* k = 2^b                                              */
  int32_t codebook_bits;            /* b_c: 16 (fp16), 8 (int8) or 4 (INT4_G128)            */
  int64_t indices_per_row;          /* K/d                                                  */
  int64_t row_stride_bytes;         /* bytes between consecutive rows of the index stream   */
  int64_t index_bytes;              /* N * row_stride_bytes                                 */
  int64_t n_blocks;                 /* (N/block_rows) * (K/block_cols)                      */
  int64_t codebook_bytes_per_block; /* k * d * b_c/8                                        */
  int64_t codebook_bytes;           /* n_blocks * codebook_bytes_per_block                  */
  int64_t scale_bytes;              /* INT8_SCALED 2*n_blocks; INT4_G128 2*N*K/128; FP16 0  */
  int64_t total_bytes;              /* index + codebook + scale bytes                       */
  double bpv_paper;                 /* log2(k)/d + k*d*b_c/l  (no scale term)               */
  double bpv_stored;                /* 8*total_bytes/(N*K), everything stored               */
} vq_pack_info_t;

/* Sizes and bits-per-value of a format (paper Sec. 4, total bits per value; Sec. 3.1 tuple).
 * Host only, no CUDA call.  Errors: NULL, FORMAT, SHAPE. */
vq_status vq_pack_info(const vq_format* fmt, vq_pack_info_t* out);

/* Bytes of device scratch the GEMV/GEMM entry points need for (fmt, batch): arrival counters
 * (one 32-bit word per 16 rows, at the start) and room for the fp32 partial sums of column
 * ranges handled by different thread blocks (Sec. 3.2 mat-vec; the split is this library's).
 * Host only.  Returns 0 for an invalid format or batch.  See WORKSPACE above for the zero rule. */
size_t vq_workspace_bytes(const vq_format* fmt, int batch);

/* Materialise W: unpack every index and look its entry up (paper App. A: the quantized matrix Q
 * is the codebook C read through the index array; Sec. 3.2 decode step; App. B transfer+decode).
 *   d_idx, d_cb, d_scale : device, layouts above; d_scale NULL iff cb_type == VQ_CB_FP16.
 *   d_W   : device, binary16 [N][K] row-major, written completely.
 * FP16 codebooks are copied bit-exactly; INT8_SCALED values are fp32(scale)*int8 rounded once
 * to binary16 (round-to-nearest-even).  Errors: NULL, FORMAT, SHAPE, ALIGN, CUDA. */
vq_status vq_decode_weights(const vq_format* fmt, const void* d_idx, const void* d_cb,
                            const void* d_scale, void* d_W, void* stream);

/* y = W x for one token (paper Sec. 3.2: indices -> LUT -> values -> matrix-vector product).
 *   d_x : device binary16 [K];  d_y : device binary16 [N], written completely.
 *   d_ws / ws_bytes : device scratch of at least vq_workspace_bytes(fmt, 1) bytes, 16-byte
 *                     aligned, zero-filled once before its first use (WORKSPACE above).
 * Errors: NULL, FORMAT, SHAPE, ALIGN, WORKSPACE, CUDA. */
vq_status vq_gemv(const vq_format* fmt, const void* d_idx, const void* d_cb, const void* d_scale,
                  const void* d_x, void* d_y, void* d_ws, size_t ws_bytes, void* stream);

/* Y[m][n] = sum_k W[n][k] X[m][k] for batch = 1..16 token rows (same passage as vq_gemv).
 *   d_X : device binary16 [batch][K];  d_Y : device binary16 [batch][N].
 *   workspace of at least vq_workspace_bytes(fmt, batch) bytes.
 * Errors: as vq_gemv plus BATCH. */
vq_status vq_gemm_small_batch(const vq_format* fmt, const void* d_idx, const void* d_cb,
                              const void* d_scale, const void* d_X, void* d_Y, int batch,
                              void* d_ws, size_t ws_bytes, void* stream);

/* Same computation as vq_gemm_small_batch with the kernel family chosen by the caller
 * (vq_impl); used by the tests to exercise every kernel against the oracle.
 * Errors: as vq_gemm_small_batch plus UNSUPPORTED. */
vq_status vq_gemm_small_batch_impl(const vq_format* fmt, const void* d_idx, const void* d_cb,
                                   const void* d_scale, const void* d_X, void* d_Y, int batch,
                                   void* d_ws, size_t ws_bytes, void* stream, int impl);

/* Several layers that read the SAME activations in one call - the q/k/v or the gate/up projections of
 * a transformer block (paper Sec. 3.2: every linear layer of a token step streams its own weights;
 * grouping is this library's): Y_i[m][n] = sum_k W_i[n][k] X[m][k] for i < n_members.
 *   fmt       : the members' common format and K; fmt->n_rows = the SUM of the members' rows
 *               (it sizes the workspace: vq_workspace_bytes(fmt, batch)).
 *   members   : HOST array of n_members (1..VQ_MAX_GROUP) entries; each holds the member's device
 *               pointers (layouts as for vq_gemm_small_batch), its output d_Y (binary16
 *               [batch][n_rows]) and its row count (a multiple of block_rows).
 *   d_X       : device binary16 [batch][K], shared by all members.
 * One kernel serves the whole group where the persistent kernel, the shared-codebook kernels or the
 * pair-table kernel cover the format (vq_grouped_kernel_launches tells); otherwise the members run one
 * after the other on `stream`.  Results are the same as n_members separate calls.
 * Errors: as vq_gemm_small_batch; SHAPE also if the rows do not add up to fmt->n_rows. */
#define VQ_MAX_GROUP 4
typedef struct {
  const void* d_idx;
  const void* d_cb;
  const void* d_scale;   /* NULL iff cb_type == VQ_CB_FP16 */
  void* d_Y;
  int32_t n_rows;
} vq_group_member;
vq_status vq_gemm_small_batch_grouped(const vq_format* fmt, const vq_group_member* members, int n_members,
                                      const void* d_X, int batch, void* d_ws, size_t ws_bytes, void* stream);
/* Kernels a grouped call of this format launches: 1 (one kernel for the group) or n_members.
 * Host only; 0 for invalid arguments. */
int vq_grouped_kernel_launches(const vq_format* fmt, int n_members, int batch);

/* Same computation with HOST activations and outputs: copies h_X (binary16 [batch][K]) to the
 * device, runs vq_gemm_small_batch, copies Y back into h_Y (binary16 [batch][N]); all three
 * steps are enqueued on `stream` and the call returns without synchronising, so the caller
 * must synchronise the stream before reading h_Y.  Pinned host memory keeps the copies
 * asynchronous; when both buffers are pinned (page-locked and mapped, as cudaHostAlloc and
 * cudaHostRegister make them) and 16-byte aligned, a small kernel fetches X and the mat-vec
 * kernel stores Y directly into h_Y instead of the two copies (same results, no hand-over to
 * the copy engines).  The compressed weights stay resident on the device (paper Sec. 1: every
 * weight is read once per generated token; only activations cross the host boundary).
 *   d_ws must hold vq_workspace_bytes(fmt, batch) + 2*batch*(K+N) bytes rounded up to 256:
 *   use vq_workspace_bytes_host(fmt, batch).
 * Errors: as vq_gemm_small_batch. */
vq_status vq_gemm_small_batch_host(const vq_format* fmt, const void* d_idx, const void* d_cb,
                                   const void* d_scale, const void* h_X, void* h_Y, int batch,
                                   void* d_ws, size_t ws_bytes, void* stream);
size_t vq_workspace_bytes_host(const vq_format* fmt, int batch);

/* vq_gemm_small_batch_grouped with HOST activations and outputs: h_X (binary16 [batch][K]) is brought to
 * the device once for the whole group, every member's result goes back to the HOST buffer its d_Y field
 * names (binary16 [batch][n_rows]; in this call d_Y is a host pointer).  Steps are enqueued on `stream`, the
 * call returns without synchronising; pinned buffers take the same direct path as
 * vq_gemm_small_batch_host (paper Sec. 1 / Sec. 3.2: per generated token only activations cross the host
 * boundary, the weights stay on the device).
 *   d_ws : at least vq_workspace_bytes_grouped_host(fmt, n_members, batch) bytes, rules as WORKSPACE above.
 * Errors: as vq_gemm_small_batch_grouped. */
vq_status vq_gemm_small_batch_grouped_host(const vq_format* fmt, const vq_group_member* members, int n_members,
                                           const void* h_X, int batch, void* d_ws, size_t ws_bytes, void* stream);
size_t vq_workspace_bytes_grouped_host(const vq_format* fmt, int n_members, int batch);

/* The same computation as vq_gemm_small_batch_host for callers that cannot allocate device memory
 * at all: code that runs where cudaMalloc is forbidden or unavailable - inside a region whose
 * memory is owned and budgeted by another allocator (an inference server's arena, a real-time
 * loop that may not block on the driver's allocator), or a plug-in that is handed device
 * pointers to the weights but no allocator.  (The paper has no counterpart: this is a packaging
 * variant of the entry point above, not a step of the method.)
 * Instead of a caller-provided workspace, the device copies of X and Y live in a fixed array of
 * vq_static_scratch_bytes() = 2 MiB that is part of the library image; every GPU that loads the
 * library holds it until the process exits.  The call performs no cudaMalloc / cudaFree and calls
 * no allocating routine.
 *   Limit: round256(2*batch*K) + round256(2*batch*N) must not exceed vq_static_scratch_bytes();
 *   larger problems return VQ_ERR_WORKSPACE and launch nothing.
 *   The first call on each device looks the array's device address up (cudaGetSymbolAddress, with
 *   that device current); make that first call outside any stream capture.
 *   All calls on a device share the one array, which keeps the previous call's contents; nothing
 *   in it has to be cleared between calls (X is overwritten by the copy in, Y by the kernel).
 *   Two calls that may overlap on the GPU (different streams, no ordering between them) race on
 *   it: order them on one stream or with events.
 *   As with vq_gemm_small_batch_host the three steps are enqueued on `stream` and the call
 *   returns without synchronising; synchronise before reading h_Y.
 * Errors: NULL, FORMAT, SHAPE, ALIGN, BATCH, WORKSPACE (problem larger than the scratch), CUDA. */
vq_status vq_gemm_small_batch_host_static(const vq_format* fmt, const void* d_idx, const void* d_cb,
                                          const void* d_scale, const void* h_X, void* h_Y, int batch,
                                          void* stream);
size_t vq_static_scratch_bytes(void);

/* Uniform INT4 group-128 reference GEMV used as the bandwidth yard-stick beside the VQ
 * kernels (paper Sec. 2.1 symmetric uniform quantiser x ~ s*x_int; Sec. 5 compares against uniform
 * 4-bit weights with one scale per 128 columns, 4.125 bits per value).
 *   d_q     : device, N rows of K/2 bytes; column k of row n is nibble (k mod 2) of byte k/2
 *             (low nibble first); stored value q in 0..15 means integer q-8.
 *   d_scale : device binary16 [N][K/128];  w[n][k] = scale[n][k/128] * (q-8).
 *   d_X binary16 [batch][K], d_Y binary16 [batch][N], batch 1..16.  K % 128 == 0, K/2 % 16 == 0.
 *   d_ws / ws_bytes : at least vq_int4g128_workspace_bytes(n_rows, batch) bytes, rules as WORKSPACE above.
 * Errors: NULL, SHAPE, ALIGN, BATCH, WORKSPACE, CUDA. */
vq_status vq_int4g128_gemm_small_batch(int32_t n_rows, int32_t k_cols, const void* d_q,
                                       const void* d_scale, const void* d_X, void* d_Y,
                                       int batch, void* d_ws, size_t ws_bytes, void* stream);
size_t vq_int4g128_workspace_bytes(int32_t n_rows, int batch);

/* E-step / VQ_quant of the quantizer (paper Sec. 3, Eq. 5; Algorithm 2's quantization step): for
 * every d-vector x of the dense matrix W (d adjacent columns of one row) the index m of the centroid
 * of its block that minimises (x - c_m)^T D (x - c_m), written in the packed index format above so
 * that vq_decode_weights / vq_gemm_small_batch read the result directly.
 *   d_W     : device binary16 [N][K].
 *   d_cb, d_scale : the codebooks to assign to, layouts above.
 *   d_hdiag : device binary32 [K], the diagonal of D (1 / [H^-1]_kk per column), or NULL for the
 *             identity (plain nearest centroid).  16-byte aligned.
 *   d_idx   : device, OUTPUT, N rows of row_stride_bytes; padding bytes are written as zero.
 * The decision is taken in binary32, each operation rounded separately, terms added in column
 * order; among equal distances the lowest index wins.
 * Covered: formats with a whole number of 8-index groups per row (K / d % 8 == 0), block_cols a
 * power of two >= 8 d, block_rows dividing or divided by 32; others return VQ_ERR_UNSUPPORTED.
 * Errors: NULL, FORMAT, SHAPE, ALIGN, UNSUPPORTED, CUDA. */
vq_status vq_assign_indices(const vq_format* fmt, const void* d_W, const void* d_cb,
                            const void* d_scale, const void* d_hdiag, void* d_idx, void* stream);

/* Block-wise data normalisation applied at the decode step (paper appendix "Blockwise data
 * normalization": every sub-row of a codebook group is divided by a scale before clustering, the scale is
 * stored as a 4-bit integer on a log2 grid, and the inverse scaling is applied when the weights are decoded).
 * Layout fixed by this library (the paper's formula for the grid is garbled and it fixes no layout):
 *   norm_block_cols : columns per sub-row (the paper names 16, 32, 64); divides block_cols, multiple of vq_dim.
 *   d_norm_codes    : device, one 4-bit code per row and sub-row, two per byte, low nibble = lower sub-row;
 *                     rows start every vq_norm_info().code_row_bytes = ceil(K / norm_block_cols / 2) bytes.
 *   d_norm_lut      : device binary16 [blocks][16], blocks ordered as the codebooks: the 16 scales a code of
 *                     that codebook block can stand for (on the paper's grid: 2^(a * code + z) with the
 *                     group's step a and offset z; the decoder needs the values only).
 *   w[n][k] = value decoded as without normalisation * d_norm_lut[blk(n, k)][code(n, k / norm_block_cols)].
 * vq_decode_weights_normalized writes binary16(w), the exact product rounded once; vq_gemm_small_batch_normalized
 * computes Y[m][n] = sum_k w[n][k] X[m][k] (fp32 accumulation, one rounding), batch 1..16.  Every valid
 * format is taken (format-generic kernels; no workspace, plain stream-order launches); the product runs in
 * the tuned pair-table kernel when the format is one of its (see vq_impl), the codebooks are fp16 or int8
 * and norm_block_cols is a power of two of at least 16 (weights then enter the sum as binary16 values);
 * the decode runs in the tile kernel of vq_decode_weights for the formats that one takes and power-of-two
 * sub-rows of at least 8 columns, bit-identical to the format-generic kernel.
 * Errors: as vq_decode_weights / vq_gemm_small_batch (without WORKSPACE); NULL for a missing code or table
 * pointer; SHAPE for a norm_block_cols that does not divide block_cols or is not a multiple of vq_dim. */
typedef struct {
  size_t code_row_bytes;   /* bytes between rows of d_norm_codes                    */
  size_t codes_bytes;      /* n_rows * code_row_bytes                                */
  size_t lut_bytes;        /* blocks * 16 * 2                                        */
} vq_norm_info_t;
vq_status vq_norm_info(const vq_format* fmt, int norm_block_cols, vq_norm_info_t* out);
vq_status vq_decode_weights_normalized(const vq_format* fmt, const void* d_idx, const void* d_cb, const void* d_scale,
                                       const void* d_norm_codes, const void* d_norm_lut, int norm_block_cols, void* d_W,
                                       void* stream);
vq_status vq_gemm_small_batch_normalized(const vq_format* fmt, const void* d_idx, const void* d_cb, const void* d_scale,
                                         const void* d_norm_codes, const void* d_norm_lut, int norm_block_cols, const void* d_X,
                                         void* d_Y, int batch, void* stream);

/* Uniformly quantized weights expanded to binary16: the yard-sticks of the transfer + decode
 * experiment (paper App. B: time to move and unpack a layer stored as FP16, INT8, INT4 or VQ),
 * timed beside vq_decode_weights.  w = s * q (Sec. 2.1), exact product rounded once to binary16.
 *   kind VQ_UNPACK_FP16     : d_src binary16 [N][K], d_scale NULL; a copy.
 *   kind VQ_UNPACK_INT8_ROW : d_src signed 8-bit q [N][K]; d_scale binary16 [N], one per row.
 *   kind VQ_UNPACK_INT4_G128: d_src and d_scale as for vq_int4g128_gemm_small_batch (q-8).
 *   d_W : device binary16 [N][K], written completely.  K % 128 == 0; pointers 16-byte aligned.
 * Errors: NULL, FORMAT (unknown kind), SHAPE, ALIGN, CUDA. */
typedef enum { VQ_UNPACK_FP16 = 0, VQ_UNPACK_INT8_ROW = 1, VQ_UNPACK_INT4_G128 = 2 } vq_unpack_kind;
vq_status vq_unpack_uniform(int kind, int32_t n_rows, int32_t k_cols, const void* d_src,
                            const void* d_scale, void* d_W, void* stream);

/* Probes behind the ceilings bench.py prints beside the achieved bandwidth (paper Sec. 3.2: the decode
 * must keep up with DRAM; these measure what the decode loop and a plain read can do on this GPU).
 * vq_probe_decode_loop: `iters` passes of the look-up + multiply-accumulate loop of one kernel policy
 *   over a stage that stays in shared memory (no global traffic), on every SM, `warps` (1..8) warps per
 *   SM, batch 1..8.  policy 0: 2-D 4-bit per-row codebooks, 1: 1-D 4-bit int8 codebooks, 2: uniform
 *   INT4 g128, 3: 2-D 6-bit shared codebooks.  d_scratch: device memory of at least
 *   8*SMs + 128*SMs*warps bytes.  Returns the average clocks per pass and the weights one pass decodes
 *   on one SM; synchronises `stream`.
 * vq_probe_read: reads every byte of d_buf once with streaming 128-bit loads; asynchronous on `stream`,
 *   the caller times it.  d_out4: 4 writable device bytes.
 * Errors: NULL, SHAPE, ALIGN, WORKSPACE, UNSUPPORTED, CUDA. */
vq_status vq_probe_decode_loop(int policy, int warps, int batch, int iters, void* d_scratch, size_t scratch_bytes,
                               double* h_clocks, double* h_weights_per_pass, void* stream);
vq_status vq_probe_read(const void* d_buf, size_t bytes, void* d_out4, void* stream);

/* Diagnostics.  The tuned kernels wait for their asynchronous copies (Sec. 3.2 index stream) with a
 * bounded number of polls; a wait that runs out increments a per-device counter and the kernel
 * carries on (its output is then wrong, but the device stays usable).  This call copies the
 * counter of the current device to *h_count; it synchronises the device.  0 in a healthy run.
 * Errors: NULL, CUDA. */
vq_status vq_device_wait_failures(int* h_count);

/* Human-readable name of a status code; never NULL. */
const char* vq_status_string(vq_status s);

#ifdef __cplusplus
}
#endif
#endif /* VQ_B200_H */
