/*
 * libkmq -- k-means-quantised linear layer for NVIDIA B200 (sm_100a).
 *
 * The layer is y = x * W^T with W^[n,k] = C_n[idx[n,k]]: every weight is a
 * b-bit index (b = 1, 2 or 4) into the 2^b-entry bf16 codebook of its output
 * row n.  This is the fused dequantise-multiply Y^T = dequantize(W~) X^T of
 * the paper's Appendix "Benchmarking" ("Kernel implementations": gather the
 * decoded values from a lookup table, then x @ W.T), with the lookup table
 * held per output row and no block scales; the indices come from the
 * nearest-centroid quantiser f_c(x) = argmin_i |x - c_i| (Section 2.1,
 * "Rounding to nearest centroids").
 *
 * Conventions shared by every entry point
 *   - Pointers marked DEVICE are CUDA device pointers valid on the current
 *     device; HOST pointers are ordinary (ideally pinned) host memory.  The
 *     caller owns every buffer.  The library allocates no memory.  The state
 *     it keeps per device: a cache of device properties and of a few symbol
 *     addresses, two sticky error words in device memory (see
 *     kmq_device_error_flags) and the fixed 512 KiB scratch array of
 *     kmq_linear_static_scratch, which is part of the library image.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Work is enqueued on it and the call returns without synchronising,
 *     unless stated otherwise.
 *   - Arguments are validated on the host before anything is launched.  A
 *     failed check returns a status and launches nothing.  Nothing aborts,
 *     throws, or asserts on the device.
 *   - bf16 values are passed as uint16_t bit patterns.
 *   - Shapes: N output rows, K input features, M batch rows.  N, M >= 1;
 *     K >= 32/bits and K % (32/bits) == 0.  Buffers must not overlap.
 *   - Packed layouts.  With wpr = K*bits/32 words per row, word j of row n
 *     holds the 32/bits indices idx[n, j*(32/bits) + i], i = 0..32/bits-1.
 *     KMQ_LAYOUT_CANONICAL (the interchange format): row-major uint32 [N, wpr],
 *     field i of a word at bits [i*bits, (i+1)*bits), fields LSB first.
 *     KMQ_LAYOUT_TUNED (what the fast kernels read; the paper names an
 *     "optimized data layout" as the way to reach bandwidth, Appendix
 *     "Benchmarking", "Micro-benchmarks"): tile-major.  Rows are grouped in
 *     tiles of 16 and the words of a row in steps of 16; with steps =
 *     ceil(wpr/16), word (n, j) is stored at word index
 *       (((n/16)*steps + j/16)*16 + n%16)*16 + j%16,
 *     so one step of one tile is a contiguous 1 KB block; rows beyond N and
 *     words beyond wpr are zero padding (kmq_packed_bytes gives the padded
 *     size).  Inside a word the fields sit where the tensor-core kernels can
 *     extract four consecutive weights with the fewest integer instructions:
 *       bits = 4: field i at bits [4i, 4i+4) (as canonical);
 *       bits = 2: field i = 4p + c (p, c in 0..3) at bits [2p + 8c, 2p + 8c + 2);
 *       bits = 1: field i = 2c at bit 15 - c, field i = 2c + 1 at bit 31 - c.
 *     KMQ_LAYOUT_TABLE (what the activation-table kernel reads: b = 1, 2 at
 *     the smallest batches; for bits = 4 it is identical to KMQ_LAYOUT_TUNED):
 *     bit planes.  Plane p holds bit p of every index, one byte per group of 8
 *     consecutive weights of a row, weight 8g + t in bit t.  Rows are grouped
 *     in tiles of 16 and the groups of a row in chunks of 32 (256 weights);
 *     with chunks = ceil(K/256), plane p of chunk c of tile T is one
 *     contiguous 512-byte unit at byte ((T*chunks + c)*bits + p)*512, and
 *     inside a unit the byte of row n, group g is at
 *       (2*(n%16) + g%2)*16 + ((g%32)/2 - n%16) mod 16.
 *     Rows beyond N and groups beyond K are zero padding.
 *     kmq_packed_bit_index() gives the position of any index bit in any layout.
 *     Every entry point accepts every layout; kmq_pack writes the one asked
 *     for, the others must be told which one `packed` is in.  Which layout is
 *     fastest depends on the batch: kmq_preferred_layout().
 *   - All device pointers must be 16-byte aligned.
 */
#ifndef KMQ_H_
#define KMQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KMQ_OK = 0,
  KMQ_ERR_NULL = 1,      /* a required pointer is NULL */
  KMQ_ERR_BITS = 2,      /* bits is not 1, 2 or 4 */
  KMQ_ERR_SHAPE = 3,     /* N, K or M out of range, or K not a multiple of 32/bits */
  KMQ_ERR_ALIGN = 4,     /* a device pointer is not 16-byte aligned */
  KMQ_ERR_WORKSPACE = 5, /* workspace missing or smaller than kmq_workspace_bytes() */
  KMQ_ERR_LAYOUT = 6,    /* unknown layout id */
  KMQ_ERR_CUDA = 7,      /* the CUDA runtime reported an error (launch, copy) */
  KMQ_ERR_SCRATCH_LIMIT = 8 /* kmq_linear_static_scratch: the shape needs more than the built-in scratch holds */
} kmq_status;

typedef enum {
  KMQ_LAYOUT_CANONICAL = 0,
  KMQ_LAYOUT_TUNED = 1,
  KMQ_LAYOUT_TABLE = 2
} kmq_layout;

/* Library version (major*10000 + minor*100 + patch). */
int kmq_version(void);

/* Static, NUL-terminated description of a status code. */
const char* kmq_status_string(int status);

/* Bytes of the packed index matrix: N * K * bits / 8 (canonical) or the padded
 * tile-major size (tuned); 0 if the arguments are invalid. */
size_t kmq_packed_bytes(int64_t N, int64_t K, int bits, int layout);

/* Where the packed layouts put things (host-side arithmetic, no GPU involved):
 * kmq_packed_word_index -- index, in 32-bit words from the start of the packed
 * buffer, of word j of row n; kmq_packed_field_shift -- bit position of field i
 * (index idx[n, j*(32/bits) + i]) inside that word.  -1 for invalid arguments. */
int64_t kmq_packed_word_index(int64_t n, int64_t j, int64_t N, int64_t K, int bits, int layout);
int kmq_packed_field_shift(int i, int bits, int layout);

/* Position, in bits from the start of the packed buffer (bit b of byte B is
 * position 8B + b; bytes of a 32-bit word little-endian), of bit `plane`
 * (0 = least significant) of idx[n, k].  Valid for every layout; the two
 * functions above describe the word-based layouts only and return -1 for
 * KMQ_LAYOUT_TABLE at bits = 1, 2.  -1 for invalid arguments. */
int64_t kmq_packed_bit_index(int64_t n, int64_t k, int plane, int64_t N, int64_t K, int bits, int layout);

/* The layout in which kmq_linear is fastest for this shape and batch on the
 * current device (KMQ_LAYOUT_TABLE or KMQ_LAYOUT_TUNED). */
int kmq_preferred_layout(int64_t N, int64_t K, int bits, int64_t M);

/* Bytes of scratch kmq_linear needs for this shape on the current device
 * (fp32 partial sums of a split along K); may be 0. */
size_t kmq_workspace_bytes(int64_t N, int64_t K, int bits, int64_t M, int layout);

/* Number of kernels one kmq_linear call launches for this shape (one per pass
 * of batch rows; 2 for the balanced split with its fix-up kernel), and a short
 * static name of the kernel variant the dispatcher picks: "tiled_*",
 * "split_*", "multi_*", "tcgen05_*" (tuned layout), "table_*" (table layout,
 * bits = 1, 2), "staged_*" (canonical layout),
 * "generic_warp_per_row", or "invalid". */
int kmq_linear_num_launches(int64_t N, int64_t K, int bits, int64_t M, int layout);
const char* kmq_linear_variant(int64_t N, int64_t K, int bits, int64_t M, int layout);

/*
 * kmq_pack -- bit-pack centroid indices along K (the paper stores the
 * quantised elements packed along the input dimension; Appendix
 * "Benchmarking", "Kernel implementations").
 *   idx    DEVICE uint8 [N, K] row-major; only the low `bits` bits are kept.
 *   packed DEVICE uint32, kmq_packed_bytes() bytes, written in `layout`.
 */
kmq_status kmq_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, int layout,
                    uint32_t* packed, void* stream);

/* kmq_unpack -- inverse of kmq_pack: idx DEVICE uint8 [N, K] is written. */
kmq_status kmq_unpack(const uint32_t* packed, int64_t N, int64_t K, int bits, int layout,
                      uint8_t* idx, void* stream);

/*
 * kmq_linear -- y[m,n] = sum_k x[m,k] * C_n[idx[n,k]], bf16 products
 * accumulated in fp32, result rounded to bf16 (round-to-nearest-even).
 * (Appendix "Benchmarking": Y^T = dequantize(W~) X^T; Appendix "Theoretical
 * model of software-decoded formats": Y^T = W X^T with X, Y of shape m x h.)
 *   packed    DEVICE uint32, kmq_packed_bytes() bytes, in `layout`.
 *   codebooks DEVICE bf16 [N, 2^bits] row-major, C_n[i] at n*2^bits + i.
 *   x         DEVICE bf16 [M, K] row-major.
 *   y         DEVICE bf16 [M, N] row-major, fully overwritten.
 *   workspace DEVICE, at least kmq_workspace_bytes(N,K,bits,M,layout) bytes; may be
 *             NULL when that is 0.  Contents on entry are ignored, contents on
 *             return are unspecified.  Calls that share a workspace must not
 *             overlap on the GPU.
 *   packed and codebooks are treated as constants of the layer: the kernels
 *             may read them before earlier work on `stream` has finished
 *             (programmatic dependent launch).  Earlier kernels of this
 *             library and ordinary kernels that write them are still ordered
 *             before the read; a foreign kernel that itself signals an early
 *             launch of its dependents must not be the one that writes them.
 * The order of the fp32 summation is fixed for a given shape and device, so
 * repeated calls give bit-identical results.  Outputs for non-finite inputs
 * are unspecified.
 * The return value covers validation and the launch itself.  The variants
 * "tcgen05_*" and "table_*" (see kmq_linear_variant) wait on hardware
 * barriers for asynchronous copies and matrix instructions; those waits are
 * bounded, and one that runs out (which takes a GPU that has stopped
 * delivering) leaves y incomplete and is reported only through
 * kmq_device_error_flags(), which synchronises the device.
 */
kmq_status kmq_linear(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x,
                      uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, int layout,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * kmq_linear_host -- the same layer for a caller whose activations live in
 * host memory: copies x (HOST bf16 [M,K]) into x_dev, runs kmq_linear, copies
 * y_dev into y (HOST bf16 [M,N]) and synchronises `stream` before returning.
 * The weights (packed, codebooks) stay resident on the device.
 *   x_dev, y_dev  DEVICE staging buffers of M*K*2 and M*N*2 bytes.
 */
kmq_status kmq_linear_host(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x_host,
                           uint16_t* y_host, int64_t N, int64_t K, int bits, int64_t M, int layout,
                           uint16_t* x_dev, uint16_t* y_dev, void* workspace, size_t workspace_bytes,
                           void* stream);

/*
 * kmq_linear_static_scratch -- kmq_linear without a workspace argument, for
 * callers that are not allowed to allocate device memory: code inside a region
 * where the allocator must not be entered (a latency-critical loop, a
 * non-blocking callback), or a component that owns nothing but the buffers it
 * was given.  (This is a convenience of this library; the paper has no
 * counterpart.)  Same arguments, result and errors as kmq_linear.  Where
 * kmq_linear would need scratch (kmq_workspace_bytes() > 0) the partial sums
 * go to a fixed 512 KiB array that is part of the library image on every GPU
 * that loads it (kmq_static_scratch_capacity() returns the size); a shape that
 * needs more is refused with KMQ_ERR_SCRATCH_LIMIT and nothing is launched.
 * The call never allocates or frees memory.
 *   - The first call on each device looks up the array's device address
 *     (once, with that device current); make that first call outside any
 *     stream capture.
 *   - All calls on a device share the one array.  Calls whose kernels may
 *     overlap on the GPU (different streams, or graph branches) race on it:
 *     serialise them.  Its contents between calls are meaningless and never
 *     need clearing: each call writes every word it later reads.
 */
kmq_status kmq_linear_static_scratch(const uint32_t* packed, const uint16_t* codebooks,
                                     const uint16_t* x, uint16_t* y, int64_t N, int64_t K, int bits,
                                     int64_t M, int layout, void* stream);
size_t kmq_static_scratch_capacity(void);

/*
 * kmq_linear_tcgen05 -- the same layer (same operands, result and tolerance
 * as kmq_linear) computed by the 5th-generation tensor-core path: weights of
 * 128 output rows are dequantised straight into tensor memory as the A
 * operand of tcgen05.mma, the activations are the B operand in shared
 * memory, the accumulator lives in tensor memory.  `packed` must be in
 * KMQ_LAYOUT_TUNED and K * bits a multiple of 128; any M >= 1 (128 batch rows
 * per launch).  This is the large-batch design the paper's roofline model
 * points to (Appendix "Theoretical model": beyond a batch of P_w * nu / 16
 * the layer is compute bound).  One tcgen05.mma (2048 weights) costs 70 to
 * 100 clocks whatever the batch, so the time does not depend on M up to 128
 * rows but a CTA covers 128 output rows: kmq_linear itself selects this
 * kernel for M > 32 (b = 1: M > 16) on shapes with enough 128-row blocks to
 * occupy most SMs
 * (kmq_linear_variant() then starts with "tcgen05"); this entry point forces
 * it for any shape.
 * It needs no workspace.  Its waits on hardware barriers are bounded, see
 * kmq_device_error_flags.
 * Errors: KMQ_ERR_NULL, KMQ_ERR_BITS, KMQ_ERR_SHAPE, KMQ_ERR_ALIGN,
 * KMQ_ERR_CUDA.
 */
kmq_status kmq_linear_tcgen05(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x,
                              uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, void* stream);

/*
 * kmq_device_error_flags -- error word of the kernels on the current device.
 * The tensor-memory kernel ("tcgen05_*" variants, kmq_linear_tcgen05) and the
 * table kernel ("table_*" variants) wait on hardware barriers for asynchronous
 * matrix instructions and bulk copies; every such wait gives up after 100 ms
 * on the GPU's global timer, and a warp whose wait runs out stops, stores
 * nothing more and sets bit 0 here; the CTA still frees its tensor memory
 * (the outputs of that call are then incomplete).  The call synchronises the
 * device, writes the word to *flags (host pointer) and clears it.  0 = no
 * kernel gave up since the last call.
 * Errors: KMQ_ERR_NULL, KMQ_ERR_CUDA.
 */
#define KMQ_DEVICE_ERROR_WAIT_TIMEOUT 1u
#define KMQ_DEVICE_ERROR_SMEM_WINDOW 2u /* the table kernel found its shared memory outside the fixed address window it needs; it stored nothing */
kmq_status kmq_device_error_flags(unsigned int* flags);

/*
 * kmq_dequant_to_bf16 -- materialise W^[n,k] = C_n[idx[n,k]] as a dense bf16
 * matrix; every element is a bit-exact copy of a stored centroid.  This is
 * the separate dequantise step the paper suggests ahead of a standard GEMM
 * at large batch sizes and prefill (Appendix "Benchmarking", "Model
 * benchmarks").
 *   W  DEVICE bf16 [N, K] row-major, fully overwritten.
 */
kmq_status kmq_dequant_to_bf16(const uint32_t* packed, const uint16_t* codebooks, uint16_t* W,
                               int64_t N, int64_t K, int bits, int layout, void* stream);

/*
 * The paper's own k-means block format (Section 2.1 "Block formats", Eq.
 * "fractional bit width"; Section 2.2 "Nonlinear k-means quantization";
 * Appendix "Benchmarking", "Kernel implementations"): one codebook of 2^bits
 * centroids per weight tensor (bits = 1, 2, 4 or 8) and one bf16 scale per
 * block of 64 consecutive inputs of an output row,
 *     W^[n, k] = scale[n, k/64] * c[idx[n, k]],     P_w = bits + 16/64 bits per weight.
 *   wq       DEVICE uint8 [N, K*bits/8] row-major: the indices packed along the
 *            input dimension, 8/bits per byte, field i of a byte at bits
 *            [i*bits, (i+1)*bits) (the paper leaves the order inside a byte
 *            open; LSB first is the reading taken here).
 *   scales   DEVICE bf16 [N, K/64] row-major.
 *   codebook DEVICE bf16 [2^bits].
 * K must be a multiple of 64; all pointers 16-byte aligned.
 *
 * kmq_block_pack -- idx DEVICE uint8 [N, K] (low `bits` bits kept) -> wq.
 * kmq_block_linear -- y[m,n] = sum_k x[m,k] * W^[n,k], fp32 accumulation,
 *   bf16 result.  scale_order picks between the paper's two listings:
 *   KMQ_SCALE_DIRECT multiplies every centroid by its block's scale before the
 *   multiply-accumulate; KMQ_SCALE_DEFERRED ("deferred scaling") accumulates
 *   the 64 unscaled products of a block and scales their sum.  Both are the
 *   same sum up to fp32 rounding and both meet the tolerance stated for
 *   kmq_linear.  x DEVICE bf16 [M,K], y DEVICE bf16 [M,N]; no workspace.
 * kmq_block_dequant_to_bf16 -- W DEVICE bf16 [N,K] = bf16(scale * centroid):
 *   the exact product rounded once, to nearest even (the separate dequantise
 *   step ahead of a standard GEMM, Appendix "Benchmarking", "Model benchmarks").
 * Errors: KMQ_ERR_NULL, KMQ_ERR_BITS, KMQ_ERR_SHAPE, KMQ_ERR_ALIGN,
 * KMQ_ERR_LAYOUT (unknown scale_order), KMQ_ERR_CUDA.
 */
#define KMQ_SCALE_DIRECT 0
#define KMQ_SCALE_DEFERRED 1
size_t kmq_block_packed_bytes(int64_t N, int64_t K, int bits);
kmq_status kmq_block_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, uint8_t* wq, void* stream);
kmq_status kmq_block_linear(const uint8_t* wq, const uint16_t* scales, const uint16_t* codebook, const uint16_t* x,
                            uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, int scale_order, void* stream);
kmq_status kmq_block_dequant_to_bf16(const uint8_t* wq, const uint16_t* scales, const uint16_t* codebook, uint16_t* W,
                                     int64_t N, int64_t K, int bits, void* stream);

/*
 * The block format through an activation table (b = 1, 2, 4; decode batches).
 * With one codebook for the whole tensor, a 256-entry table per byte of packed
 * indices can hold finished partial dot products of the activations with the
 * centroids (the byte table of the paper's listing, Appendix "Benchmarking",
 * "Kernel implementations", built over x instead of over the weights); the layer
 * is then one shared-memory lookup per byte of weights and one multiply-add per
 * block (deferred scaling).  The kernel reads its own layout, which holds the
 * index bytes and the block scales of 16 rows x 32 bytes side by side:
 *   unit (tile T = n / 16, chunk c = byte / 32) at byte offset
 *   (T * chunks + c) * (512 + 32 * (4 / bits)),  chunks = ceil(K * bits / 256);
 *   512 index bytes, then the bf16 scales scale[row r][block q of the chunk] at
 *   512 + (r * (4 / bits) + q) * 2.  Lane L = 2 r + a owns the index bytes
 *   [16 L, 16 L + 16); with S = 4 * bits, r = r_hi * S + r_lo, byte i = S * j + f
 *   of the lane holds byte number
 *   (8 * bits) * ((j + r_hi) % (4 / bits)) + a + 2 * ((f + r_lo) % S)
 *   of the chunk of row 16 T + r.  Padding (rows >= N, bytes beyond K) is zero.
 * kmq_block_table_bytes -- size of the table layout (0 for invalid arguments).
 * kmq_block_table_index_offset / _scale_offset -- byte offset of the byte that
 *   holds the index of weight (n, k), and of the scale of its block (-1 for
 *   invalid arguments): the layout above as a function, for tools and tests.
 * kmq_block_table_pack -- (wq, scales) of kmq_block_pack's layout -> table.
 * kmq_block_table_unpack -- the inverse.
 * kmq_block_table_workspace_bytes -- scratch kmq_block_table_linear needs for
 *   this shape (0 when every CTA sees the whole of K).
 * kmq_block_table_linear -- y[m, n] = sum_k x[m, k] * scale[n, k/64] *
 *   c[idx[n, k]]: fp32 tables, fp32 accumulation, bf16 result, the tolerance
 *   stated for kmq_linear for any finite codebook (a table entry is the sum of
 *   the selected products themselves).  One pass over the weights per batch
 *   row: meant for M = 1 .. 4.  Two launches per pass when scratch is needed.
 *   Waits on copies are bounded; a run-out is reported by
 *   kmq_device_error_flags only.  Needs 227 KB of shared memory per CTA
 *   (KMQ_ERR_CUDA otherwise).
 * bits = 1, 2 or 4 (KMQ_ERR_BITS), K a multiple of 64, pointers 16-byte aligned.
 */
size_t kmq_block_table_bytes(int64_t N, int64_t K, int bits);
int64_t kmq_block_table_index_offset(int64_t n, int64_t k, int64_t N, int64_t K, int bits);
int64_t kmq_block_table_scale_offset(int64_t n, int64_t k, int64_t N, int64_t K, int bits);
kmq_status kmq_block_table_pack(const uint8_t* wq, const uint16_t* scales, int64_t N, int64_t K, int bits,
                                uint8_t* table, void* stream);
kmq_status kmq_block_table_unpack(const uint8_t* table, int64_t N, int64_t K, int bits, uint8_t* wq, uint16_t* scales,
                                  void* stream);
size_t kmq_block_table_workspace_bytes(int64_t N, int64_t K, int bits);
kmq_status kmq_block_table_linear(const uint8_t* table, const uint16_t* codebook, const uint16_t* x, uint16_t* y,
                                  int64_t N, int64_t K, int bits, int64_t M, void* workspace, size_t workspace_bytes,
                                  void* stream);

/*
 * The quantiser side: from float32 weights to codebooks, scales and packed
 * indices (Section 2.1 "Rounding to nearest centroids", Eq. "centroid
 * quantizer": f_c(x) = argmin_{c_i} |x - c_i|, the centroids "obtained
 * algorithmically by 1D k-means clustering"; "Block formats"; Section 2.2: the
 * scale functions absmax and absmean, "Nonlinear k-means quantization").  The
 * value Q(w) that quantisation-aware training substitutes for w in the forward
 * pass (Section 2.1, "Quantization-Aware Training") is what
 * kmq_dequant_to_bf16 / kmq_block_dequant_to_bf16 return for the output of
 * these calls.  Where the paper is silent the rules are: start at the 2^bits
 * linearly interpolated quantiles (i + 1/2) / 2^bits of the values; `iters`
 * Lloyd iterations (assign, then move each centroid to the float64 mean of its
 * values; an empty cluster keeps its centroid); a value half-way between two
 * centroids goes to the lower one; equal centroids are represented by the
 * lowest index; the stored centroid is the float64 mean rounded to float32 and
 * then to bf16, to nearest even, a zero of either sign as +0.  Weights must be
 * finite.
 *
 * kmq_kmeans_rows -- one fit per row.
 *   W          DEVICE float32 [N, K] row-major, read only.
 *   bits       1, 2, 4 or 8 (8 for the shared codebook of the block format).
 *   codebooks  DEVICE bf16 [N, 2^bits], non-decreasing along a row.
 *   centroids  DEVICE float64 [N, 2^bits] or NULL: the unrounded centroids.
 *   A row is sorted in shared memory: 2^bits <= K <= 32768, else KMQ_ERR_SHAPE.
 * kmq_assign_pack -- packed[n, k] = index of the centroid of codebooks[n, :]
 *   nearest to W[n, k], written directly in `layout` (the argument rules of
 *   kmq_pack).  Codebook rows must be non-decreasing (otherwise the indices are
 *   valid but need not be the nearest).  The decision is exact: no rounding is
 *   involved in comparing a weight with the midpoint of two stored centroids.
 * kmq_quantize_rows -- kmq_kmeans_rows, then kmq_assign_pack with the stored
 *   codebooks, on one stream.
 * kmq_block_scales -- scales[n, g] = bf16(lambda(W[n, 64g .. 64g+64))), lambda
 *   = max |w| (KMQ_LAMBDA_ABSMAX) or mean |w| (KMQ_LAMBDA_ABSMEAN, the 64
 *   magnitudes added in float64 in index order); a scale that would be stored
 *   as zero is stored as 1.  K a multiple of 64.
 * kmq_block_sample -- the normalised weights w / scale (float64 quotient with
 *   the stored scale, not clipped: within [-1, 1] up to the rounding of an
 *   absmax scale, beyond it under absmean) at the flat positions 0, s, 2s, ... with
 *   s = max(1, N*K / samples), the first kmq_block_sample_count(N, K, samples)
 *   of them, rounded to float32 into `out` (DEVICE): the values the shared
 *   codebook is fitted on (kmq_kmeans_rows with N = 1, bits up to 8).
 * kmq_block_assign_pack -- wq = the packed indices (layout of kmq_block_pack)
 *   of the centroid of `codebook` (DEVICE bf16 [2^bits], non-decreasing)
 *   nearest to each normalised weight.
 * kmq_block_quantize -- the four steps above in order on one stream;
 *   `sample_workspace` DEVICE float32 [samples], 2^bits <= samples <= 32768.
 * All pointers 16-byte aligned.  Errors: KMQ_ERR_NULL, KMQ_ERR_BITS,
 * KMQ_ERR_SHAPE, KMQ_ERR_ALIGN, KMQ_ERR_LAYOUT (unknown layout or lambda),
 * KMQ_ERR_CUDA.
 */
#define KMQ_LAMBDA_ABSMAX 0
#define KMQ_LAMBDA_ABSMEAN 1
kmq_status kmq_kmeans_rows(const float* W, int64_t N, int64_t K, int bits, int iters, uint16_t* codebooks,
                           double* centroids, void* stream);
kmq_status kmq_assign_pack(const float* W, const uint16_t* codebooks, int64_t N, int64_t K, int bits, int layout,
                           uint32_t* packed, void* stream);
kmq_status kmq_quantize_rows(const float* W, int64_t N, int64_t K, int bits, int iters, int layout,
                             uint16_t* codebooks, uint32_t* packed, void* stream);
kmq_status kmq_block_scales(const float* W, int64_t N, int64_t K, int lambda, uint16_t* scales, void* stream);
int64_t kmq_block_sample_count(int64_t N, int64_t K, int64_t samples);
kmq_status kmq_block_sample(const float* W, const uint16_t* scales, int64_t N, int64_t K, int64_t samples, float* out,
                            void* stream);
kmq_status kmq_block_assign_pack(const float* W, const uint16_t* scales, const uint16_t* codebook, int64_t N,
                                 int64_t K, int bits, uint8_t* wq, void* stream);
kmq_status kmq_block_quantize(const float* W, int64_t N, int64_t K, int bits, int lambda, int iters, int64_t samples,
                              uint16_t* scales, uint16_t* codebook, uint8_t* wq, float* sample_workspace,
                              void* stream);

/*
 * Measurement helpers (conveniences of this library; the paper has no
 * counterpart).  They put the layer's timings into proportion on the GPU at
 * hand:
 * kmq_probe_launch -- enqueue a kernel that does nothing, launched exactly as
 *   the layer's kernels are (programmatic dependent launch): timing a chain of
 *   these gives the fixed cost of a call, the floor under every layer whose
 *   ideal time is a microsecond or two.
 * kmq_probe_read -- read `bytes` (a multiple of 16) of DEVICE memory `buf`
 *   once with 128-bit streaming loads and fold them into `out` (DEVICE,
 *   kmq_probe_read_out_bytes() bytes): bytes / time is the read-only bandwidth
 *   a kernel of this library can reach, the ceiling next to the copy
 *   bandwidth that roofline fractions are quoted against.
 * Errors: KMQ_ERR_NULL, KMQ_ERR_ALIGN, KMQ_ERR_CUDA.
 */
kmq_status kmq_probe_launch(void* stream);
size_t kmq_probe_read_out_bytes(void);
kmq_status kmq_probe_read(const void* buf, size_t bytes, void* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* KMQ_H_ */
