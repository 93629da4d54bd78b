/*
 * bt_oracle.h -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, single-threaded CPU statement of the BitTrain sparse-bitmap
 * codec (Algorithm 1 "Dense to Bitmap Matrix Compression" and Algorithm 2
 * "Bitmap to Dense Matrix Decompression", section 3.3 of the paper) in the
 * concrete layout this project fixes:
 *
 *   bitmap  : uint32 words, element i <-> word i>>5, bit i&31 (LSB first),
 *             ceil(n/32) words, padding bits of the last word are 0
 *   values  : the elements whose bit pattern is not all-zero, raw copies,
 *             in flattened element order
 *   prefix  : uint64, one entry per 4096-element chunk, prefix[c] = number of
 *             non-zero elements in chunks 0..c-1 (exclusive, no trailing total)
 *
 * Nothing here shares code, headers or constants with the CUDA library; only
 * tests, the smoke check and the CPU-baseline leg of the benchmark call it.
 * All pointers are host pointers owned by the caller.
 *
 * Element kinds for the ReLU pair (the codec itself only needs the size):
 */
#ifndef BT_ORACLE_H
#define BT_ORACLE_H
#include <stdint.h>
#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_F32 = 0, ORACLE_F16 = 1, ORACLE_BF16 = 2, ORACLE_F64 = 3 };

/* bytes of one element of kind `kind`, 0 if the kind is unknown */
int oracle_elem_size(int kind);

/* Algorithm 1. elem_size in {2,4,8}. Returns nnz (also the number of values written). */
uint64_t oracle_compress(const void *dense, uint64_t n, int elem_size,
                         uint32_t *bitmap, void *values, uint64_t *prefix);

/* Algorithm 2, literal: one running counter j over the whole bitmap. */
void oracle_decompress(const uint32_t *bitmap, const void *values,
                       uint64_t n, int elem_size, void *dense_out);

/* Algorithm 2 restarted per chunk with j = prefix[c]: shows the prefix array
 * alone is enough to decode chunks independently. */
void oracle_decompress_chunked(const uint32_t *bitmap, const void *values,
                               const uint64_t *prefix, uint64_t n, int elem_size,
                               void *dense_out);

/* y = (x <= 0) ? +0 : x with IEEE comparison (NaN kept with payload), then
 * Algorithm 1 on y. y may be NULL. Returns nnz. */
uint64_t oracle_relu_fwd_compress(const void *pre_act, uint64_t n, int kind,
                                  void *y, uint32_t *bitmap, void *values,
                                  uint64_t *prefix);

/* Activation pruning with threshold tau joined to the stash: y = (x <= tau) ? +0 : x
 * (the element widened exactly, IEEE comparison, NaN kept), then Algorithm 1 on
 * y.  tau = 0 is oracle_relu_fwd_compress.  y may be NULL.  Returns nnz. */
uint64_t oracle_prune_fwd_compress(const void *x, uint64_t n, int kind, float tau,
                                   void *y, uint32_t *bitmap, void *values,
                                   uint64_t *prefix);

/* Double-mask batch normalisation: values = the elements of x at the set bits
 * of mask_bitmap, in element order (pushed whatever their value); y (may be
 * NULL) = x at set bits, +0 elsewhere.  The stash of the result is
 * (mask_bitmap, values, the mask's own prefix array).  Returns the count. */
uint64_t oracle_mask_compress(const void *x, uint64_t n, int elem_size,
                              const uint32_t *mask_bitmap, void *y, void *values);

/* ReLU6 joined to the stash: y = (x <= 0) ? +0 : (x >= 6 ? 6 : x), NaN kept, then
 * Algorithm 1 on y.  y may be NULL.  Returns nnz. */
uint64_t oracle_relu6_fwd_compress(const void *pre_act, uint64_t n, int kind,
                                   void *y, uint32_t *bitmap, void *values,
                                   uint64_t *prefix);

/* ReLU6 backward: grad_in[i] = (bit i set and its stashed value < 6) ? grad_out[i] : +0 */
void oracle_relu6_bwd_from_stash(const uint32_t *bitmap, const void *values,
                                 uint64_t n, int kind, const void *grad_out,
                                 void *grad_in);

/* grad_in[i] = bit i ? grad_out[i] (raw copy) : +0 */
void oracle_relu_bwd_from_bitmap(const uint32_t *bitmap, const void *grad_out,
                                 uint64_t n, int elem_size, void *grad_in);

/* M_b of section 3.2 generalised: bitmap words + values + prefix entries */
uint64_t oracle_compressed_bytes(uint64_t n, uint64_t nnz, int elem_size);

/* Down-cast on stash (the low-precision study of the paper's evaluation, as a
 * hybrid: binary32 tensor, 16-bit stashed values).  act = fused ? ((x <= tau) ?
 * +0 : x) : x; bitmap / prefix / count are those of act in binary32; values[k]
 * is the k-th non-zero of act narrowed to to_kind (ORACLE_F16 / ORACLE_BF16)
 * by the conversions below.  y (binary32, may be NULL) = act.  Returns nnz. */
uint64_t oracle_narrow_compress(const void *x, uint64_t n, int to_kind, int fused, float tau,
                                void *y, uint32_t *bitmap, uint16_t *values, uint64_t *prefix);

/* 2x2 / stride 2 max pooling of planes x height x width elements (height and
 * width even) with a 2-bit code per output naming the winning window position
 * (2*dy + dx; window order (0,0),(0,1),(1,0),(1,1); a later element wins when
 * greater or NaN), sixteen codes per 32-bit word, LSB first.  The pooled output
 * is what the stash then compresses; the codes replace the saved input and the
 * index tensor in the backward pass. */
void oracle_maxpool2x2_fwd(const void *x, uint64_t planes, uint64_t height, uint64_t width,
                           int kind, void *y, uint32_t *codes);
void oracle_maxpool2x2_bwd(const uint32_t *codes, const void *grad_out, uint64_t planes,
                           uint64_t height, uint64_t width, int elem_size, void *grad_in);

/* Algorithm 2 on a narrowed stash, each value widened exactly to binary32 */
void oracle_widen_decompress(const uint32_t *bitmap, const uint16_t *values, uint64_t n,
                             int from_kind, void *dense_f32);

/* binary32 pattern -> binary16 / bfloat16 pattern: round to nearest, ties to
 * even; overflow to infinity; every NaN to 0x7FFF */
uint16_t oracle_float_to_half(uint32_t bits);
uint16_t oracle_float_to_bfloat16(uint32_t bits);

/* exact widening of one IEEE binary16 pattern to binary32 (used by the ReLU test) */
float oracle_half_to_float(uint16_t h);

#ifdef __cplusplus
}
#endif
#endif
