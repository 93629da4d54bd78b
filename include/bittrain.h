/*
 * bittrain.h -- C ABI of the sparse-bitmap activation codec for NVIDIA B200 (sm_100a).
 *
 * The method is BitTrain's stash format: in the forward pass a layer's (mostly
 * zero, post-ReLU) activation is turned into a bitmap plus the vector of its
 * non-zero elements, and in the backward pass it is turned back (paper,
 * section 3.2 "Bitmap Format", Algorithm 1 and Algorithm 2).  The paper leaves
 * the concrete layout open; this library fixes it as
 *
 *   bitmap       uint32 words; element i <-> word i>>5, bit i&31 (LSB first);
 *                ceil(n/32) words; unused high bits of the last word are 0
 *   values       the elements whose bit pattern is not all-zero, copied
 *                verbatim, in flattened (row-major) element order; nnz entries
 *   chunk_prefix uint64; one entry per 4096-element chunk; entry c is the
 *                number of non-zero elements before chunk c (exclusive; entry
 *                0 is 0; there is no trailing total).  It replaces the single
 *                running counter j of Algorithm 2 so that chunks decode
 *                independently.
 *
 * "Zero" means an all-zero bit pattern: -0.0, NaN, infinities and subnormals
 * are kept, so decompress(compress(x)) is x bit for bit.
 *
 * General rules for every call below
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *     The caller owns every buffer; the library allocates nothing and neither
 *     synchronises nor prints.  Nothing about a tensor or a call outlives the
 *     call.  What the library does keep, all of it on the host: the calling
 *     thread's CTA limit (bt_set_max_ctas, off by default), a process-wide
 *     counter from which every compress launch draws its 64-bit tag, and, per
 *     device, the address of bt_compress_noalloc's built-in scratch array.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL
 *     for the default stream) on the current device.
 *   - Tensors are flat contiguous arrays of n elements (Algorithm 1 flattens
 *     the tensor first; the shape is the caller's metadata).
 *   - dense / values / y / gradient pointers must be 16-byte aligned, the
 *     bitmap 4-byte aligned (a 16-byte aligned bitmap is read with wider
 *     loads), chunk_prefix, nnz_out and the arena words 8-byte aligned, a
 *     workspace 16-byte aligned.
 *   - The return value reports what the host can see: BT_OK, an argument
 *     error (nothing was launched), or BT_ERR_CUDA if the launch itself
 *     failed.  Conditions only the device can see are written to *dev_status
 *     (when that pointer is not NULL).
 *   - n == 0 is valid: *nnz_out = 0 and *dev_status = BT_OK are written,
 *     nothing else is touched.
 *   - Buffers of one call must not overlap, except where a parameter says it
 *     may alias another.
 */
#ifndef BITTRAIN_H
#define BITTRAIN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BT_CHUNK_ELEMS 4096u

/* element types: the codec proper only needs the width, the ReLU pair the format
 * (the paper's format covers the usual floating-point widths, double included) */
enum { BT_F32 = 0, BT_F16 = 1, BT_BF16 = 2, BT_F64 = 3 };

enum {
    BT_OK = 0,
    BT_ERR_NULL = 1,       /* a required pointer is NULL                               */
    BT_ERR_DTYPE = 2,      /* unknown element type                                     */
    BT_ERR_ALIGN = 3,      /* a pointer breaks the alignment rule above                */
    BT_ERR_WORKSPACE = 4,  /* workspace smaller than bt_workspace_bytes(n)             */
    BT_ERR_CAPACITY = 5,   /* device: nnz > values_capacity (see bt_compress)          */
    BT_ERR_TIMEOUT = 6,    /* device: a bounded wait inside the kernel ran out         */
    BT_ERR_CUDA = 7,       /* the CUDA runtime reported an error at launch             */
    BT_ERR_TOO_LARGE = 8,  /* n exceeds what the call can handle (bt_compress_noalloc) */
    BT_ERR_SHAPE = 9       /* a dimension the call cannot take (bt_maxpool2x2_*: odd or zero) */
};

/* ======================================================================================
 * The codec proper: the size query, Algorithm 1, Algorithm 2, the fused ReLU forward and
 * the ReLU backward from the bitmap (plus the workspace query the two compressors need).
 * ====================================================================================== */

/*
 * Size in bytes of the compressed form: 4*ceil(n/32) + nnz*sizeof(dtype) +
 * 8*ceil(n/4096).  This is M_b of section 3.2 (element bytes times the
 * non-zero count plus one bit per element) with whole bitmap words and the
 * chunk prefix array added.  Pure host arithmetic; returns 0 for an unknown
 * dtype.
 */
size_t bt_compressed_bytes(uint64_t n, uint64_t nnz, int dtype);

/*
 * Bytes of device scratch bt_compress / bt_relu_fwd_compress need for n
 * elements: the tile descriptors and per-wave totals of the single-pass scan
 * plus a small header.  The contents need no initialisation and are
 * unspecified after a call: a tile descriptor counts as written by the running
 * call only if it carries that call's 64-bit tag, which no other call shares,
 * and the per-wave totals are cleared by the running launch itself, before a
 * grid-wide meeting that precedes the first addition to them.  Two calls that
 * run concurrently must not share a workspace; calls ordered on the device
 * (one stream, or events) may.  No counterpart in the paper (its scan is
 * sequential).
 */
size_t bt_workspace_bytes(uint64_t n);

/*
 * Algorithm 1 (dense -> bitmap).  Reads dense[0..n), writes bitmap
 * (ceil(n/32) words), values[0..nnz), chunk_prefix (ceil(n/4096) entries) and
 * *nnz_out.  values_capacity is the number of ELEMENTS the values buffer can
 * hold; n always suffices.  If nnz exceeds it, stores past the capacity are
 * suppressed, bitmap, chunk_prefix and *nnz_out are still complete and
 * correct, and *dev_status = BT_ERR_CAPACITY, so the caller can run again with
 * a buffer of nnz elements.  values[nnz..capacity) is left untouched or
 * unspecified.  *dev_status = BT_ERR_TIMEOUT means an internal bounded wait
 * gave up (two seconds without the data it waits for; every CTA then leaves
 * the kernel) and every output is undefined; the workspace and the context
 * stay usable and the next call runs normally.  The kernel is launched
 * cooperatively (all its CTAs resident at once, one per SM at most).
 */
int bt_compress(const void *dense, uint64_t n, int dtype,
                uint32_t *bitmap, void *values, uint64_t values_capacity,
                uint64_t *chunk_prefix, uint64_t *nnz_out,
                void *workspace, size_t workspace_bytes,
                int32_t *dev_status, void *stream);

/*
 * Algorithm 2 (bitmap -> dense).  dense_out[i] = bit i set ? the next value :
 * all-zero bits.  Chunks are decoded independently from chunk_prefix; values
 * must hold at least the nnz elements the bitmap calls for.
 */
int bt_decompress(const uint32_t *bitmap, const void *values,
                  const uint64_t *chunk_prefix, uint64_t n, int dtype,
                  void *dense_out, void *stream);

/*
 * ReLU forward fused with Algorithm 1: y[i] = (x[i] <= 0) ? +0 : x[i] under
 * IEEE comparison (so -0, negatives and -inf give +0 and a NaN passes through
 * with its payload), and y is stashed in compressed form in the same pass
 * (ReLU is the source of the sparsity, section 3.1; the activation is saved in
 * the forward pass, section 3.2).  y_out may be NULL (only the stash is
 * written) and may alias pre_act (in-place ReLU).  Other parameters as
 * bt_compress.
 */
int bt_relu_fwd_compress(const void *pre_act, uint64_t n, int dtype, void *y_out,
                         uint32_t *bitmap, void *values, uint64_t values_capacity,
                         uint64_t *chunk_prefix, uint64_t *nnz_out,
                         void *workspace, size_t workspace_bytes,
                         int32_t *dev_status, void *stream);

/*
 * ReLU backward from the stash: grad_in[i] = bit i set ? grad_out[i] : +0.
 * The backward pass restores activations to form gradients (section 3.2); for
 * ReLU itself only the bitmap is needed.  A select, not a multiply: masked
 * lanes are +0 even where grad_out is negative, infinite or NaN.  grad_in may
 * alias grad_out.
 */
int bt_relu_bwd_from_bitmap(const uint32_t *bitmap, const void *grad_out,
                            uint64_t n, int dtype, void *grad_in, void *stream);

/* ======================================================================================
 * Everything below is an extension around the six calls above: batched, fused, narrowing,
 * pooling, arena and host-buffer forms.  Each says what in the paper it serves.
 * ====================================================================================== */

/*
 * Batched forms of bt_compress and bt_relu_fwd_compress: `count` tensors of one element type in ONE
 * pass.  Algorithm 1 runs per tensor -- every tensor gets its own bitmap, values, chunk_prefix
 * (starting again at 0), *nnz_out and *dev_status, exactly what the single-tensor call writes -- but
 * the tiles of all tensors are dealt to the same resident grid, so a training step that stashes many
 * activations of a few megabytes each pays the fixed cost of a launch (a few microseconds: load,
 * compact, exchange counts, copy out) once per batch, not once per tensor.  `items` is a HOST array
 * read before the call returns; the pointers inside are device pointers with the alignment rules of
 * bt_compress.  bt_compress_batch: y_out must be NULL in every item; bt_relu_fwd_compress_batch: y_out
 * NULL in every item or in none (BT_ERR_SHAPE otherwise).  Tensors with n == 0 get *nnz_out = 0 and
 * *dev_status = BT_OK.  More than 32 non-empty tensors are handled as several launches on `stream`.
 * workspace_bytes >= bt_batch_workspace_bytes(n of every item); contents as for bt_workspace_bytes.
 * Nothing is launched on an argument error.  No counterpart in the paper (its loop is sequential).
 */
typedef struct bt_batch_item {
    const void *dense;          /* input: the activation, or the pre-activation for the fused form */
    void *y_out;                /* fused form: dense output, may alias dense; else NULL            */
    uint32_t *bitmap;
    void *values;
    uint64_t values_capacity;   /* in elements                                                     */
    uint64_t *chunk_prefix;
    uint64_t *nnz_out;
    int32_t *dev_status;        /* may be NULL                                                     */
    uint64_t n;
} bt_batch_item;

size_t bt_batch_workspace_bytes(const uint64_t *n /* host */, uint32_t count);

int bt_compress_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype,
                      void *workspace, size_t workspace_bytes, void *stream);

int bt_relu_fwd_compress_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype,
                               void *workspace, size_t workspace_bytes, void *stream);

/*
 * Batched forms of the two consumers, for the backward pass of a step that restores many stashes: `count`
 * tensors of one element type per launch (more than 32 non-empty tensors: several launches), each handled
 * exactly as by the single-tensor call.  The items are the ones the batched compressors took, read as
 *   bt_decompress_batch             y_out[i] = bit i ? next value : +0 from (bitmap, values, chunk_prefix);
 *                                   dense, values_capacity, nnz_out and dev_status are ignored
 *   bt_relu_bwd_from_bitmap_batch   y_out[i] = bit i ? dense[i] : +0 (dense: the upstream gradient; y_out may
 *                                   alias it); values, chunk_prefix, nnz_out and dev_status are ignored
 * Tensors with n == 0 are skipped.  No workspace.  Nothing is launched on an argument error.
 */
int bt_decompress_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype, void *stream);

int bt_relu_bwd_from_bitmap_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype, void *stream);

/*
 * Launch configuration for callers that keep several compress calls in flight
 * (on several streams, or in the branches of a CUDA graph).  The compress
 * kernel is launched cooperatively with one CTA per SM, and a cooperative
 * launch starts only when all its CTAs can be resident: two launches of more
 * than half the SMs each therefore run one after the other, whatever their
 * streams.  bt_set_max_ctas(m) limits every later compress-family launch MADE
 * BY THE CALLING THREAD to m CTAs (0: no limit, the default), so that
 * floor(SMs / m) launches can run side by side, each somewhat slower than it
 * would be alone.  Results do not depend on the limit.  Returns the limit it
 * replaces, or -1 (and changes nothing) if m < 0.  Host-side state only: a
 * launch captured into a CUDA graph keeps the limit it was captured with.
 * No counterpart in the paper.
 */
int bt_set_max_ctas(int max_ctas);

/*
 * Activation pruning fused with Algorithm 1 (section 4, "Combining BitTrain
 * with Activation Pruning": only activations that exceed a close-to-zero
 * threshold are stored, the others are taken to be zero; the paper studies
 * thresholds 0, 0.01, 0.05 and 0.1).  y[i] = (x[i] <= tau) ? +0 : x[i] under
 * IEEE comparison, the element widened exactly to binary32 (for BT_F64, tau
 * widened to binary64) and compared with the binary32 tau: "exceeds" is read as a strict comparison, so tau = 0 is
 * exactly bt_relu_fwd_compress, and a NaN (which neither exceeds nor falls
 * below anything) is kept with its payload.  tau may be negative; a NaN tau
 * prunes nothing.  Applied to an activation that is already non-negative this
 * is the thresholded compressor; applied to a pre-activation it is ReLU and
 * pruning in one pass.  y_out may be NULL and may alias x.  Lossy by design
 * for tau > 0; what is kept is kept bit for bit.  Other parameters, outputs and
 * *dev_status as bt_compress.  The backward pass is bt_relu_bwd_from_bitmap /
 * bt_decompress on the stash, unchanged.
 */
int bt_prune_fwd_compress(const void *x, uint64_t n, int dtype, float tau, void *y_out,
                          uint32_t *bitmap, void *values, uint64_t values_capacity,
                          uint64_t *chunk_prefix, uint64_t *nnz_out,
                          void *workspace, size_t workspace_bytes,
                          int32_t *dev_status, void *stream);

/*
 * Down-cast on stash (the evaluation's "Combining BitTrain with Low Precision"
 * study stores half-precision activation values in the bitmap format; these
 * two calls are its hybrid form for a training run that computes in binary32):
 * the tensor is BT_F32, the stashed values are to_dtype (BT_F16 or BT_BF16).
 * bitmap, chunk_prefix and *nnz_out are exactly those bt_compress /
 * bt_prune_fwd_compress give for the binary32 tensor -- the zero test is on
 * the binary32 pattern, so bt_relu_bwd_from_bitmap is unchanged -- and
 * values[k] (16 bits each; values_capacity counts 16-bit elements) is the k-th
 * kept element converted with round-to-nearest-even: overflow gives +-inf, a
 * magnitude of 2^-25 or less gives +-0 in binary16 (a zero stored under a set
 * bit), every NaN gives 0x7FFF.  bt_decompress with to_dtype restores the
 * narrowed dense tensor; bt_compressed_bytes(n, nnz, to_dtype) is the stash's
 * size.  y_out (BT_F32, may be NULL, may alias x) receives the unnarrowed
 * activation.  Lossy by design; no host-buffer form (arena forms below).
 * Other parameters and *dev_status as bt_compress.
 */
int bt_compress_narrow(const void *dense, uint64_t n, int to_dtype,
                       uint32_t *bitmap, void *values, uint64_t values_capacity,
                       uint64_t *chunk_prefix, uint64_t *nnz_out,
                       void *workspace, size_t workspace_bytes,
                       int32_t *dev_status, void *stream);
int bt_prune_fwd_compress_narrow(const void *x, uint64_t n, int to_dtype, float tau, void *y_out,
                                 uint32_t *bitmap, void *values, uint64_t values_capacity,
                                 uint64_t *chunk_prefix, uint64_t *nnz_out,
                                 void *workspace, size_t workspace_bytes,
                                 int32_t *dev_status, void *stream);

/*
 * Max pooling with winner codes.  The evaluation's per-layer analysis finds the
 * activations of max-pooling layers among the largest and sparsest; a
 * framework keeps, for such a layer's backward pass, its input and an index
 * tensor (8 bytes per output).  bt_maxpool2x2_fwd pools planes x height x width
 * elements (row-major, e.g. N*C planes of an NCHW tensor; height and width even
 * and non-zero, else BT_ERR_SHAPE) with a 2x2 window and stride 2 into y
 * (planes x height/2 x width/2) and writes, if codes is not NULL, 2 bits per
 * output naming the winning window position 2*dy + dx: sixteen outputs per
 * 32-bit word, output o in bits 2*(o%16).. of word o/16, ceil(outputs/16)
 * words, unused bits 0.  The window is visited in the order (0,0), (0,1),
 * (1,0), (1,1) and a later element replaces the maximum when it is greater
 * (IEEE comparison of the exactly widened values) or when it is a NaN: the
 * first of equal maxima wins, a NaN wins over everything, the last NaN over an
 * earlier one -- the positions a framework's index tensor would name.  y
 * receives a raw copy of the winner (then stashed with bt_compress like any
 * activation).  bt_maxpool2x2_bwd needs only the codes: grad_in (planes x
 * height x width) gets grad_out[o] at the coded position of window o and +0
 * at the other three; every element of grad_in is written.  x / y and
 * grad_out / grad_in must not overlap.  Tensors 16-byte aligned, codes and bitmaps 4-byte.
 */
int bt_maxpool2x2_fwd(const void *x, uint64_t planes, uint64_t height, uint64_t width, int dtype,
                      void *y, uint32_t *codes, void *stream);
int bt_maxpool2x2_bwd(const uint32_t *codes, const void *grad_out, uint64_t planes, uint64_t height,
                      uint64_t width, int dtype, void *grad_in, void *stream);

/*
 * Backward pass of ReLU followed by this pooling, for a forward pass that pooled first (the maximum
 * commutes with the ReLU: pool the pre-activation with bt_maxpool2x2_fwd, then run bt_relu_fwd_compress
 * on the pooled quarter).  pooled_bitmap is the bitmap of the pooled activation's stash (bit o set: output
 * o is non-zero after the ReLU).  grad_in gets grad_out[o] at the coded position of window o if bit o is
 * set, and +0 everywhere else: bt_relu_bwd_from_bitmap and bt_maxpool2x2_bwd in one pass.  Other
 * parameters as bt_maxpool2x2_bwd; pooled_bitmap 4-byte aligned, ceil(outputs / 32) words.
 */
int bt_maxpool2x2_bwd_masked(const uint32_t *codes, const uint32_t *pooled_bitmap, const void *grad_out,
                             uint64_t planes, uint64_t height, uint64_t width, int dtype, void *grad_in,
                             void *stream);

/*
 * Algorithm 2 on a narrowed stash, straight into a BT_F32 tensor: dense_out[i]
 * = the stashed 16-bit value of element i (from_dtype: BT_F16 or BT_BF16)
 * widened to binary32 -- exact for both types, a NaN keeps its sign and its
 * payload moves into the upper mantissa bits -- where bit i is set, +0
 * elsewhere.  The result equals bt_decompress in from_dtype followed by a cast
 * to binary32.  Other parameters as bt_decompress.
 */
int bt_decompress_widen(const uint32_t *bitmap, const void *values, const uint64_t *chunk_prefix,
                        uint64_t n, int from_dtype, void *dense_out, void *stream);

/*
 * ReLU6 (the activation of the MobileNetV2 family among the paper's models) fused with Algorithm 1:
 * y[i] = (x[i] <= 0) ? +0 : (x[i] >= 6 ? 6 : x[i]) under IEEE comparison of the exactly widened element
 * (a NaN fails both comparisons and is kept), stashed in the same pass.  Parameters as
 * bt_relu_fwd_compress.
 */
int bt_relu6_fwd_compress(const void *pre_act, uint64_t n, int dtype, void *y_out,
                          uint32_t *bitmap, void *values, uint64_t values_capacity,
                          uint64_t *chunk_prefix, uint64_t *nnz_out,
                          void *workspace, size_t workspace_bytes,
                          int32_t *dev_status, void *stream);

/*
 * ReLU6 backward from the stash: grad_in[i] = (bit i set and its stashed value < 6) ? grad_out[i] : +0.
 * The bitmap alone cannot tell a saturated unit (stashed value 6) from an active one, so the values and
 * the chunk prefix array are read as well.  A select, not a multiply.  grad_in may alias grad_out.
 */
int bt_relu6_bwd_from_stash(const uint32_t *bitmap, const void *values, const uint64_t *chunk_prefix,
                            const void *grad_out, uint64_t n, int dtype, void *grad_in, void *stream);

/*
 * Double-mask batch normalisation support (section 3.1: the zero pattern of
 * the normalisation layer's input is applied as a mask to its output, which
 * carries the sparsity through the layer).  mask_bitmap / mask_chunk_prefix are
 * the bitmap and prefix array of the INPUT's stash (as bt_compress or
 * bt_relu_fwd_compress wrote them); x is the layer's dense output.  Writes
 * values[k] = x[i] for the k-th set bit i, in element order, whatever x[i] is
 * (a zero under a set bit is stored as a value), so that (mask_bitmap, values,
 * mask_chunk_prefix) is the stash of the masked output -- bitmap, prefix array
 * and nnz are shared with the input's stash and are not written again -- and
 * bt_decompress restores it.  y_out, if not NULL, receives the masked dense
 * tensor (x at set bits, +0 elsewhere) and may alias x.  values must hold the
 * mask's nnz elements; stores at or beyond values_capacity are suppressed.
 * Bits of the last bitmap word beyond n are ignored.  No workspace, no scan:
 * ranks come from the prefix array.
 */
int bt_mask_compress(const void *x, uint64_t n, int dtype,
                     const uint32_t *mask_bitmap, const uint64_t *mask_chunk_prefix,
                     void *y_out, void *values, uint64_t values_capacity, void *stream);

/*
 * bt_compress for callers that cannot allocate device memory.  (The paper has
 * no counterpart: its implementation runs on the host and allocates freely.)
 *
 * Who needs it: code that runs where asking for device memory is not an
 * option -- a training hook called while the framework's allocator is frozen
 * (every byte of a memory plan already handed out, or a region in which an
 * allocation would synchronise the device or simply fail), or a plug-in that
 * receives its input and output buffers from a runtime that owns the device
 * memory and gives it no way to request a workspace.  bt_compress wants such a
 * workspace; here it is built into the library instead: a 393,488-byte array in
 * device memory that every GPU which loads the library holds until the process
 * exits.  That fixes the largest tensor: n <= BT_NOALLOC_MAX_ELEMS (2^26
 * elements); a larger n returns BT_ERR_TOO_LARGE and nothing is launched.
 *
 * The call allocates nothing and frees nothing, on the host path or on the
 * device.  The caller still passes every input and output buffer; arguments,
 * outputs and *dev_status are exactly those of bt_compress without the two
 * workspace parameters.  The first call on each device looks up the array's
 * device address (one runtime query, made with that device current) -- make
 * that first call outside any stream capture; later calls only launch.  All
 * calls on a device share the one array: nothing in it outlives a call
 * (its words are tagged per call), but two calls
 * whose execution overlaps on the GPU (different streams) race on it and give
 * undefined results -- keep them on one stream or order them with events.
 */
#define BT_NOALLOC_MAX_ELEMS (1ull << 26)

int bt_compress_noalloc(const void *dense, uint64_t n, int dtype,
                        uint32_t *bitmap, void *values, uint64_t values_capacity,
                        uint64_t *chunk_prefix, uint64_t *nnz_out,
                        int32_t *dev_status, void *stream);

/*
 * Arena forms (no counterpart in the paper; they serve a training loop that stashes one activation after
 * another).  A stash needs exactly nnz values, but nnz is known only on the device; sizing a buffer from
 * it costs a device-to-host read per tensor.  Here the caller owns one arena (a device buffer of
 * arena_bytes bytes, 16-byte aligned) and one device word, *arena_cursor, holding the number of bytes in
 * use (set it to 0, or back to an earlier value, with a device write in stream order).  A call reads the
 * cursor c, writes its packed values at arena + c, and -- if all nnz values fit behind the cursor --
 * stores c in *values_offset_out and advances the cursor to c + nnz * sizeof(dtype), rounded up to 16
 * bytes.  If they do not fit, *dev_status = BT_ERR_CAPACITY, the cursor and *values_offset_out stay as
 * they were, bitmap, chunk_prefix and *nnz_out are still complete.  For n == 0 the offset is the cursor
 * and the cursor does not move.  Calls that share an arena must be ordered on the device (one stream, or
 * events).  bt_prune_fwd_compress_arena with tau = 0 is the fused ReLU forward.  All other parameters as
 * in bt_compress / bt_prune_fwd_compress / bt_decompress.
 */
int bt_compress_arena(const void *dense, uint64_t n, int dtype, uint32_t *bitmap,
                      void *arena, uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offset_out,
                      uint64_t *chunk_prefix, uint64_t *nnz_out,
                      void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

int bt_prune_fwd_compress_arena(const void *x, uint64_t n, int dtype, float tau, void *y_out, uint32_t *bitmap,
                                void *arena, uint64_t arena_bytes, uint64_t *arena_cursor,
                                uint64_t *values_offset_out, uint64_t *chunk_prefix, uint64_t *nnz_out,
                                void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/* values_offset: the device word a *_arena compressor wrote (byte offset of the values inside the arena) */
int bt_decompress_arena(const uint32_t *bitmap, const void *arena, const uint64_t *values_offset,
                        const uint64_t *chunk_prefix, uint64_t n, int dtype, void *dense_out, void *stream);

/*
 * Batched arena forms: the tensors of a step pushed into the arena, or restored from it, by one launch per 32
 * tensors.  bt_compress_arena_batch / bt_relu_fwd_compress_arena_batch: what `count` calls of bt_compress_arena /
 * bt_prune_fwd_compress_arena (tau = 0) in the items' order would do -- tensor k's values start where tensor k-1's
 * ended, each rounded up to 16 bytes, and values_offsets_out[k] (a DEVICE array of `count` words) receives the byte
 * offset of tensor k's values; a tensor that does not fit reports BT_ERR_CAPACITY in its *dev_status, leaves its
 * offset word and the cursor where they were, and the next tensor starts at the same place.  The items' values and
 * values_capacity are ignored; a tensor with n == 0 gets *nnz_out = 0, *dev_status = BT_OK and offset 0.
 * workspace_bytes >= bt_batch_workspace_bytes(n of every item).  bt_decompress_arena_batch restores every item's
 * y_out from (bitmap, arena + values_offsets[k], chunk_prefix).  Calls that share an arena must be ordered on the
 * device, as for the single-tensor forms.
 */
int bt_compress_arena_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype, void *arena,
                            uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offsets_out,
                            void *workspace, size_t workspace_bytes, void *stream);

int bt_relu_fwd_compress_arena_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype, void *arena,
                                     uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offsets_out,
                                     void *workspace, size_t workspace_bytes, void *stream);

int bt_decompress_arena_batch(const bt_batch_item *items /* host */, uint32_t count, int dtype, const void *arena,
                              const uint64_t *values_offsets, void *stream);

/*
 * Arena forms of the later calls.  The narrowing compressors push 16-bit values: the cursor advances by
 * 2 * nnz bytes rounded up to 16, and the room behind the cursor is counted in 16-bit elements;
 * bt_decompress_widen_arena (or bt_decompress_arena with the 16-bit type) reads them back.  The ReLU6
 * pair pushes and reads values of the tensor's own type.  Everything else as in the arena forms above
 * and in bt_compress_narrow / bt_prune_fwd_compress_narrow / bt_decompress_widen / bt_relu6_fwd_compress
 * / bt_relu6_bwd_from_stash.
 */
int bt_compress_narrow_arena(const void *dense, uint64_t n, int to_dtype, uint32_t *bitmap,
                             void *arena, uint64_t arena_bytes, uint64_t *arena_cursor,
                             uint64_t *values_offset_out, uint64_t *chunk_prefix, uint64_t *nnz_out,
                             void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

int bt_prune_fwd_compress_narrow_arena(const void *x, uint64_t n, int to_dtype, float tau, void *y_out,
                                       uint32_t *bitmap, void *arena, uint64_t arena_bytes,
                                       uint64_t *arena_cursor, uint64_t *values_offset_out,
                                       uint64_t *chunk_prefix, uint64_t *nnz_out,
                                       void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

int bt_decompress_widen_arena(const uint32_t *bitmap, const void *arena, const uint64_t *values_offset,
                              const uint64_t *chunk_prefix, uint64_t n, int from_dtype, void *dense_out,
                              void *stream);

int bt_relu6_fwd_compress_arena(const void *pre_act, uint64_t n, int dtype, void *y_out, uint32_t *bitmap,
                                void *arena, uint64_t arena_bytes, uint64_t *arena_cursor,
                                uint64_t *values_offset_out, uint64_t *chunk_prefix, uint64_t *nnz_out,
                                void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

int bt_relu6_bwd_from_stash_arena(const uint32_t *bitmap, const void *arena, const uint64_t *values_offset,
                                  const uint64_t *chunk_prefix, const void *grad_out, uint64_t n, int dtype,
                                  void *grad_in, void *stream);

/*
 * Host-buffer forms.  The paper's own implementation keeps the stash in host
 * memory (section 4, "Implementation Details": std::bitset and std::vector);
 * these calls serve callers whose dense tensors or stashes live there.  Every
 * `host_*` pointer is a HOST pointer (pinned memory is copied fastest, pageable
 * memory works), `dev_staging` is a DEVICE buffer of at least
 * bt_host_staging_bytes(n, dtype) bytes, 256-byte aligned, owned by the caller
 * and free for reuse after the call.  Each call copies its inputs to the
 * staging area, runs the same kernels as the device forms, copies the results
 * back and SYNCHRONISES the stream before it returns, so device-side conditions
 * (BT_ERR_CAPACITY, BT_ERR_TIMEOUT) arrive in the return value.  The packed
 * values are nnz elements, a number only the device knows: into a page-locked
 * host_values buffer (16-byte aligned) the device writes exactly that many
 * itself and the call synchronises once, at its end; for pageable memory the
 * call synchronises a first time to learn nnz, then copies.  On any error
 * after the first copy was enqueued the stream is synchronised before the call
 * returns: nothing of a finished call is still pending on the caller's memory.  host_values_capacity counts
 * elements; if nnz exceeds it the first host_values_capacity values are
 * copied, *host_nnz holds the true count and BT_ERR_CAPACITY is returned.
 * Otherwise arguments mean what they mean in the device forms.
 */
size_t bt_host_staging_bytes(uint64_t n, int dtype);

int bt_compress_host(const void *host_dense, uint64_t n, int dtype,
                     uint32_t *host_bitmap, void *host_values, uint64_t host_values_capacity,
                     uint64_t *host_chunk_prefix, uint64_t *host_nnz,
                     void *dev_staging, size_t dev_staging_bytes, void *stream);

/* nnz: number of packed values in host_values (as returned by the compressor) */
int bt_decompress_host(const uint32_t *host_bitmap, const void *host_values,
                       const uint64_t *host_chunk_prefix, uint64_t nnz, uint64_t n, int dtype,
                       void *host_dense_out, void *dev_staging, size_t dev_staging_bytes, void *stream);

/* host_y_out may be NULL */
int bt_relu_fwd_compress_host(const void *host_pre_act, uint64_t n, int dtype, void *host_y_out,
                              uint32_t *host_bitmap, void *host_values, uint64_t host_values_capacity,
                              uint64_t *host_chunk_prefix, uint64_t *host_nnz,
                              void *dev_staging, size_t dev_staging_bytes, void *stream);

int bt_relu_bwd_from_bitmap_host(const uint32_t *host_bitmap, const void *host_grad_out,
                                 uint64_t n, int dtype, void *host_grad_in,
                                 void *dev_staging, size_t dev_staging_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* BITTRAIN_H */
