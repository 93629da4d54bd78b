// The extern "C" boundary: argument checks on the host, then one launch.
#include "bt_internal.cuh"

namespace {

inline int elem_size_of(int dtype)
{
    switch (dtype) {
    case BT_F32: return 4;
    case BT_F16: return 2;
    case BT_BF16: return 2;
    case BT_F64: return 8;
    default: return 0;
    }
}

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline uint64_t ceil_div(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

struct Arena {
    uint64_t *cursor     = nullptr;   // device word: bytes of the arena in use
    uint64_t *offset_out = nullptr;   // device word: receives the byte offset of this call's values
    uint64_t  bytes      = 0;
};

int compress_common(const void *src, uint64_t n, int dtype, int fused, float tau, void *y, uint32_t *bitmap, void *values,
                    uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace,
                    size_t workspace_bytes, int32_t *dev_status, void *stream, const Arena &arena = Arena(), int cast = 0)
{
    if (elem_size_of(dtype) == 0) return BT_ERR_DTYPE;
    if (cast != 0 && (dtype != BT_F32 || (cast != BT_F16 && cast != BT_BF16))) return BT_ERR_DTYPE;
    if (!nnz_out) return BT_ERR_NULL;
    if (!aligned(nnz_out, 8) || !aligned(dev_status, 4)) return BT_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (arena.cursor && (!arena.offset_out || !aligned(arena.cursor, 8) || !aligned(arena.offset_out, 8)))
        return arena.offset_out ? BT_ERR_ALIGN : BT_ERR_NULL;
    if (n == 0) {
        // nothing is pushed: the values of an empty tensor start where the cursor stands
        if (arena.cursor &&
            cudaMemcpyAsync(arena.offset_out, arena.cursor, sizeof(uint64_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
            return BT_ERR_CUDA;
        if (cudaMemsetAsync(nnz_out, 0, sizeof(uint64_t), s) != cudaSuccess) return BT_ERR_CUDA;
        if (dev_status && cudaMemsetAsync(dev_status, 0, sizeof(int32_t), s) != cudaSuccess) return BT_ERR_CUDA;
        return BT_OK;
    }
    if (!src || !bitmap || !chunk_prefix || !workspace) return BT_ERR_NULL;
    if (!values && values_capacity != 0) return BT_ERR_NULL;
    if (!aligned(src, 16) || !aligned(y, 16) || !aligned(bitmap, 4) || !aligned(values, 16) ||
        !aligned(chunk_prefix, 8) || !aligned(workspace, 16))
        return BT_ERR_ALIGN;
    if (workspace_bytes < bt_workspace_bytes(n)) return BT_ERR_WORKSPACE;

    bt::CompressArgs a{};
    a.src        = src;
    a.y          = y;
    a.bitmap     = bitmap;
    a.values     = values;
    a.capacity   = values_capacity;
    a.prefix     = chunk_prefix;
    a.nnz_out    = nnz_out;
    a.dev_status = dev_status;
    a.ws_header  = static_cast<uint64_t *>(workspace);
    a.ws_desc    = reinterpret_cast<uint64_t *>(static_cast<unsigned char *>(workspace) + bt::kWsHeaderBytes);
    a.cast       = cast;
    a.tau        = tau;
    a.arena_cursor      = arena.cursor;
    a.values_offset_out = arena.offset_out;
    a.arena_bytes       = arena.bytes;
    a.n          = n;
    return bt::launch_compress(a, dtype, fused, s) == cudaSuccess ? BT_OK : BT_ERR_CUDA;
}

// The batched forms: every tensor is checked before anything is launched; empty tensors get their nnz and status
// words and take no part in the launches; the others go out kMaxBatch at a time, one launch after the other on
// the stream, all through the same workspace.
int compress_batch_common(const bt_batch_item *items, uint32_t count, int dtype, int fused, void *workspace,
                          size_t workspace_bytes, void *stream, const bt::BatchArena *arena = nullptr,
                          uint64_t *offsets_out = nullptr)
{
    if (elem_size_of(dtype) == 0) return BT_ERR_DTYPE;
    if (count == 0) return BT_OK;
    if (!items) return BT_ERR_NULL;
    if (arena) {
        if (!arena->arena || !arena->arena_cursor || !offsets_out) return BT_ERR_NULL;
        if (!aligned(arena->arena, 16) || !aligned(arena->arena_cursor, 8) || !aligned(offsets_out, 8)) return BT_ERR_ALIGN;
    }
    uint64_t chunks = 0;
    bool     any_y = false, all_y = true, any = false;
    for (uint32_t k = 0; k < count; ++k) {
        const bt_batch_item &it = items[k];
        if (!it.nnz_out) return BT_ERR_NULL;
        if (!aligned(it.nnz_out, 8) || !aligned(it.dev_status, 4)) return BT_ERR_ALIGN;
        if (it.n == 0) continue;
        if (!it.dense || !it.bitmap || !it.chunk_prefix) return BT_ERR_NULL;
        if (!arena && !it.values && it.values_capacity != 0) return BT_ERR_NULL;
        if (!aligned(it.dense, 16) || !aligned(it.y_out, 16) || !aligned(it.bitmap, 4) || (!arena && !aligned(it.values, 16)) ||
            !aligned(it.chunk_prefix, 8))
            return BT_ERR_ALIGN;
        any = true;
        any_y |= it.y_out != nullptr;
        all_y &= it.y_out != nullptr;
        chunks += ceil_div(it.n, BT_CHUNK_ELEMS);
    }
    if (fused == 0 && any_y) return BT_ERR_SHAPE;            // the plain compressor has no dense output
    if (any_y && !all_y) return BT_ERR_SHAPE;                // a dense output for every tensor of a batch or for none
    if (any && !workspace) return BT_ERR_NULL;
    if (any && !aligned(workspace, 16)) return BT_ERR_ALIGN;
    if (any && workspace_bytes < bt::batch_workspace_bytes(chunks, count)) return BT_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bt::CompressJob jobs[bt::kMaxBatch];
    uint32_t        m = 0;
    for (uint32_t k = 0; k < count; ++k) {
        const bt_batch_item &it = items[k];
        if (it.n == 0) {
            if (cudaMemsetAsync(it.nnz_out, 0, sizeof(uint64_t), s) != cudaSuccess) return BT_ERR_CUDA;
            if (it.dev_status && cudaMemsetAsync(it.dev_status, 0, sizeof(int32_t), s) != cudaSuccess) return BT_ERR_CUDA;
            if (arena && cudaMemsetAsync(offsets_out + k, 0, sizeof(uint64_t), s) != cudaSuccess) return BT_ERR_CUDA;
        } else {
            bt::CompressJob &j = jobs[m++];
            j                  = bt::CompressJob{};
            j.src              = it.dense;
            j.y                = fused ? it.y_out : nullptr;
            j.bitmap           = it.bitmap;
            j.values           = arena ? nullptr : it.values;
            j.capacity         = arena ? 0 : it.values_capacity;
            j.prefix           = it.chunk_prefix;
            j.nnz_out          = it.nnz_out;
            j.dev_status       = it.dev_status;
            j.n                = it.n;
            j.offset_out       = arena ? offsets_out + k : nullptr;
        }
        if (m == bt::kMaxBatch || (k + 1 == count && m > 0)) {
            if (bt::launch_compress_batch(jobs, m, 0.0f, workspace, dtype, fused, arena, s) != cudaSuccess) return BT_ERR_CUDA;
            m = 0;
        }
    }
    return BT_OK;
}

// The consumers of a batch of stashes: backward == false restores items[k].y_out from (bitmap, values, chunk_prefix),
// backward == true writes items[k].y_out = bit ? items[k].dense : +0.
int consume_batch_common(const bt_batch_item *items, uint32_t count, int dtype, bool backward, void *stream,
                         const void *arena = nullptr, const uint64_t *offsets = nullptr)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (count == 0) return BT_OK;
    if (!items) return BT_ERR_NULL;
    for (uint32_t k = 0; k < count; ++k) {
        const bt_batch_item &it = items[k];
        if (it.n == 0) continue;
        if (!it.bitmap || !it.y_out) return BT_ERR_NULL;
        if (backward ? !it.dense : ((!arena && !it.values) || !it.chunk_prefix)) return BT_ERR_NULL;
        if (!aligned(it.bitmap, 4) || !aligned(it.y_out, 16)) return BT_ERR_ALIGN;
        if (backward ? !aligned(it.dense, 16) : ((!arena && !aligned(it.values, 16)) || !aligned(it.chunk_prefix, 8))) return BT_ERR_ALIGN;
    }
    cudaStream_t      s = static_cast<cudaStream_t>(stream);
    bt::DecompressJob jobs[bt::kMaxBatch];
    uint32_t          m = 0;
    for (uint32_t k = 0; k < count; ++k) {
        const bt_batch_item &it = items[k];
        if (it.n != 0)
            jobs[m++] = bt::DecompressJob{it.bitmap, arena ? arena : it.values, it.chunk_prefix, it.dense, it.y_out, it.n,
                                          arena ? offsets + k : nullptr};
        if (m == bt::kMaxBatch || (k + 1 == count && m > 0)) {
            const cudaError_t e = backward ? bt::launch_relu_bwd_batch(jobs, m, es, s) : bt::launch_decompress_batch(jobs, m, es, s);
            if (e != cudaSuccess) return BT_ERR_CUDA;
            m = 0;
        }
    }
    return BT_OK;
}

}  // namespace

#ifdef BT_BOUNDS_CHECK
namespace bt {
__device__ unsigned long long g_bounds_violations = 0;
}
#endif

extern "C" {

size_t bt_compressed_bytes(uint64_t n, uint64_t nnz, int dtype)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return 0;
    return static_cast<size_t>(4 * ceil_div(n, 32) + nnz * static_cast<uint64_t>(es) + 8 * ceil_div(n, BT_CHUNK_ELEMS));
}

int bt_set_max_ctas(int max_ctas)
{
    if (max_ctas < 0) return -1;
    return static_cast<int>(bt::set_compress_max_ctas(static_cast<uint32_t>(max_ctas)));
}

#ifdef BT_BOUNDS_CHECK
// Checking build only: the number of stores the kernels skipped because they fell outside their buffer, since
// the last reset.  Synchronises the device.  Returns a negative number if the runtime refuses the copy.
long long bt_test_bounds_violations(int reset)
{
    unsigned long long v = 0;
    if (cudaMemcpyFromSymbol(&v, bt::g_bounds_violations, sizeof(v)) != cudaSuccess) return -1;
    if (reset) {
        const unsigned long long zero = 0;
        if (cudaMemcpyToSymbol(bt::g_bounds_violations, &zero, sizeof(zero)) != cudaSuccess) return -1;
    }
    return static_cast<long long>(v);
}
#endif

#ifdef BT_TEST_HOOKS
// Test builds only (never the product library): the bound of every wait inside the compress kernels, so that a
// test can make a wait run out by itself and see the kernel return BT_ERR_TIMEOUT.
uint64_t bt_test_set_wait_ns(uint64_t wait_ns) { return bt::set_compress_wait_ns(wait_ns); }
#endif

size_t bt_workspace_bytes(uint64_t n)
{
    return bt::compress_workspace_bytes(ceil_div(n, BT_CHUNK_ELEMS));
}

size_t bt_batch_workspace_bytes(const uint64_t *n, uint32_t count)
{
    uint64_t chunks = 0;
    for (uint32_t k = 0; n && k < count; ++k) chunks += ceil_div(n[k], BT_CHUNK_ELEMS);
    return bt::batch_workspace_bytes(chunks, count);
}

int bt_compress_batch(const bt_batch_item *items, uint32_t count, int dtype, void *workspace, size_t workspace_bytes,
                      void *stream)
{
    return compress_batch_common(items, count, dtype, 0, workspace, workspace_bytes, stream);
}

int bt_compress_arena_batch(const bt_batch_item *items, uint32_t count, int dtype, void *arena, uint64_t arena_bytes,
                            uint64_t *arena_cursor, uint64_t *values_offsets_out, void *workspace, size_t workspace_bytes,
                            void *stream)
{
    const bt::BatchArena a{arena, arena_bytes, arena_cursor};
    return compress_batch_common(items, count, dtype, 0, workspace, workspace_bytes, stream, &a, values_offsets_out);
}

int bt_relu_fwd_compress_arena_batch(const bt_batch_item *items, uint32_t count, int dtype, void *arena,
                                     uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offsets_out,
                                     void *workspace, size_t workspace_bytes, void *stream)
{
    const bt::BatchArena a{arena, arena_bytes, arena_cursor};
    return compress_batch_common(items, count, dtype, 1, workspace, workspace_bytes, stream, &a, values_offsets_out);
}

int bt_decompress_batch(const bt_batch_item *items, uint32_t count, int dtype, void *stream)
{
    return consume_batch_common(items, count, dtype, false, stream);
}

int bt_decompress_arena_batch(const bt_batch_item *items, uint32_t count, int dtype, const void *arena,
                              const uint64_t *values_offsets, void *stream)
{
    if (count != 0 && (!arena || !values_offsets)) return BT_ERR_NULL;
    if (!aligned(arena, 16) || !aligned(values_offsets, 8)) return BT_ERR_ALIGN;
    return consume_batch_common(items, count, dtype, false, stream, arena, values_offsets);
}

int bt_relu_bwd_from_bitmap_batch(const bt_batch_item *items, uint32_t count, int dtype, void *stream)
{
    return consume_batch_common(items, count, dtype, true, stream);
}

int bt_relu_fwd_compress_batch(const bt_batch_item *items, uint32_t count, int dtype, void *workspace,
                               size_t workspace_bytes, void *stream)
{
    return compress_batch_common(items, count, dtype, 1, workspace, workspace_bytes, stream);
}

int bt_compress(const void *dense, uint64_t n, int dtype, uint32_t *bitmap, void *values, uint64_t values_capacity,
                uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace, size_t workspace_bytes,
                int32_t *dev_status, void *stream)
{
    return compress_common(dense, n, dtype, 0, 0.0f, nullptr, bitmap, values, values_capacity, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream);
}

int bt_relu_fwd_compress(const void *pre_act, uint64_t n, int dtype, void *y_out, uint32_t *bitmap, void *values,
                         uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace,
                         size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    return compress_common(pre_act, n, dtype, 1, 0.0f, y_out, bitmap, values, values_capacity, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream);
}

int bt_prune_fwd_compress(const void *x, uint64_t n, int dtype, float tau, void *y_out, uint32_t *bitmap, void *values,
                          uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace,
                          size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    return compress_common(x, n, dtype, 1, tau, y_out, bitmap, values, values_capacity, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream);
}

int bt_compress_narrow(const void *dense, uint64_t n, int to_dtype, uint32_t *bitmap, void *values,
                       uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace,
                       size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    if (to_dtype != BT_F16 && to_dtype != BT_BF16) return BT_ERR_DTYPE;
    return compress_common(dense, n, BT_F32, 0, 0.0f, nullptr, bitmap, values, values_capacity, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream, Arena(), to_dtype);
}

int bt_prune_fwd_compress_narrow(const void *x, uint64_t n, int to_dtype, float tau, void *y_out, uint32_t *bitmap,
                                 void *values, uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out,
                                 void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    if (to_dtype != BT_F16 && to_dtype != BT_BF16) return BT_ERR_DTYPE;
    return compress_common(x, n, BT_F32, 1, tau, y_out, bitmap, values, values_capacity, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream, Arena(), to_dtype);
}

int bt_relu6_fwd_compress(const void *pre_act, uint64_t n, int dtype, void *y_out, uint32_t *bitmap, void *values,
                          uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace,
                          size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    return compress_common(pre_act, n, dtype, 2, 0.0f, y_out, bitmap, values, values_capacity, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream);
}

int bt_relu6_bwd_from_stash(const uint32_t *bitmap, const void *values, const uint64_t *chunk_prefix,
                            const void *grad_out, uint64_t n, int dtype, void *grad_in, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !chunk_prefix || !grad_out || !grad_in) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(values, 16) || !aligned(chunk_prefix, 8) || !aligned(grad_out, 16) ||
        !aligned(grad_in, 16))
        return BT_ERR_ALIGN;
    return bt::launch_relu6_bwd(bitmap, values, nullptr, chunk_prefix, grad_out, n, dtype, grad_in,
                                static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_compress_arena(const void *dense, uint64_t n, int dtype, uint32_t *bitmap, void *arena, uint64_t arena_bytes,
                      uint64_t *arena_cursor, uint64_t *values_offset_out, uint64_t *chunk_prefix, uint64_t *nnz_out,
                      void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    if (!arena_cursor) return BT_ERR_NULL;
    Arena ar;
    ar.cursor = arena_cursor, ar.offset_out = values_offset_out, ar.bytes = arena_bytes;
    return compress_common(dense, n, dtype, 0, 0.0f, nullptr, bitmap, arena, arena_bytes, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream, ar);
}

int bt_prune_fwd_compress_arena(const void *x, uint64_t n, int dtype, float tau, void *y_out, uint32_t *bitmap, void *arena,
                                uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offset_out,
                                uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace, size_t workspace_bytes,
                                int32_t *dev_status, void *stream)
{
    if (!arena_cursor) return BT_ERR_NULL;
    Arena ar;
    ar.cursor = arena_cursor, ar.offset_out = values_offset_out, ar.bytes = arena_bytes;
    return compress_common(x, n, dtype, 1, tau, y_out, bitmap, arena, arena_bytes, chunk_prefix, nnz_out, workspace,
                           workspace_bytes, dev_status, stream, ar);
}

int bt_decompress_arena(const uint32_t *bitmap, const void *arena, const uint64_t *values_offset,
                        const uint64_t *chunk_prefix, uint64_t n, int dtype, void *dense_out, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !chunk_prefix || !dense_out || !arena || !values_offset) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(arena, 16) || !aligned(values_offset, 8) || !aligned(chunk_prefix, 8) ||
        !aligned(dense_out, 16))
        return BT_ERR_ALIGN;
    return bt::launch_decompress(bitmap, arena, values_offset, chunk_prefix, n, es, dense_out,
                                 static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_compress_narrow_arena(const void *dense, uint64_t n, int to_dtype, uint32_t *bitmap, void *arena,
                             uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offset_out,
                             uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace, size_t workspace_bytes,
                             int32_t *dev_status, void *stream)
{
    if (to_dtype != BT_F16 && to_dtype != BT_BF16) return BT_ERR_DTYPE;
    if (!arena_cursor) return BT_ERR_NULL;
    Arena ar;
    ar.cursor = arena_cursor, ar.offset_out = values_offset_out, ar.bytes = arena_bytes;
    return compress_common(dense, n, BT_F32, 0, 0.0f, nullptr, bitmap, arena, arena_bytes, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream, ar, to_dtype);
}

int bt_prune_fwd_compress_narrow_arena(const void *x, uint64_t n, int to_dtype, float tau, void *y_out, uint32_t *bitmap,
                                       void *arena, uint64_t arena_bytes, uint64_t *arena_cursor,
                                       uint64_t *values_offset_out, uint64_t *chunk_prefix, uint64_t *nnz_out,
                                       void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream)
{
    if (to_dtype != BT_F16 && to_dtype != BT_BF16) return BT_ERR_DTYPE;
    if (!arena_cursor) return BT_ERR_NULL;
    Arena ar;
    ar.cursor = arena_cursor, ar.offset_out = values_offset_out, ar.bytes = arena_bytes;
    return compress_common(x, n, BT_F32, 1, tau, y_out, bitmap, arena, arena_bytes, chunk_prefix, nnz_out, workspace,
                           workspace_bytes, dev_status, stream, ar, to_dtype);
}

int bt_relu6_fwd_compress_arena(const void *pre_act, uint64_t n, int dtype, void *y_out, uint32_t *bitmap, void *arena,
                                uint64_t arena_bytes, uint64_t *arena_cursor, uint64_t *values_offset_out,
                                uint64_t *chunk_prefix, uint64_t *nnz_out, void *workspace, size_t workspace_bytes,
                                int32_t *dev_status, void *stream)
{
    if (!arena_cursor) return BT_ERR_NULL;
    Arena ar;
    ar.cursor = arena_cursor, ar.offset_out = values_offset_out, ar.bytes = arena_bytes;
    return compress_common(pre_act, n, dtype, 2, 0.0f, y_out, bitmap, arena, arena_bytes, chunk_prefix, nnz_out,
                           workspace, workspace_bytes, dev_status, stream, ar);
}

int bt_decompress_widen_arena(const uint32_t *bitmap, const void *arena, const uint64_t *values_offset,
                              const uint64_t *chunk_prefix, uint64_t n, int from_dtype, void *dense_out, void *stream)
{
    if (from_dtype != BT_F16 && from_dtype != BT_BF16) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !chunk_prefix || !dense_out || !arena || !values_offset) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(arena, 16) || !aligned(values_offset, 8) || !aligned(chunk_prefix, 8) ||
        !aligned(dense_out, 16))
        return BT_ERR_ALIGN;
    return bt::launch_decompress_widen(bitmap, arena, values_offset, chunk_prefix, n, from_dtype, dense_out,
                                       static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_relu6_bwd_from_stash_arena(const uint32_t *bitmap, const void *arena, const uint64_t *values_offset,
                                  const uint64_t *chunk_prefix, const void *grad_out, uint64_t n, int dtype,
                                  void *grad_in, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !chunk_prefix || !grad_out || !grad_in || !arena || !values_offset) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(arena, 16) || !aligned(values_offset, 8) || !aligned(chunk_prefix, 8) ||
        !aligned(grad_out, 16) || !aligned(grad_in, 16))
        return BT_ERR_ALIGN;
    return bt::launch_relu6_bwd(bitmap, arena, values_offset, chunk_prefix, grad_out, n, dtype, grad_in,
                                static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_decompress(const uint32_t *bitmap, const void *values, const uint64_t *chunk_prefix, uint64_t n, int dtype,
                  void *dense_out, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !chunk_prefix || !dense_out) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(values, 16) || !aligned(chunk_prefix, 8) || !aligned(dense_out, 16))
        return BT_ERR_ALIGN;
    // values may be NULL only when the bitmap has no set bit; the kernel then never reads it
    return bt::launch_decompress(bitmap, values, nullptr, chunk_prefix, n, es, dense_out, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_decompress_widen(const uint32_t *bitmap, const void *values, const uint64_t *chunk_prefix, uint64_t n,
                        int from_dtype, void *dense_out, void *stream)
{
    if (from_dtype != BT_F16 && from_dtype != BT_BF16) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !chunk_prefix || !dense_out) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(values, 16) || !aligned(chunk_prefix, 8) || !aligned(dense_out, 16))
        return BT_ERR_ALIGN;
    return bt::launch_decompress_widen(bitmap, values, nullptr, chunk_prefix, n, from_dtype, dense_out,
                                       static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_mask_compress(const void *x, uint64_t n, int dtype, const uint32_t *mask_bitmap, const uint64_t *mask_chunk_prefix,
                     void *y_out, void *values, uint64_t values_capacity, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!x || !mask_bitmap || !mask_chunk_prefix) return BT_ERR_NULL;
    if (!values && values_capacity != 0) return BT_ERR_NULL;
    if (!aligned(x, 16) || !aligned(y_out, 16) || !aligned(mask_bitmap, 4) || !aligned(values, 16) ||
        !aligned(mask_chunk_prefix, 8))
        return BT_ERR_ALIGN;
    return bt::launch_mask_gather(x, mask_bitmap, mask_chunk_prefix, n, es, y_out, values, values_capacity,
                                  static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

int bt_maxpool2x2_fwd(const void *x, uint64_t planes, uint64_t height, uint64_t width, int dtype, void *y, uint32_t *codes,
                      void *stream)
{
    if (elem_size_of(dtype) == 0) return BT_ERR_DTYPE;
    if (height == 0 || width == 0 || (height & 1) || (width & 1)) return BT_ERR_SHAPE;
    if (planes == 0) return BT_OK;
    if (planes > (1ull << 40) / height / width) return BT_ERR_TOO_LARGE;
    if (!x || !y) return BT_ERR_NULL;
    if (!aligned(x, 16) || !aligned(y, 16) || !aligned(codes, 4)) return BT_ERR_ALIGN;
    return bt::launch_maxpool2x2_fwd(x, planes, height, width, dtype, y, codes, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

namespace {
int maxpool_bwd_common(const uint32_t *codes, const uint32_t *mask, bool masked, const void *grad_out, uint64_t planes,
                       uint64_t height, uint64_t width, int dtype, void *grad_in, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (height == 0 || width == 0 || (height & 1) || (width & 1)) return BT_ERR_SHAPE;
    if (planes == 0) return BT_OK;
    if (planes > (1ull << 40) / height / width) return BT_ERR_TOO_LARGE;
    if (!codes || !grad_out || !grad_in || (masked && !mask)) return BT_ERR_NULL;
    if (!aligned(codes, 4) || !aligned(mask, 4) || !aligned(grad_out, 16) || !aligned(grad_in, 16)) return BT_ERR_ALIGN;
    return bt::launch_maxpool2x2_bwd(codes, mask, grad_out, planes, height, width, es, grad_in,
                                     static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}
}  // namespace

int bt_maxpool2x2_bwd(const uint32_t *codes, const void *grad_out, uint64_t planes, uint64_t height, uint64_t width, int dtype,
                      void *grad_in, void *stream)
{
    return maxpool_bwd_common(codes, nullptr, false, grad_out, planes, height, width, dtype, grad_in, stream);
}

int bt_maxpool2x2_bwd_masked(const uint32_t *codes, const uint32_t *pooled_bitmap, const void *grad_out, uint64_t planes,
                             uint64_t height, uint64_t width, int dtype, void *grad_in, void *stream)
{
    return maxpool_bwd_common(codes, pooled_bitmap, true, grad_out, planes, height, width, dtype, grad_in, stream);
}

int bt_relu_bwd_from_bitmap(const uint32_t *bitmap, const void *grad_out, uint64_t n, int dtype, void *grad_in,
                            void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!bitmap || !grad_out || !grad_in) return BT_ERR_NULL;
    if (!aligned(bitmap, 4) || !aligned(grad_out, 16) || !aligned(grad_in, 16)) return BT_ERR_ALIGN;
    return bt::launch_relu_bwd(bitmap, grad_out, n, es, grad_in, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? BT_OK
               : BT_ERR_CUDA;
}

}  // extern "C"
