// Host-buffer forms of the four entry points: inputs are copied from host memory into a
// caller-provided device staging area, the same kernels run, results are copied back.  These
// calls synchronise the stream, so device-side conditions come back in the return value.
//
// The packed values are nnz elements and nnz is known only on the device.  Where the caller's
// value buffer is page-locked (the device can address it), a small kernel reads nnz and writes
// exactly that many values into it, and the call synchronises once, at its end.  Pageable memory
// cannot be written by a kernel: there the call synchronises to learn nnz, then copies.
#include "bt_internal.cuh"

namespace {

constexpr int kCopyThreads = 256;

// dst[0 .. min(*nnz, capacity, n) * es) = src[same range]; dst is host memory mapped into the device's address space,
// 16-byte aligned like src.  Whole 16-byte vectors by a grid-stride loop, the last bytes one by one.
__global__ void __launch_bounds__(kCopyThreads)
copy_values_sized(const unsigned char *__restrict__ src, unsigned char *__restrict__ dst, const uint64_t *__restrict__ nnz,
                  const uint64_t capacity, const uint64_t n, const uint32_t es)
{
    uint64_t count = *nnz < capacity ? *nnz : capacity;
    count          = count < n ? count : n;     // src holds n elements whatever a failed launch left in *nnz
    const uint64_t   bytes = count * es;
    const bt::Extent dx    = bt::extent_of(dst, capacity * es);
    const uint64_t   vecs  = bytes / 16;
    for (uint64_t v = static_cast<uint64_t>(blockIdx.x) * kCopyThreads + threadIdx.x; v < vecs;
         v += static_cast<uint64_t>(gridDim.x) * kCopyThreads)
        if (dx.holds(dst + 16 * v, 16)) reinterpret_cast<uint4 *>(dst)[v] = reinterpret_cast<const uint4 *>(src)[v];
    if (blockIdx.x == 0) {
        const uint64_t at = vecs * 16 + threadIdx.x;
        if (threadIdx.x < 16 && at < bytes && dx.holds(dst + at, 1)) dst[at] = src[at];
    }
}

// The device's address of a page-locked host buffer, or nullptr if a kernel cannot write there.
unsigned char *device_view_of_host(void *host)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        cudaGetLastError();   // an unknown pointer is not an error of this call
        return nullptr;
    }
    if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return nullptr;
    if ((reinterpret_cast<uintptr_t>(attr.devicePointer) & 15u) != 0) return nullptr;
    return static_cast<unsigned char *>(attr.devicePointer);
}

constexpr size_t kAlign = 256;
inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int    elem_size_of(int dtype) { return dtype == BT_F64 ? 8 : dtype == BT_F32 ? 4 : (dtype == BT_F16 || dtype == BT_BF16) ? 2 : 0; }

// Carves the staging area; every region starts 256-byte aligned.
struct Staging {
    unsigned char *dense, *dense2, *bitmap, *values, *prefix, *nnz, *status, *workspace;
    size_t         workspace_bytes, total;
    Staging(void *base, uint64_t n, int es)
    {
        unsigned char *p = static_cast<unsigned char *>(base);
        size_t         o = 0;
        auto take = [&](size_t bytes) { unsigned char *r = p + o; o += up(bytes ? bytes : 1); return r; };
        dense           = take(n * es);
        dense2          = take(n * es);
        bitmap          = take(4 * ((n + 31) / 32));
        values          = take(n * es);
        prefix          = take(8 * ((n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS));
        nnz             = take(8);
        status          = take(4);
        workspace_bytes = bt_workspace_bytes(n);
        workspace       = take(workspace_bytes);
        total           = o;
    }
};

inline bool ok(cudaError_t e) { return e == cudaSuccess; }

int compress_host_common(bool relu, const void *host_in, uint64_t n, int dtype, void *host_y, uint32_t *host_bitmap,
                         void *host_values, uint64_t host_values_capacity, uint64_t *host_prefix, uint64_t *host_nnz,
                         void *dev_staging, size_t dev_staging_bytes, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (!host_nnz) return BT_ERR_NULL;
    if (n == 0) {
        *host_nnz = 0;
        return BT_OK;
    }
    if (!host_in || !host_bitmap || !host_prefix || !dev_staging || (!host_values && host_values_capacity)) return BT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(dev_staging) & (kAlign - 1)) != 0) return BT_ERR_ALIGN;
    if (dev_staging_bytes < bt_host_staging_bytes(n, dtype)) return BT_ERR_WORKSPACE;
    cudaStream_t  s = static_cast<cudaStream_t>(stream);
    const Staging g(dev_staging, n, es);
    if (!ok(cudaMemcpyAsync(g.dense, host_in, n * es, cudaMemcpyHostToDevice, s))) return BT_ERR_CUDA;
    int rc;
    if (relu)
        rc = bt_relu_fwd_compress(g.dense, n, dtype, host_y ? g.dense2 : nullptr, reinterpret_cast<uint32_t *>(g.bitmap),
                                  g.values, n, reinterpret_cast<uint64_t *>(g.prefix),
                                  reinterpret_cast<uint64_t *>(g.nnz), g.workspace, g.workspace_bytes,
                                  reinterpret_cast<int32_t *>(g.status), stream);
    else
        rc = bt_compress(g.dense, n, dtype, reinterpret_cast<uint32_t *>(g.bitmap), g.values, n,
                         reinterpret_cast<uint64_t *>(g.prefix), reinterpret_cast<uint64_t *>(g.nnz), g.workspace,
                         g.workspace_bytes, reinterpret_cast<int32_t *>(g.status), stream);
    if (rc != BT_OK) {
        cudaStreamSynchronize(s);   // the copy of the input out of the caller's memory may still run
        return rc;
    }
    // From here on copies into the caller's memory (and into `status` below) may be pending: every way out
    // synchronises the stream first.
    int32_t status = BT_OK;
    auto    fail   = [&]() {
        cudaStreamSynchronize(s);
        return BT_ERR_CUDA;
    };
    if (!ok(cudaMemcpyAsync(host_bitmap, g.bitmap, 4 * ((n + 31) / 32), cudaMemcpyDeviceToHost, s)) ||
        !ok(cudaMemcpyAsync(host_prefix, g.prefix, 8 * ((n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS),
                            cudaMemcpyDeviceToHost, s)) ||
        !ok(cudaMemcpyAsync(host_nnz, g.nnz, 8, cudaMemcpyDeviceToHost, s)) ||
        !ok(cudaMemcpyAsync(&status, g.status, 4, cudaMemcpyDeviceToHost, s)) ||
        (host_y && !ok(cudaMemcpyAsync(host_y, g.dense2, n * es, cudaMemcpyDeviceToHost, s))))
        return fail();
    unsigned char *const mapped = host_values_capacity ? device_view_of_host(host_values) : nullptr;
    if (mapped) {
        // page-locked value buffer: the device copies exactly min(nnz, capacity) values; one synchronisation
        int dev = 0, sms = 0;
        if (!ok(cudaGetDevice(&dev)) || !ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return fail();
        copy_values_sized<<<sms * 4, kCopyThreads, 0, s>>>(g.values, mapped, reinterpret_cast<const uint64_t *>(g.nnz),
                                                            host_values_capacity, n, static_cast<uint32_t>(es));
        if (!ok(cudaGetLastError())) return fail();
    }
    if (!ok(cudaStreamSynchronize(s))) return BT_ERR_CUDA;
    if (status != BT_OK) return status;
    const uint64_t nnz = *host_nnz;
    if (!mapped) {
        const uint64_t cp = nnz < host_values_capacity ? nnz : host_values_capacity;
        if (cp && (!ok(cudaMemcpyAsync(host_values, g.values, cp * es, cudaMemcpyDeviceToHost, s)) ||
                   !ok(cudaStreamSynchronize(s))))
            return fail();
    }
    return nnz > host_values_capacity ? BT_ERR_CAPACITY : BT_OK;
}

}  // namespace

extern "C" {

size_t bt_host_staging_bytes(uint64_t n, int dtype)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return 0;
    return Staging(nullptr, n, es).total;
}

int bt_compress_host(const void *host_dense, uint64_t n, int dtype, uint32_t *host_bitmap, void *host_values,
                     uint64_t host_values_capacity, uint64_t *host_chunk_prefix, uint64_t *host_nnz,
                     void *dev_staging, size_t dev_staging_bytes, void *stream)
{
    return compress_host_common(false, host_dense, n, dtype, nullptr, host_bitmap, host_values, host_values_capacity,
                                host_chunk_prefix, host_nnz, dev_staging, dev_staging_bytes, stream);
}

int bt_relu_fwd_compress_host(const void *host_pre_act, uint64_t n, int dtype, void *host_y_out, uint32_t *host_bitmap,
                              void *host_values, uint64_t host_values_capacity, uint64_t *host_chunk_prefix,
                              uint64_t *host_nnz, void *dev_staging, size_t dev_staging_bytes, void *stream)
{
    return compress_host_common(true, host_pre_act, n, dtype, host_y_out, host_bitmap, host_values,
                                host_values_capacity, host_chunk_prefix, host_nnz, dev_staging, dev_staging_bytes,
                                stream);
}

int bt_decompress_host(const uint32_t *host_bitmap, const void *host_values, const uint64_t *host_chunk_prefix,
                       uint64_t nnz, uint64_t n, int dtype, void *host_dense_out, void *dev_staging,
                       size_t dev_staging_bytes, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!host_bitmap || !host_chunk_prefix || !host_dense_out || !dev_staging || (!host_values && nnz)) return BT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(dev_staging) & (kAlign - 1)) != 0) return BT_ERR_ALIGN;
    if (dev_staging_bytes < bt_host_staging_bytes(n, dtype)) return BT_ERR_WORKSPACE;
    if (nnz > n) return BT_ERR_CAPACITY;
    cudaStream_t  s = static_cast<cudaStream_t>(stream);
    const Staging g(dev_staging, n, es);
    if (!ok(cudaMemcpyAsync(g.bitmap, host_bitmap, 4 * ((n + 31) / 32), cudaMemcpyHostToDevice, s)) ||
        !ok(cudaMemcpyAsync(g.prefix, host_chunk_prefix, 8 * ((n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS),
                            cudaMemcpyHostToDevice, s)) ||
        (nnz && !ok(cudaMemcpyAsync(g.values, host_values, nnz * es, cudaMemcpyHostToDevice, s)))) {
        cudaStreamSynchronize(s);   // nothing of this call stays pending on the caller's memory
        return BT_ERR_CUDA;
    }
    const int rc = bt_decompress(reinterpret_cast<const uint32_t *>(g.bitmap), g.values,
                                 reinterpret_cast<const uint64_t *>(g.prefix), n, dtype, g.dense, stream);
    if (rc != BT_OK) {
        cudaStreamSynchronize(s);
        return rc;
    }
    if (!ok(cudaMemcpyAsync(host_dense_out, g.dense, n * es, cudaMemcpyDeviceToHost, s)) | !ok(cudaStreamSynchronize(s)))
        return BT_ERR_CUDA;
    return BT_OK;
}

int bt_relu_bwd_from_bitmap_host(const uint32_t *host_bitmap, const void *host_grad_out, uint64_t n, int dtype,
                                 void *host_grad_in, void *dev_staging, size_t dev_staging_bytes, void *stream)
{
    const int es = elem_size_of(dtype);
    if (es == 0) return BT_ERR_DTYPE;
    if (n == 0) return BT_OK;
    if (!host_bitmap || !host_grad_out || !host_grad_in || !dev_staging) return BT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(dev_staging) & (kAlign - 1)) != 0) return BT_ERR_ALIGN;
    if (dev_staging_bytes < bt_host_staging_bytes(n, dtype)) return BT_ERR_WORKSPACE;
    cudaStream_t  s = static_cast<cudaStream_t>(stream);
    const Staging g(dev_staging, n, es);
    if (!ok(cudaMemcpyAsync(g.bitmap, host_bitmap, 4 * ((n + 31) / 32), cudaMemcpyHostToDevice, s)) ||
        !ok(cudaMemcpyAsync(g.dense, host_grad_out, n * es, cudaMemcpyHostToDevice, s))) {
        cudaStreamSynchronize(s);
        return BT_ERR_CUDA;
    }
    const int rc = bt_relu_bwd_from_bitmap(reinterpret_cast<const uint32_t *>(g.bitmap), g.dense, n, dtype, g.dense2, stream);
    if (rc != BT_OK) {
        cudaStreamSynchronize(s);
        return rc;
    }
    if (!ok(cudaMemcpyAsync(host_grad_in, g.dense2, n * es, cudaMemcpyDeviceToHost, s)) | !ok(cudaStreamSynchronize(s)))
        return BT_ERR_CUDA;
    return BT_OK;
}

}  // extern "C"
