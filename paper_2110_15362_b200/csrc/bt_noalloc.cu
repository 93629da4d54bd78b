// bt_compress_noalloc: Algorithm 1 for callers that may not allocate device memory.
//
// bt_compress needs a scratch buffer (wave totals and tile descriptors of its scan).  Normally the
// caller allocates it.  Some callers cannot: a hook that runs while its framework's allocator is
// frozen (inside a memory plan whose every byte is already assigned, or in a region where an
// allocation would synchronise or fail), or a plug-in that is handed its input and output buffers
// by a runtime that owns the device memory and offers no way to ask for more.  For them the scratch
// lives here, in a file-scope device array that every GPU loading this library carries until the
// process exits (kScratchBytes, three eighths of a megabyte), which bounds the tensor size to
// BT_NOALLOC_MAX_ELEMS elements.
#include <mutex>

#include "bt_internal.cuh"

namespace {

// scratch for at most BT_NOALLOC_MAX_ELEMS elements: the same layout bt_workspace_bytes() sizes
constexpr size_t kScratchBytes = bt::compress_workspace_bytes(BT_NOALLOC_MAX_ELEMS / BT_CHUNK_ELEMS);

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

// In host code `g_scratch` is only a handle for the runtime, not a device address; the address on a
// given device comes from cudaGetSymbolAddress, asked once per device with that device current.
std::mutex g_lock;
void      *g_scratch_of_device[64] = {};

int scratch_for_current_device(void **out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BT_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_lock);
    if (g_scratch_of_device[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) return BT_ERR_CUDA;
        g_scratch_of_device[dev] = p;
    }
    *out = g_scratch_of_device[dev];
    return BT_OK;
}

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace

extern "C" int bt_compress_noalloc(const void *dense, uint64_t n, int dtype, uint32_t *bitmap, void *values,
                                   uint64_t values_capacity, uint64_t *chunk_prefix, uint64_t *nnz_out,
                                   int32_t *dev_status, void *stream)
{
    if (dtype != BT_F32 && dtype != BT_F16 && dtype != BT_BF16 && dtype != BT_F64) return BT_ERR_DTYPE;
    if (n > BT_NOALLOC_MAX_ELEMS) return BT_ERR_TOO_LARGE;      // the built-in scratch cannot describe more tiles
    if (!nnz_out) return BT_ERR_NULL;
    if (!aligned(nnz_out, 8) || !aligned(dev_status, 4)) return BT_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        if (cudaMemsetAsync(nnz_out, 0, sizeof(uint64_t), s) != cudaSuccess) return BT_ERR_CUDA;
        if (dev_status && cudaMemsetAsync(dev_status, 0, sizeof(int32_t), s) != cudaSuccess) return BT_ERR_CUDA;
        return BT_OK;
    }
    if (!dense || !bitmap || !chunk_prefix) return BT_ERR_NULL;
    if (!values && values_capacity != 0) return BT_ERR_NULL;
    if (!aligned(dense, 16) || !aligned(bitmap, 4) || !aligned(values, 16) || !aligned(chunk_prefix, 8))
        return BT_ERR_ALIGN;

    void     *scratch = nullptr;
    const int rc      = scratch_for_current_device(&scratch);   // first call on a device: looks the address up
    if (rc != BT_OK) return rc;

    bt::CompressArgs a{};
    a.src        = dense;
    a.bitmap     = bitmap;
    a.values     = values;
    a.capacity   = values_capacity;
    a.prefix     = chunk_prefix;
    a.nnz_out    = nnz_out;
    a.dev_status = dev_status;
    a.ws_header  = static_cast<uint64_t *>(scratch);
    a.ws_desc    = reinterpret_cast<uint64_t *>(static_cast<unsigned char *>(scratch) + bt::kWsHeaderBytes);
    a.n          = n;
    // nothing in the scratch is cleared between calls: the kernel tells this call's words by their tag
    return bt::launch_compress(a, dtype, 0, s) == cudaSuccess ? BT_OK : BT_ERR_CUDA;
}
