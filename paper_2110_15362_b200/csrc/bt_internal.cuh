// Shared declarations of the CUDA side of the codec: launcher prototypes, the
// workspace layout and thin wrappers over the sm_100a PTX the kernels use
// (mbarrier, 1-D bulk async copies, relaxed device-scope loads and stores).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "bittrain.h"

namespace bt {

// ---------------------------------------------------------------- workspace layout
// The workspace arrives with unspecified contents.  It holds
//   a 256-byte header, 64-bit words: [0] seq, the launch sequence number of this workspace; [1] abort, equal to
//     the launch's tag once a bounded wait of that launch ran out;
//   one 64-bit total per wave of tiles of every tensor of the launch (an even number of words): sums made by
//     reductions, zeroed by the launch itself before the grid's one meeting, used only by tensors of more than
//     one wave;
//   one 16-byte descriptor per tile, never cleared: word 0 = (tag >> 32) << 32 | count, word 1 = (tag & 0xFFFFFFFF)
//     << 32 | count.  A reader takes a descriptor only if both halves carry its own launch's tag and agree on
//     the count (the two halves may be written and read separately).
// tag = mix64(call_tag + seq * odd) | 1: call_tag comes from the host (a process-wide counter: two calls never
// share one), seq is header word 0 as the launch found it.  Every launch changes seq before it ends (the CTA of
// the last tile adds 1 once all counts are in; a CTA that gives up adds 2^32), so replays of one captured launch
// -- same call_tag -- get different tags too.  Memory this library never wrote matches by chance only: 2^-64
// per word for the tag, and the repeated count on top.
// Sized for the smallest tile: 24 bytes per 4096 elements.
constexpr size_t   kWsHeaderBytes = 256;
constexpr uint32_t kMinTileElems  = BT_CHUNK_ELEMS;
constexpr uint32_t kMaxBatch      = 32;                        // tensors of one batched launch
constexpr uint64_t kDefaultWaitNs = 2000000000ull;             // bound of every in-kernel wait: 2 s
// bytes of workspace for tensors holding `chunks` 4096-element chunks in all
__host__ __device__ constexpr size_t compress_workspace_bytes(uint64_t chunks) { return kWsHeaderBytes + 16 + 24 * static_cast<size_t>(chunks); }

// One tensor, one launch.
struct CompressArgs {
    const void *src;        // dense input (pre-activation for the fused form)
    void       *y;          // optional dense ReLU output
    uint32_t   *bitmap;
    void       *values;
    uint64_t    capacity;   // in elements
    uint64_t   *prefix;
    uint64_t   *nnz_out;
    int32_t    *dev_status;
    uint64_t   *ws_header;
    uint64_t   *ws_desc;    // wave totals, then tile descriptors
    uint32_t    ws_waves;   // number of wave-total words (even; set by launch_compress)
    uint64_t    call_tag;   // unique to the call (set by launch_compress)
    uint64_t    wait_ns;    // bound of every in-kernel wait (set by launch_compress)
    int         cast;       // 0, or the 16-bit type (BT_F16 / BT_BF16) the stashed values of a binary32 tensor are narrowed to
    float       tau;        // fused forms: elements <= tau become +0 (0 for plain ReLU)
    // arena forms: `values` is the arena's base, the packed values go to values + *arena_cursor (bytes);
    // on success the kernel stores the old cursor in *values_offset_out and advances the cursor past the
    // values (rounded up to 16 bytes).  All three are NULL / 0 for the plain forms.
    uint64_t   *arena_cursor;
    uint64_t   *values_offset_out;
    uint64_t    arena_bytes;
    uint64_t    n;
};

// One tensor of a batched launch.
struct CompressJob {
    const void *src;        // dense input (pre-activation for the fused form)
    void       *y;          // optional dense output of the fused form
    uint32_t   *bitmap;
    void       *values;
    uint64_t    capacity;   // in elements
    uint64_t   *prefix;
    uint64_t   *nnz_out;
    int32_t    *dev_status;
    uint64_t    n;
    uint64_t   *offset_out; // arena form: where the byte offset of the tensor's values in the arena goes
    // set by launch_compress_batch:
    uint32_t    tiles;      // number of tiles of the tensor
    uint32_t    rot;        // the CTA that takes the tensor's tile 0 (tile t goes to CTA (rot + t) mod grid)
    uint32_t    total0;     // index of the tensor's first wave-total word
    uint32_t    desc0;      // index of the tensor's first tile descriptor
};

// What the tensors of a batched launch share (all set by launch_compress_batch but tau).
struct CompressCommon {
    uint64_t   *ws_header;
    uint64_t   *ws_total;   // wave totals
    uint64_t   *ws_desc;    // tile descriptors
    uint32_t    ws_totals;  // number of wave-total words (even)
    uint64_t    ws_words;   // 8-byte words of the workspace behind its header (what the size query promises)
    uint32_t    jobs;       // number of tensors
    uint64_t    call_tag;   // unique to the call
    uint64_t    wait_ns;    // bound of every in-kernel wait
    float       tau;        // fused form: elements <= tau become +0 (0 for plain ReLU)
    // arena form (arena != nullptr): the tensors' values go back to back behind *arena_cursor
    void       *arena;
    uint64_t    arena_bytes;
    uint64_t   *arena_cursor;
    uint64_t   *ws_arena;   // two tagged words per tensor: the cursor behind that tensor (set by launch_compress_batch)
};

// What the caller of launch_compress_batch gives for the arena form.
struct BatchArena {
    void     *arena;
    uint64_t  arena_bytes;
    uint64_t *arena_cursor;
};

// bytes of workspace for a batched launch: the tensors' descriptors and totals, and two words per tensor for the
// arena form's chain of cursors
__host__ __device__ constexpr size_t batch_workspace_bytes(uint64_t chunks, uint32_t count)
{
    return compress_workspace_bytes(chunks) + 16 * static_cast<size_t>(count);
}

// fused: 0 plain compressor, 1 threshold form (ReLU at tau = 0), 2 ReLU6
cudaError_t launch_compress(const CompressArgs &a, int dtype, int fused, cudaStream_t s);
// `jobs` (count of them: 1 .. kMaxBatch, every n > 0) are the tensors of one launch; `workspace` holds at least
// batch_workspace_bytes() of their chunks; fused: 0 plain compressor, 1 threshold form; arena: nullptr, or the arena
// the values go to (the jobs' values / capacity are then ignored and their offset_out must be set)
cudaError_t launch_compress_batch(const CompressJob *jobs, uint32_t count, float tau, void *workspace, int dtype, int fused,
                                  const BatchArena *arena, cudaStream_t s);
// the calling thread's limit on the CTAs of one compress launch (0: none); returns the limit it replaces
uint32_t set_compress_max_ctas(uint32_t max_ctas);
// the bound of the compress kernels' waits for later launches of the process; returns the one it replaces
// (reachable only from a test build of the library)
uint64_t set_compress_wait_ns(uint64_t wait_ns);
// values_offset: NULL, or a device word holding the byte offset of the packed values inside `values`
cudaError_t launch_decompress(const uint32_t *bitmap, const void *values, const uint64_t *values_offset,
                              const uint64_t *prefix, uint64_t n, int elem_size, void *out, cudaStream_t s);
// One tensor of a batched restore / batched ReLU backward (every n > 0); `in` is the upstream gradient of the
// backward form and unused by the restore.
struct DecompressJob {
    const uint32_t *bitmap;
    const void     *values;
    const uint64_t *prefix;
    const void     *in;
    void           *out;
    uint64_t        n;
    const uint64_t *values_offset;   // restore only: NULL, or a device word with the byte offset of the values inside `values`
};
cudaError_t launch_decompress_batch(const DecompressJob *jobs, uint32_t count, int elem_size, cudaStream_t s);
cudaError_t launch_relu_bwd_batch(const DecompressJob *jobs, uint32_t count, int elem_size, cudaStream_t s);
cudaError_t launch_decompress_widen(const uint32_t *bitmap, const void *values16, const uint64_t *values_offset,
                                    const uint64_t *prefix, uint64_t n, int from_dtype, void *out_f32, cudaStream_t s);
cudaError_t launch_mask_gather(const void *x, const uint32_t *bitmap, const uint64_t *prefix, uint64_t n,
                               int elem_size, void *y, void *values, uint64_t capacity, cudaStream_t s);
cudaError_t launch_relu6_bwd(const uint32_t *bitmap, const void *values, const uint64_t *values_offset,
                             const uint64_t *prefix, const void *gout, uint64_t n, int dtype, void *gin, cudaStream_t s);
cudaError_t launch_maxpool2x2_fwd(const void *x, uint64_t planes, uint64_t height, uint64_t width, int dtype, void *y,
                                  uint32_t *codes, cudaStream_t s);
// mask: NULL, or a bitmap over the pooled outputs (the gradient of an output whose bit is clear counts as +0)
cudaError_t launch_maxpool2x2_bwd(const uint32_t *codes, const uint32_t *mask, const void *gout, uint64_t planes,
                                  uint64_t height, uint64_t width, int elem_size, void *gin, cudaStream_t s);
cudaError_t launch_relu_bwd(const uint32_t *bitmap, const void *gout, uint64_t n, int elem_size,
                            void *gin, cudaStream_t s);

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

// makes the barrier initialisation and earlier generic-proxy shared-memory
// writes visible to the async proxy (the bulk-copy engine)
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

// ---------------------------------------------------------------------------------------------
// Checking build (-DBT_BOUNDS_CHECK, a library of its own that only the tests load): every store to
// global memory is tested against the extent of the buffer it belongs to.  A store that would fall
// outside is skipped and counted in a device word the test reads back; nothing traps.  In the
// product build an Extent is empty and `holds` is the constant true, so the checks cost nothing.
#ifdef BT_BOUNDS_CHECK
extern __device__ unsigned long long g_bounds_violations;   // one word for the library: relocatable device code
struct Extent {
    uintptr_t lo, hi;   // [lo, hi) in bytes
    __device__ __forceinline__ bool holds(const void *p, const size_t bytes) const
    {
        const uintptr_t a  = reinterpret_cast<uintptr_t>(p);
        const bool      ok = a >= lo && a + bytes <= hi;
        if (!ok) atomicAdd(&g_bounds_violations, 1ull);
        return ok;
    }
};
__device__ __forceinline__ Extent extent_of(const void *base, const uint64_t bytes)
{
    return Extent{reinterpret_cast<uintptr_t>(base), reinterpret_cast<uintptr_t>(base) + bytes};
}
#else
struct Extent {
    __device__ __forceinline__ bool holds(const void *, const size_t) const { return true; }
};
__device__ __forceinline__ Extent extent_of(const void *, const uint64_t) { return Extent{}; }
#endif

// A lane's four consecutive words of a chunk's bitmap, w0 a multiple of four; words past the end of the
// bitmap read as zero.  One 16-byte load where the bitmap's base address allows it (the format only
// asks for 4-byte alignment), four word loads otherwise.
__device__ __forceinline__ uint4 load_words4(const uint32_t *__restrict__ bitmap, const uint64_t w0,
                                             const uint64_t words_total)
{
    uint4 w4 = make_uint4(0, 0, 0, 0);
    if (w0 + 3 < words_total && (reinterpret_cast<uintptr_t>(bitmap) & 15u) == 0) {
        w4 = *reinterpret_cast<const uint4 *>(bitmap + w0);
    } else {
        if (w0 < words_total) w4.x = bitmap[w0];
        if (w0 + 1 < words_total) w4.y = bitmap[w0 + 1];
        if (w0 + 2 < words_total) w4.z = bitmap[w0 + 2];
        if (w0 + 3 < words_total) w4.w = bitmap[w0 + 3];
    }
    return w4;
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// 1-D bulk async copy global -> this CTA's shared memory, completing on an mbarrier.
// Both addresses 16-byte aligned, bytes a non-zero multiple of 16.
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// 1-D bulk async copy this CTA's shared memory -> global (bulk-group completion).
__device__ __forceinline__ void bulk_store(void *gmem_dst, const void *smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst),
                 "r"(smem_addr(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t *p)
{
    uint64_t v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(uint64_t *p, uint64_t v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// 16-byte descriptor accesses (the two halves may be performed separately: each is self-validating)
__device__ __forceinline__ void ld_relaxed_2xu64(const uint64_t *p, uint64_t &w0, uint64_t &w1)
{
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_relaxed_2xu64(uint64_t *p, uint64_t w0, uint64_t w1)
{
    asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(w0), "l"(w1) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u32(uint32_t *p, uint32_t v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ uint32_t lanemask_lt()
{
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// ---------------------------------------------------------------- decisions of the fused forward forms
// Elem<DT>::widen(u): the element's value, widened exactly (binary16 / bfloat16 -> binary32; binary32 and
// binary64 as they are).  The 16-bit forms take the pattern in the low half of the register (the upper half
// may hold a sign extension).  Elem<DT>::kSix: the pattern of 6.0 in the element type (exact in all four).
template <int DT>
struct Elem;
template <>
struct Elem<BT_F32> {
    static constexpr uint32_t kSix = 0x40C00000u;
    __device__ static __forceinline__ float widen(uint32_t u) { return __uint_as_float(u); }
};
template <>
struct Elem<BT_F64> {
    static constexpr uint64_t kSix = 0x4018000000000000ull;
    __device__ static __forceinline__ double widen(uint64_t u) { return __longlong_as_double(static_cast<long long>(u)); }
};
template <>
struct Elem<BT_F16> {
    static constexpr uint32_t kSix = 0x4600u;
    __device__ static __forceinline__ float widen(uint32_t u)
    {
        float f;
        asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"(static_cast<unsigned short>(u)));
        return f;
    }
};
template <>
struct Elem<BT_BF16> {
    static constexpr uint32_t kSix = 0x40C0u;
    __device__ static __forceinline__ float widen(uint32_t u) { return __uint_as_float(u << 16); }
};

// v >= 6 as an opaque 0/1 (false for a NaN).  Written as inline PTX on purpose: given the comparison and the
// select that follows it in C++, the compiler may fuse the two into a floating-point minimum, which returns the
// canonical NaN for a NaN input and so loses the payload and sign that the format keeps.
__device__ __forceinline__ uint32_t at_least_six(float v)
{
    uint32_t r;
    asm("{\n\t.reg .pred p;\n\tsetp.ge.f32 p, %1, 0f40C00000;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ uint32_t at_least_six(double v)
{
    uint32_t r;
    asm("{\n\t.reg .pred p;\n\tsetp.ge.f64 p, %1, 0d4018000000000000;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "d"(v));
    return r;
}

// (v > b) || isnan(v) as an opaque 0/1, for the same reason: a compare-and-select chain written in C++ may
// become a floating-point maximum, which does not keep a NaN's payload.
__device__ __forceinline__ uint32_t greater_or_nan(float v, float b)
{
    uint32_t r;
    asm("{\n\t.reg .pred p, q;\n\tsetp.gt.f32 p, %1, %2;\n\tsetp.nan.f32 q, %1, %1;\n\tor.pred p, p, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "f"(v), "f"(b));
    return r;
}
__device__ __forceinline__ uint32_t greater_or_nan(double v, double b)
{
    uint32_t r;
    asm("{\n\t.reg .pred p, q;\n\tsetp.gt.f64 p, %1, %2;\n\tsetp.nan.f64 q, %1, %1;\n\tor.pred p, p, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "d"(v), "d"(b));
    return r;
}

// The fused forward forms are numbered by one template argument: -1 none (plain compressor), DT (0..3) keep
// what exceeds the threshold (tau = 0: ReLU), 4 + DT ReLU6, and for the 2-byte types 8 + DT the ReLU and 12 + DT
// the ReLU6 decided by compares in the element's own type.
constexpr int kFusedRelu6     = 4;
constexpr int kFusedReluHalf  = 8;
constexpr int kFusedRelu6Half = 12;

// ReLU and ReLU6 of a 2-byte element (x: its pattern, possibly sign-extended) without widening it, by binary16 /
// bfloat16 compare instructions: kept iff x > 0 or x is a NaN -- exactly the elements for which x <= 0 is false
// under IEEE comparison --, saturated iff x >= 6 (false for a NaN).  One instruction per decision instead of a
// conversion, a float compare, a select and the zero test, and not on the integer pipe that the rest of the
// compaction step loads (integer compares of the bit pattern, two per decision, measured slower than the float
// form without the dense output; these are faster than both, with and without it).
template <int DT>
__device__ __forceinline__ bool relu_keeps_half(const uint32_t x)
{
    static_assert(DT == BT_F16 || DT == BT_BF16, "2-byte element types");
    uint32_t r;
    if constexpr (DT == BT_F16)
        asm("{\n\t.reg .pred p;\n\t.reg .b16 h, z;\n\tcvt.u16.u32 h, %1;\n\tmov.b16 z, 0;\n\tsetp.gtu.f16 p, h, z;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "r"(x));
    else
        asm("{\n\t.reg .pred p;\n\t.reg .b16 h, z;\n\tcvt.u16.u32 h, %1;\n\tmov.b16 z, 0;\n\tsetp.gtu.bf16 p, h, z;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "r"(x));
    return r != 0;
}
template <int DT>
__device__ __forceinline__ bool relu6_saturates_half(const uint32_t x)
{
    static_assert(DT == BT_F16 || DT == BT_BF16, "2-byte element types");
    uint32_t r;
    if constexpr (DT == BT_F16)
        asm("{\n\t.reg .pred p;\n\t.reg .b16 h, z;\n\tcvt.u16.u32 h, %1;\n\tmov.b16 z, 0x4600;\n\tsetp.ge.f16 p, h, z;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "r"(x));
    else
        asm("{\n\t.reg .pred p;\n\t.reg .b16 h, z;\n\tcvt.u16.u32 h, %1;\n\tmov.b16 z, 0x40C0;\n\tsetp.ge.bf16 p, h, z;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "r"(x));
    return r != 0;
}

// y = (x <= tau) ? +0 : x, and for ReLU6 additionally 6 where x >= 6; IEEE comparisons, so a NaN is kept.
template <int FUSED, typename R>
__device__ __forceinline__ R fused_forward(R x, float tau)
{
    constexpr int DT   = FUSED & 3;
    const auto    v    = Elem<DT>::widen(x);
    const bool    drop = v <= static_cast<decltype(v)>(tau);
    if constexpr (FUSED >= kFusedRelu6) {
        const uint32_t saturated = at_least_six(v);
        x                        = saturated ? static_cast<R>(Elem<DT>::kSix) : x;     // selects, no branches
    }
    return drop ? R(0) : x;
}

}  // namespace bt
