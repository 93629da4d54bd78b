// ReLU backward from the stashed bitmap: grad_in[i] = bit i ? grad_out[i] : +0.
// A pure streaming select: every thread moves 16-byte vectors (2 fp64, 4 fp32 or
// 8 16-bit elements, i.e. 2, 4 or 8 consecutive bits of one bitmap word), several
// independent vectors in flight per thread.
#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll  = 2;   // independent 16-byte vectors per thread (four: 1.6 % slower on few-MB tensors, the same on 1 GiB)

template <typename U>
__device__ __forceinline__ uint4 select_vec(uint4 g, uint32_t bits);

template <>
__device__ __forceinline__ uint4 select_vec<uint32_t>(uint4 g, uint32_t bits)
{
    g.x = (bits & 1u) ? g.x : 0u;
    g.y = (bits & 2u) ? g.y : 0u;
    g.z = (bits & 4u) ? g.z : 0u;
    g.w = (bits & 8u) ? g.w : 0u;
    return g;
}

template <>
__device__ __forceinline__ uint4 select_vec<uint64_t>(uint4 g, uint32_t bits)
{
    if (!(bits & 1u)) g.x = g.y = 0u;
    if (!(bits & 2u)) g.z = g.w = 0u;
    return g;
}

// two 16-bit lanes per register: build a byte-pair mask from two bits
__device__ __forceinline__ uint32_t mask2(uint32_t two_bits)
{
    return ((two_bits & 1u) ? 0x0000FFFFu : 0u) | ((two_bits & 2u) ? 0xFFFF0000u : 0u);
}

template <>
__device__ __forceinline__ uint4 select_vec<uint16_t>(uint4 g, uint32_t bits)
{
    g.x &= mask2(bits);
    g.y &= mask2(bits >> 2);
    g.z &= mask2(bits >> 4);
    g.w &= mask2(bits >> 6);
    return g;
}

// `block`: index of this CTA among those that work on the tensor
template <typename U>
__device__ __forceinline__ void relu_bwd_body(const uint32_t *__restrict__ bitmap, const U *gout, const uint64_t n, U *gin,
                                              const uint64_t block)
{
    constexpr int      kVec  = 16 / sizeof(U);
    constexpr uint32_t kMask = (1u << kVec) - 1u;
    const uint64_t vecs      = n / kVec;                       // whole 16-byte vectors
    const uint64_t block0    = block * (kThreads * kUnroll);

    const Extent ox = extent_of(gin, n * sizeof(U));
    uint4    g[kUnroll];
    uint32_t w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const uint64_t v = block0 + u * kThreads + threadIdx.x;
        if (v < vecs) {
            g[u] = reinterpret_cast<const uint4 *>(gout)[v];
            w[u] = bitmap[(v * kVec) >> 5];
        }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const uint64_t v = block0 + u * kThreads + threadIdx.x;
        if (v < vecs) {
            const uint32_t bits = (w[u] >> ((v * kVec) & 31u)) & kMask;
            if (ox.holds(reinterpret_cast<uint4 *>(gin) + v, 16)) reinterpret_cast<uint4 *>(gin)[v] = select_vec<U>(g[u], bits);
        }
    }
    // the last n % kVec elements, one by one
    if (block == 0 && threadIdx.x < n - vecs * kVec) {
        const uint64_t i = vecs * kVec + threadIdx.x;
        const bool set   = (bitmap[i >> 5] >> (i & 31u)) & 1u;
        if (ox.holds(gin + i, sizeof(U))) gin[i] = set ? gout[i] : U(0);
    }
}

template <typename U>
__global__ void __launch_bounds__(kThreads)
relu_bwd_kernel(const uint32_t *__restrict__ bitmap, const U *gout, const uint64_t n, U *gin)
{
    relu_bwd_body<U>(bitmap, gout, n, gin, blockIdx.x);
}

// Several tensors of one element type in ONE launch: every CTA looks up its tensor in the job table (in the
// kernel's parameters) and masks its share of that tensor's gradient exactly as the single-tensor kernel does.
struct MaskJob {
    const uint32_t *bitmap;
    const void     *gout;
    void           *gin;
    uint64_t        n;
    uint32_t        first_block;
};
template <int kJobs>
struct MaskParams {
    MaskJob  job[kJobs];
    uint32_t jobs;
};

template <typename U, int kJobs>
__global__ void __launch_bounds__(kThreads)
relu_bwd_batch_kernel(const __grid_constant__ MaskParams<kJobs> p)
{
    uint32_t k = 0;
    for (uint32_t j = 1; j < p.jobs; ++j) k = p.job[j].first_block <= blockIdx.x ? j : k;
    const MaskJob &j = p.job[k];
    relu_bwd_body<U>(j.bitmap, static_cast<const U *>(j.gout), j.n, static_cast<U *>(j.gin), blockIdx.x - j.first_block);
}

template <typename U>
cudaError_t launch_typed(const uint32_t *bitmap, const void *gout, uint64_t n, void *gin, cudaStream_t stream)
{
    constexpr int  kVec = 16 / sizeof(U);
    const uint64_t vecs = n / kVec;
    uint64_t       grid = (vecs + kThreads * kUnroll - 1) / (kThreads * kUnroll);
    if (grid == 0) grid = 1;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    relu_bwd_kernel<U><<<static_cast<unsigned>(grid), kThreads, 0, stream>>>(bitmap, static_cast<const U *>(gout), n,
                                                                             static_cast<U *>(gin));
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_relu_bwd(const uint32_t *bitmap, const void *gout, uint64_t n, int elem_size, void *gin,
                            cudaStream_t stream)
{
    return elem_size == 8   ? launch_typed<uint64_t>(bitmap, gout, n, gin, stream)
           : elem_size == 4 ? launch_typed<uint32_t>(bitmap, gout, n, gin, stream)
                            : launch_typed<uint16_t>(bitmap, gout, n, gin, stream);
}

cudaError_t launch_relu_bwd_batch(const DecompressJob *jobs, uint32_t count, int elem_size, cudaStream_t stream)
{
    if (count == 0 || count > kMaxBatch) return cudaErrorInvalidValue;
    MaskParams<kMaxBatch> p{};
    uint64_t              blocks = 0;
    for (uint32_t k = 0; k < count; ++k) {
        const uint64_t vecs = jobs[k].n / (16 / elem_size);
        uint64_t       g    = (vecs + kThreads * kUnroll - 1) / (kThreads * kUnroll);
        if (g == 0) g = 1;
        p.job[k] = MaskJob{jobs[k].bitmap, jobs[k].in, jobs[k].out, jobs[k].n, static_cast<uint32_t>(blocks)};
        blocks += g;
        if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    }
    p.jobs = count;
    const unsigned grid = static_cast<unsigned>(blocks);
    if (elem_size == 8) relu_bwd_batch_kernel<uint64_t, kMaxBatch><<<grid, kThreads, 0, stream>>>(p);
    else if (elem_size == 4) relu_bwd_batch_kernel<uint32_t, kMaxBatch><<<grid, kThreads, 0, stream>>>(p);
    else relu_bwd_batch_kernel<uint16_t, kMaxBatch><<<grid, kThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace bt
