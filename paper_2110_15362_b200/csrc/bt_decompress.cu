// Algorithm 2 (bitmap -> dense), chunk-parallel.  The single running counter j
// of the algorithm is replaced by chunk_prefix[c] plus popcounts inside the
// chunk, so every warp decodes its 1024 elements without talking to any other.
//
// One warp, one quarter chunk (1024 elements = 32 bitmap words):
//   - lane l loads the 4 words 4l..4l+3 of the WHOLE chunk (one 512-byte
//     coalesced read, issued together with the read of chunk_prefix[c]); the
//     popcounts of the lanes in front of this warp's quarter give the count in
//     front of it, and four shuffles hand lane l word l of its own quarter, so
//     the only dependent round trip left is the gather itself;
//   - a warp scan of the 32 word popcounts gives word offsets;
//   - the quarter is written with 16-byte stores: a lane owns kE consecutive
//     elements, i.e. kE consecutive bits of one word; the rank of its first set
//     bit is  chunk base + quarter base + word offset + popc(lower bits of the
//     word),  and the set bits gather from values[] at consecutive addresses.
#include <type_traits>

#include "bt_internal.cuh"
#include "bt_quarter16.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull = 0xFFFFFFFFu;

// kE: elements a lane decodes per step (a multiple of one 16-byte vector: 2 for 8-byte, 4 for 4-byte, 8 for 2-byte elements)
// WIDEN: 0, or the 16-bit type of the stashed values of a binary32 tensor (1 binary16, 2 bfloat16): the value
// is widened exactly on its way out (the restore side of the down-cast on stash).
template <int WIDEN>
__device__ __forceinline__ uint32_t widened(const uint16_t h)
{
    if constexpr (WIDEN == 1) {
        // exponent and mantissa moved into place, then rebiased by an exact multiplication (subnormals included);
        // infinities and NaNs get the all-ones exponent by hand, which keeps a NaN payload and sign
        const uint32_t t = static_cast<uint32_t>(h & 0x7FFFu) << 13;
        uint32_t       r = __float_as_uint(__uint_as_float(t) * 5.192296858534828e33f);      // 2^112
        r                = (h & 0x7C00u) == 0x7C00u ? (t | 0x7F800000u) : r;
        return r | (static_cast<uint32_t>(h & 0x8000u) << 16);
    } else {
        return static_cast<uint32_t>(h) << 16;
    }
}

// One tensor restored by a batched launch (see decompress_batch_kernel).
struct RestoreJob {
    const uint32_t *bitmap;
    const void     *values;
    const uint64_t *values_offset;  // NULL, or the device word holding the byte offset of the values inside `values`
    const uint64_t *prefix;
    void           *out;
    uint64_t        n;
    uint32_t        first_block;    // the launch's blocks [first_block, next job's first_block) restore this tensor
};
template <int kJobs>
struct RestoreParams {
    RestoreJob job[kJobs];
    uint32_t   jobs;
};

// `block`: index of this CTA among those that restore the tensor
template <typename U, int kE, int kGrp, int kWarps>
__device__ __forceinline__ void
decompress_body(const uint32_t *__restrict__ bitmap, const U *values,
                const uint64_t *__restrict__ values_offset, const uint64_t *__restrict__ prefix, const uint64_t n,
                U *__restrict__ out, const uint64_t block)
{
    constexpr int kVec          = 16 / sizeof(U);          // elements per 16-byte store
    constexpr int kLanesPerWord = 32 / kE;                 // lanes that share one bitmap word
    constexpr int kWordsPerStep = kE;                      // words one warp-wide step covers (32 * kE / 32)
    constexpr int kSteps        = 32 / kWordsPerStep;
    static_assert(kE % kVec == 0 && 32 % kE == 0 && kE < 32, "a lane takes whole vectors of one word");

    const uint32_t lane        = threadIdx.x & 31u;
    const uint64_t warp_global = block * kWarps + (threadIdx.x >> 5);
    const uint64_t quarters    = (n + 1023) >> 10;
    if (warp_global >= quarters) return;

    const uint64_t chunk       = warp_global >> 2;
    const uint32_t q           = static_cast<uint32_t>(warp_global & 3u);
    const uint64_t words_total = (n + 31) >> 5;
    const uint64_t w0          = chunk * 128 + 4 * lane;   // this lane's four words of the chunk

    // the chunk's 128 words (zero past the end of the bitmap) and its prefix entry: independent loads
    const uint4 w4 = load_words4(bitmap, w0, words_total);
    const uint64_t chunk_base = prefix[chunk];
    // arena form: the packed values start *values_offset bytes into `values`
    using V = U;
    if (values_offset) values = reinterpret_cast<const V *>(reinterpret_cast<const unsigned char *>(values) + *values_offset);

    // non-zeros of the chunk in front of this quarter
    uint32_t before = lane < 8 * q ? __popc(w4.x) + __popc(w4.y) + __popc(w4.z) + __popc(w4.w) : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(kFull, before, o);

    // lane l takes word l of its own quarter: component l & 3 of lane 8q + (l >> 2)
    const int      src = 8 * q + (lane >> 2);
    const uint32_t c0 = __shfl_sync(kFull, w4.x, src), c1 = __shfl_sync(kFull, w4.y, src);
    const uint32_t c2 = __shfl_sync(kFull, w4.z, src), c3 = __shfl_sync(kFull, w4.w, src);
    const uint32_t word = (lane & 2u) ? ((lane & 1u) ? c3 : c2) : ((lane & 1u) ? c1 : c0);

    uint32_t incl = __popc(word);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(kFull, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += u;
    }
    const uint32_t excl = incl - __popc(word);
    const V *const vp   = values + (chunk_base + before);   // packed values of this quarter

    const uint64_t e0    = warp_global << 10;               // first element of the quarter
    const uint32_t shift = (lane % kLanesPerWord) * kE;     // which kE-bit group of the word
    const Extent   ox    = extent_of(out, n * sizeof(U));
    // the gathers of kGrp steps are issued before their stores, so that a lane has kGrp * kE independent loads
    // in flight.  All 32 of the quarter (kGrp = kSteps) is the setting used: smaller groups raise the occupancy
    // and are 2 % faster on a 1 GiB tensor, but 10 % slower on the few-MB layers of a ResNet, whose cold
    // gathers need the depth.
    static_assert(kSteps % kGrp == 0, "whole groups of steps");
    U e[kGrp][kE];
#pragma unroll
    for (int k0 = 0; k0 < kSteps; k0 += kGrp) {
#pragma unroll
    for (int kk = 0; kk < kGrp; ++kk) {
        const int      k    = k0 + kk;
        const int      from = k * kWordsPerStep + lane / kLanesPerWord;
        const uint32_t w    = __shfl_sync(kFull, word, from);
        const uint32_t wex  = __shfl_sync(kFull, excl, from);
        const uint32_t bits = (w >> shift) & ((1u << kE) - 1u);
        uint32_t       off  = wex + __popc(w & ((1u << shift) - 1u));
#pragma unroll
        for (int j = 0; j < kE; ++j) {
            const bool set = (bits >> j) & 1u;
            e[kk][j] = set ? vp[off] : U(0);
            off += set;
        }
    }
#pragma unroll
    for (int kk = 0; kk < kGrp; ++kk) {
        const int      k  = k0 + kk;
        const uint64_t eo = e0 + static_cast<uint64_t>(k) * (32 * kE) + lane * kE;
#pragma unroll
        for (int v = 0; v < kE / kVec; ++v) {
            const uint64_t at = eo + v * kVec;
            const U       *ev = e[kk] + v * kVec;
            if (at + kVec <= n) {
                uint4 pack;
                if constexpr (kVec == 2) {
                    pack = make_uint4(static_cast<uint32_t>(ev[0]), static_cast<uint32_t>(ev[0] >> 32),
                                      static_cast<uint32_t>(ev[1]), static_cast<uint32_t>(ev[1] >> 32));
                } else if constexpr (kVec == 4) {
                    pack = make_uint4(ev[0], ev[1], ev[2], ev[3]);
                } else {
                    pack = make_uint4(ev[0] | (uint32_t(ev[1]) << 16), ev[2] | (uint32_t(ev[3]) << 16),
                                      ev[4] | (uint32_t(ev[5]) << 16), ev[6] | (uint32_t(ev[7]) << 16));
                }
                if (ox.holds(out + at, 16)) *reinterpret_cast<uint4 *>(out + at) = pack;
            } else {
#pragma unroll
                for (int j = 0; j < kVec; ++j)
                    if (at + j < n && ox.holds(out + at + j, sizeof(U))) out[at + j] = ev[j];
            }
        }
    }
    }
}

// ---------------------------------------------------------------------------------------------
// The decompressor for 2-byte elements: the quarter's packed run staged in shared memory, expanded from there
// (bt_quarter16.cuh).  WIDEN: 0 restores 2-byte elements; 1 (binary16) / 2 (bfloat16) widens every restored value
// to binary32 on its way out.
template <int kWarps, int WIDEN = 0>
__device__ __forceinline__ void
decompress16_body(const uint32_t *__restrict__ bitmap, const uint16_t *values, const uint64_t *__restrict__ values_offset,
                  const uint64_t *__restrict__ prefix, const uint64_t n,
                  std::conditional_t<WIDEN != 0, uint32_t, uint16_t> *__restrict__ out, const uint64_t block)
{
    q16::Quarter qt;
    if (!q16::stage_quarter<kWarps>(bitmap, values, values_offset, prefix, n, block, qt)) return;
    const uint32_t lane = threadIdx.x & 31u;
    const Extent   ox   = extent_of(out, n * sizeof(*out));
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        uint32_t       bits;
        const uint2    v  = q16::expand_step(qt, k, lane, bits);
        const uint64_t at = qt.e0 + static_cast<uint64_t>(k) * 128 + lane * 4;
        if constexpr (WIDEN == 0) {
            if (qt.whole || at + 4 <= n) {
                if (ox.holds(out + at, 8)) *reinterpret_cast<uint2 *>(out + at) = v;
            } else {
                const uint32_t h[2] = {v.x, v.y};
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (at + j < n && ox.holds(out + at + j, 2)) out[at + j] = static_cast<uint16_t>(h[j >> 1] >> (16 * (j & 1)));
            }
        } else {
            // a clear bit gave the pattern 0, which widens to +0
            uint32_t f[4];
            if constexpr (WIDEN == 2) {
                f[0] = v.x << 16, f[1] = v.x & 0xFFFF0000u, f[2] = v.y << 16, f[3] = v.y & 0xFFFF0000u;
            } else {
                f[0] = widened<WIDEN>(static_cast<uint16_t>(v.x)), f[1] = widened<WIDEN>(static_cast<uint16_t>(v.x >> 16));
                f[2] = widened<WIDEN>(static_cast<uint16_t>(v.y)), f[3] = widened<WIDEN>(static_cast<uint16_t>(v.y >> 16));
            }
            if (qt.whole || at + 4 <= n) {
                if (ox.holds(out + at, 16)) *reinterpret_cast<uint4 *>(out + at) = make_uint4(f[0], f[1], f[2], f[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (at + j < n && ox.holds(out + at + j, 4)) out[at + j] = f[j];
            }
        }
    }
}

template <typename U, int kE, int kGrp, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
decompress_kernel(const uint32_t *__restrict__ bitmap, const U *values,
                  const uint64_t *__restrict__ values_offset, const uint64_t *__restrict__ prefix, const uint64_t n,
                  U *__restrict__ out)
{
    decompress_body<U, kE, kGrp, kWarps>(bitmap, values, values_offset, prefix, n, out, blockIdx.x);
}

template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1536 / (kWarps * 32))
decompress16_kernel(const uint32_t *__restrict__ bitmap, const uint16_t *values, const uint64_t *__restrict__ values_offset,
                    const uint64_t *__restrict__ prefix, const uint64_t n, uint16_t *__restrict__ out)
{
    decompress16_body<kWarps>(bitmap, values, values_offset, prefix, n, out, blockIdx.x);
}

template <int kWarps, int WIDEN>
__global__ void __launch_bounds__(kWarps * 32, 1536 / (kWarps * 32))
decompress16_widen_kernel(const uint32_t *__restrict__ bitmap, const uint16_t *values, const uint64_t *__restrict__ values_offset,
                          const uint64_t *__restrict__ prefix, const uint64_t n, uint32_t *__restrict__ out)
{
    decompress16_body<kWarps, WIDEN>(bitmap, values, values_offset, prefix, n, out, blockIdx.x);
}

// The tensor a CTA of a batched launch works on: the last job whose first block is not behind this one.
template <int kJobs>
__device__ __forceinline__ uint32_t job_of_block(const RestoreParams<kJobs> &p)
{
    uint32_t k = 0;
    for (uint32_t j = 1; j < p.jobs; ++j) k = p.job[j].first_block <= blockIdx.x ? j : k;
    return k;
}

// Several tensors of one element type restored by ONE launch: every CTA looks up its tensor in the job table (in
// the kernel's parameters) and restores its four quarters of it exactly as the single-tensor kernel does.
template <typename U, int kE, int kGrp, int kWarps, int kJobs>
__global__ void __launch_bounds__(kWarps * 32)
decompress_batch_kernel(const __grid_constant__ RestoreParams<kJobs> p)
{
    const RestoreJob &j = p.job[job_of_block(p)];
    decompress_body<U, kE, kGrp, kWarps>(j.bitmap, static_cast<const U *>(j.values), j.values_offset, j.prefix, j.n, static_cast<U *>(j.out),
                                            blockIdx.x - j.first_block);
}

template <int kWarps, int kJobs>
__global__ void __launch_bounds__(kWarps * 32, 1536 / (kWarps * 32))
decompress16_batch_kernel(const __grid_constant__ RestoreParams<kJobs> p)
{
    const RestoreJob &j = p.job[job_of_block(p)];
    decompress16_body<kWarps>(j.bitmap, static_cast<const uint16_t *>(j.values), j.values_offset, j.prefix, j.n, static_cast<uint16_t *>(j.out),
                              blockIdx.x - j.first_block);
}

template <typename U, int kE, int kGrp>
cudaError_t launch_typed(const uint32_t *bitmap, const void *values, const uint64_t *values_offset,
                         const uint64_t *prefix, uint64_t n, void *out, cudaStream_t stream)
{
    constexpr int  kWarps   = 4;   // four warps per CTA: 3 % faster than eight on few-MB tensors, 1.5 % on 1 GiB (two: the same)
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    decompress_kernel<U, kE, kGrp, kWarps><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
        bitmap, static_cast<const U *>(values), values_offset, prefix, n, static_cast<U *>(out));
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decompress_widen(const uint32_t *bitmap, const void *values16, const uint64_t *values_offset,
                                    const uint64_t *prefix, uint64_t n, int from_dtype, void *out_f32, cudaStream_t stream)
{
    constexpr int  kWarps   = 4;
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    const auto *v = static_cast<const uint16_t *>(values16);
    auto       *o = static_cast<uint32_t *>(out_f32);
    // the 2-byte decompressor (packed run staged in shared memory) with the widening in its store path
    if (from_dtype == BT_F16) decompress16_widen_kernel<kWarps, 1><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(bitmap, v, values_offset, prefix, n, o);
    else decompress16_widen_kernel<kWarps, 2><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(bitmap, v, values_offset, prefix, n, o);
    return cudaGetLastError();
}

cudaError_t launch_decompress(const uint32_t *bitmap, const void *values, const uint64_t *values_offset,
                              const uint64_t *prefix, uint64_t n, int elem_size, void *out, cudaStream_t stream)
{
    if (elem_size == 8) return launch_typed<uint64_t, 2, 16>(bitmap, values, values_offset, prefix, n, out, stream);
    if (elem_size == 4) return launch_typed<uint32_t, 4, 8>(bitmap, values, values_offset, prefix, n, out, stream);
    constexpr int  kWarps   = 4;
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    decompress16_kernel<kWarps><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
        bitmap, static_cast<const uint16_t *>(values), values_offset, prefix, n, static_cast<uint16_t *>(out));
    return cudaGetLastError();
}

cudaError_t launch_decompress_batch(const DecompressJob *jobs, uint32_t count, int elem_size, cudaStream_t stream)
{
    constexpr int kWarps = 4;
    if (count == 0 || count > kMaxBatch) return cudaErrorInvalidValue;
    RestoreParams<kMaxBatch> p{};
    uint64_t                 blocks = 0;
    for (uint32_t k = 0; k < count; ++k) {
        const uint64_t quarters = (jobs[k].n + 1023) >> 10;
        p.job[k] = RestoreJob{jobs[k].bitmap, jobs[k].values, jobs[k].values_offset, jobs[k].prefix, jobs[k].out, jobs[k].n, static_cast<uint32_t>(blocks)};
        blocks += (quarters + kWarps - 1) / kWarps;
        if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    }
    p.jobs = count;
    const unsigned grid = static_cast<unsigned>(blocks);
    if (elem_size == 8) decompress_batch_kernel<uint64_t, 2, 16, kWarps, kMaxBatch><<<grid, kWarps * 32, 0, stream>>>(p);
    else if (elem_size == 4) decompress_batch_kernel<uint32_t, 4, 8, kWarps, kMaxBatch><<<grid, kWarps * 32, 0, stream>>>(p);
    else decompress16_batch_kernel<kWarps, kMaxBatch><<<grid, kWarps * 32, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace bt
