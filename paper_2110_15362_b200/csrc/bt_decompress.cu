// Algorithm 2 (bitmap -> dense), chunk-parallel.  The single running counter j
// of the algorithm is replaced by chunk_prefix[c] plus popcounts inside the
// chunk, so every warp decodes its 1024 elements without talking to any other.
//
// One warp, one quarter chunk (1024 elements = 32 bitmap words):
//   - lane l loads the 4 words 4l..4l+3 of the WHOLE chunk (one 512-byte
//     coalesced read) to count the non-zeros in front of this warp's quarter;
//   - lane l keeps word l of its own quarter and an exclusive scan of the 32
//     word popcounts;
//   - the quarter is written with 16-byte stores: per store a lane owns kVec
//     consecutive elements, i.e. kVec consecutive bits of one word; the rank
//     of its first set bit is  chunk base + warp base + word offset +
//     popc(lower bits of the word),  and the set bits gather from values[].
#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull = 0xFFFFFFFFu;

template <typename U>
struct Vec16;
template <>
struct Vec16<uint32_t> {
    static constexpr int kVec = 4;
};
template <>
struct Vec16<uint16_t> {
    static constexpr int kVec = 8;
};

template <typename U, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
decompress_kernel(const uint32_t *__restrict__ bitmap, const U *__restrict__ values,
                  const uint64_t *__restrict__ prefix, const uint64_t n, U *__restrict__ out)
{
    constexpr int kVec          = Vec16<U>::kVec;          // elements per 16-byte store
    constexpr int kLanesPerWord = 32 / kVec;               // lanes that share one bitmap word
    constexpr int kWordsPerStep = 32 / kLanesPerWord;      // words one warp-wide store covers
    constexpr int kSteps        = 32 / kWordsPerStep;

    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp_global = static_cast<uint64_t>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    const uint64_t quarters = (n + 1023) >> 10;
    if (warp_global >= quarters) return;

    const uint64_t chunk = warp_global >> 2;
    const uint32_t q     = static_cast<uint32_t>(warp_global & 3u);
    const uint64_t words_total = (n + 31) >> 5;
    const uint64_t cw0 = chunk * 128;                      // first word of the chunk

    // non-zeros of the chunk in front of this quarter
    uint32_t before = 0;
    if (q != 0 && lane < 8 * q) {
        const uint4 w4 = *reinterpret_cast<const uint4 *>(bitmap + cw0 + 4 * lane);   // whole quarters precede: in range
        before = __popc(w4.x) + __popc(w4.y) + __popc(w4.z) + __popc(w4.w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(kFull, before, o);

    const uint64_t wi   = cw0 + 32 * q + lane;
    const uint32_t word = wi < words_total ? bitmap[wi] : 0u;
    uint32_t       incl = __popc(word);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(kFull, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += u;
    }
    const uint32_t excl = incl - __popc(word);
    const uint64_t base = prefix[chunk] + before;

    const uint64_t e0      = warp_global << 10;            // first element of the quarter
    const uint32_t sub     = lane % kLanesPerWord;         // which kVec-bit group of the word
    const uint32_t shift   = sub * kVec;
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        const int      src_lane = k * kWordsPerStep + lane / kLanesPerWord;
        const uint32_t w        = __shfl_sync(kFull, word, src_lane);
        const uint32_t wex      = __shfl_sync(kFull, excl, src_lane);
        const uint32_t bits     = (w >> shift) & ((1u << kVec) - 1u);
        uint64_t       idx      = base + wex + __popc(w & ((1u << shift) - 1u));
        U              e[kVec];
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            const bool set = (bits >> j) & 1u;
            e[j]           = set ? values[idx] : U(0);
            idx += set;
        }
        const uint64_t eo = e0 + static_cast<uint64_t>(k) * (32 * kVec) + lane * kVec;
        if (eo + kVec <= n) {
            uint4 pack;
            if constexpr (kVec == 4) {
                pack = make_uint4(e[0], e[1], e[2], e[3]);
            } else {
                pack = make_uint4(e[0] | (uint32_t(e[1]) << 16), e[2] | (uint32_t(e[3]) << 16),
                                  e[4] | (uint32_t(e[5]) << 16), e[6] | (uint32_t(e[7]) << 16));
            }
            *reinterpret_cast<uint4 *>(out + eo) = pack;
        } else {
#pragma unroll
            for (int j = 0; j < kVec; ++j)
                if (eo + j < n) out[eo + j] = e[j];
        }
    }
}

template <typename U>
cudaError_t launch_typed(const uint32_t *bitmap, const void *values, const uint64_t *prefix, uint64_t n, void *out,
                         cudaStream_t stream)
{
    constexpr int  kWarps   = 8;
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    decompress_kernel<U, kWarps><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
        bitmap, static_cast<const U *>(values), prefix, n, static_cast<U *>(out));
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decompress(const uint32_t *bitmap, const void *values, const uint64_t *prefix, uint64_t n,
                              int elem_size, void *out, cudaStream_t stream)
{
    return elem_size == 4 ? launch_typed<uint32_t>(bitmap, values, prefix, n, out, stream)
                          : launch_typed<uint16_t>(bitmap, values, prefix, n, out, stream);
}

}  // namespace bt
