// Double-mask batch normalisation support (section 3.1): the zero pattern of a
// normalisation layer's input, which that input's stash already holds as a
// bitmap, is applied to the layer's output.  The output's stash reuses the
// bitmap and its chunk prefix array, so all this pass has to produce is the
// vector of values: x[i] at every set bit, in element order.
//
// Ranks come from the existing prefix array plus popcounts inside the chunk, so
// there is no scan and no communication: the mirror image of the decompressor.
// One warp, one quarter chunk (1024 elements = 32 bitmap words):
//   - lane l loads the 4 words 4l..4l+3 of the WHOLE chunk together with
//     chunk_prefix[c]; the popcounts of the lanes in front of this warp's quarter
//     give the count in front of it, four shuffles hand lane l word l of its own
//     quarter, a warp scan of the 32 word popcounts gives word offsets;
//   - the quarter of x is read with 16-byte loads (all of them issued before the
//     first store): a lane owns kE consecutive elements, i.e. kE consecutive bits
//     of one word; the rank of its first set bit is  chunk base + quarter base +
//     word offset + popc(lower bits of the word);  its set elements go to the
//     warp's staging area in shared memory at that rank (the lanes' runs abut),
//     shifted so that a staged element and its place in values[] have the same
//     position within a 16-byte vector;
//   - the staged run leaves for values[] with 16-byte stores (single elements at
//     its ragged ends): scattered 2-byte stores straight to global memory ran at
//     a third of the bandwidth;
//   - optionally the masked dense tensor leaves with 16-byte stores.
#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull = 0xFFFFFFFFu;

// A 16-byte vector of elements to and from its elements (element 0 at the lowest address).
template <typename U>
__device__ __forceinline__ void unpack_vec(const uint4 pack, U *ev)
{
    if constexpr (sizeof(U) == 8) {
        ev[0] = pack.x | (static_cast<uint64_t>(pack.y) << 32);
        ev[1] = pack.z | (static_cast<uint64_t>(pack.w) << 32);
    } else if constexpr (sizeof(U) == 4) {
        ev[0] = pack.x, ev[1] = pack.y, ev[2] = pack.z, ev[3] = pack.w;
    } else {
        ev[0] = static_cast<U>(pack.x), ev[1] = static_cast<U>(pack.x >> 16);
        ev[2] = static_cast<U>(pack.y), ev[3] = static_cast<U>(pack.y >> 16);
        ev[4] = static_cast<U>(pack.z), ev[5] = static_cast<U>(pack.z >> 16);
        ev[6] = static_cast<U>(pack.w), ev[7] = static_cast<U>(pack.w >> 16);
    }
}
template <typename U>
__device__ __forceinline__ uint4 pack_vec(const U *ev)
{
    if constexpr (sizeof(U) == 8)
        return make_uint4(static_cast<uint32_t>(ev[0]), static_cast<uint32_t>(ev[0] >> 32), static_cast<uint32_t>(ev[1]),
                          static_cast<uint32_t>(ev[1] >> 32));
    else if constexpr (sizeof(U) == 4)
        return make_uint4(ev[0], ev[1], ev[2], ev[3]);
    else
        return make_uint4(ev[0] | (uint32_t(ev[1]) << 16), ev[2] | (uint32_t(ev[3]) << 16), ev[4] | (uint32_t(ev[5]) << 16),
                          ev[6] | (uint32_t(ev[7]) << 16));
}

template <typename U, int kE, int kWarps, bool WRITE_Y>
__global__ void __launch_bounds__(kWarps * 32)
mask_gather_kernel(const U *x, const uint32_t *__restrict__ bitmap, const uint64_t *__restrict__ prefix,
                   const uint64_t n, U *y, U *__restrict__ values, const uint64_t capacity)   // y may alias x
{
    constexpr int kVec          = 16 / sizeof(U);          // elements per 16-byte vector
    constexpr int kLanesPerWord = 32 / kE;
    constexpr int kWordsPerStep = kE;
    constexpr int kSteps        = 32 / kWordsPerStep;
    static_assert(kE % kVec == 0 && 32 % kE == 0 && kE < 32, "a lane takes whole vectors of one word");

    const uint32_t lane        = threadIdx.x & 31u;
    const uint64_t warp_global = static_cast<uint64_t>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    const uint64_t quarters    = (n + 1023) >> 10;
    if (warp_global >= quarters) return;

    const uint64_t chunk       = warp_global >> 2;
    const uint32_t q           = static_cast<uint32_t>(warp_global & 3u);
    const uint64_t words_total = (n + 31) >> 5;
    const uint64_t w0          = chunk * 128 + 4 * lane;   // this lane's four words of the chunk
    const uint64_t e0          = warp_global << 10;        // first element of the quarter

    // the quarter of x first: these loads do not depend on the bitmap.  2-byte elements stay in their 16-byte
    // vectors until their step comes (unpacked at once they hold 32 registers per lane and cost occupancy: 56 -> 40
    // registers, 0.142 -> 0.127 ms on a 392 MiB tensor); wider elements are unpacked at once (8-byte elements
    // measured 25 % slower the other way).
    constexpr bool kLate = sizeof(U) == 2;
    uint4 xv[kLate ? kSteps : 1][kE / kVec];
    U     xe[kLate ? 1 : kSteps][kE];
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        const uint64_t eo = e0 + static_cast<uint64_t>(k) * (32 * kE) + lane * kE;
#pragma unroll
        for (int v = 0; v < kE / kVec; ++v) {
            const uint64_t at = eo + v * kVec;
            if constexpr (kLate) {
                if (at + kVec <= n) {
                    xv[k][v] = *reinterpret_cast<const uint4 *>(x + at);
                } else {
                    U t[kVec];
#pragma unroll
                    for (int j = 0; j < kVec; ++j) t[j] = at + j < n ? x[at + j] : U(0);
                    xv[k][v] = pack_vec<U>(t);
                }
            } else {
                U *ev = xe[k] + v * kVec;
                if (at + kVec <= n) {
                    unpack_vec<U>(*reinterpret_cast<const uint4 *>(x + at), ev);
                } else {
#pragma unroll
                    for (int j = 0; j < kVec; ++j) ev[j] = at + j < n ? x[at + j] : U(0);
                }
            }
        }
    }

    // the chunk's 128 words (zero past the end of the bitmap) and its prefix entry
    const uint4 w4 = load_words4(bitmap, w0, words_total);
    const uint64_t chunk_base = prefix[chunk];

    uint32_t before = lane < 8 * q ? __popc(w4.x) + __popc(w4.y) + __popc(w4.z) + __popc(w4.w) : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(kFull, before, o);

    // lane l takes word l of its own quarter: component l & 3 of lane 8q + (l >> 2)
    const int      src = 8 * q + (lane >> 2);
    const uint32_t c0 = __shfl_sync(kFull, w4.x, src), c1 = __shfl_sync(kFull, w4.y, src);
    const uint32_t c2 = __shfl_sync(kFull, w4.z, src), c3 = __shfl_sync(kFull, w4.w, src);
    uint32_t       word = (lane & 2u) ? ((lane & 1u) ? c3 : c2) : ((lane & 1u) ? c1 : c0);
    // bits past the end of the tensor do not count (a well-formed bitmap has none)
    const uint64_t word_first = e0 + 32ull * lane;
    if (word_first >= n) word = 0;
    else if (n - word_first < 32) word &= (1u << static_cast<uint32_t>(n - word_first)) - 1u;

    uint32_t incl = __popc(word);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(kFull, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += u;
    }
    const uint32_t excl = incl - __popc(word);
    const uint64_t vbase = chunk_base + before;             // rank of the quarter's first set bit

    // staging area of this warp: 1024 elements plus one vector of slack for the alignment shift
    __shared__ __align__(16) U s_stage[kWarps][1024 + kVec];
    U *const       stage = s_stage[threadIdx.x >> 5];
    const uint32_t skew  = static_cast<uint32_t>(vbase % kVec);   // staged index i <-> values[vbase - skew + i]
    const uint32_t total = __shfl_sync(kFull, incl, 31);          // set bits of the quarter

    const uint32_t shift = (lane % kLanesPerWord) * kE;     // which kE-bit group of the word
    uint32_t       one, two;                                 // registers the compiler cannot see through
    asm volatile("mov.u32 %0, 1;\n\tmov.u32 %1, 2;" : "=r"(one), "=r"(two));
    const Extent   yx    = extent_of(y, n * sizeof(U));
    const Extent   vx    = extent_of(values, capacity * sizeof(U));
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        U (&e)[kE] = xe[kLate ? 0 : k];                        // this step's elements
        if constexpr (kLate) {
#pragma unroll
            for (int v = 0; v < kE / kVec; ++v) unpack_vec<U>(xv[k][v], e + v * kVec);
        }
        const int      from = k * kWordsPerStep + lane / kLanesPerWord;
        const uint32_t w    = __shfl_sync(kFull, word, from);
        const uint32_t wex  = __shfl_sync(kFull, excl, from);
        const uint32_t bits = (w >> shift) & ((1u << kE) - 1u);
        uint32_t       off  = skew + wex + __popc(w & ((1u << shift) - 1u));
        if constexpr (sizeof(U) == 2) {
            // 2-byte elements: this loop is bound by the integer pipe, so the running position advances by a
            // predicated multiply-add (FMA pipe) and the staged address is a byte address kept in one register
            uint32_t at = smem_addr(stage) + 2u * off;
#pragma unroll
            for (int j = 0; j < kE; ++j) {
                asm volatile(
                    "{\n\t.reg .pred p;\n\t.reg .b32 t;\n\t"
                    "and.b32 t, %1, %2;\n\tsetp.ne.u32 p, t, 0;\n\t"
                    "@p st.shared.u16 [%0], %3;\n\t"
                    "@p mad.lo.u32 %0, %4, %5, %0;\n\t}"
                    : "+r"(at)
                    : "r"(bits), "r"(1u << j), "h"(e[j]), "r"(one), "r"(two)
                    : "memory");
                if constexpr (WRITE_Y) e[j] = ((bits >> j) & 1u) ? e[j] : U(0);
            }
        } else {
#pragma unroll
            for (int j = 0; j < kE; ++j) {
                const bool set = (bits >> j) & 1u;
                if (set) stage[off] = e[j];
                off += set;
                if constexpr (WRITE_Y) e[j] = set ? e[j] : U(0);
            }
        }
        if constexpr (WRITE_Y) {
            const uint64_t eo = e0 + static_cast<uint64_t>(k) * (32 * kE) + lane * kE;
#pragma unroll
            for (int v = 0; v < kE / kVec; ++v) {
                const uint64_t at = eo + v * kVec;
                const U       *ev = e + v * kVec;
                if (at + kVec <= n) {
                    const uint4 pack = pack_vec<U>(ev);
                    if (yx.holds(y + at, 16)) *reinterpret_cast<uint4 *>(y + at) = pack;
                } else {
#pragma unroll
                    for (int j = 0; j < kVec; ++j)
                        if (at + j < n && yx.holds(y + at + j, sizeof(U))) y[at + j] = ev[j];
                }
            }
        }
    }
    __syncwarp();

    // staged [skew, skew + total) -> values[vbase, vbase + total), clipped to the capacity
    const uint64_t gbase = vbase - skew;                    // a multiple of kVec: staged vector v <-> values + gbase + v * kVec
    const uint32_t end   = skew + total;
    const uint32_t vecs  = (end + kVec - 1) / kVec;
    for (uint32_t v = lane; v < vecs; v += 32) {
        const uint32_t lo = v * kVec, hi = lo + kVec;
        const uint64_t g  = gbase + lo;
        if (lo >= skew && hi <= end && g + kVec <= capacity) {
            if (vx.holds(values + g, 16)) *reinterpret_cast<uint4 *>(values + g) = *reinterpret_cast<const uint4 *>(stage + lo);
        } else {
#pragma unroll
            for (int j = 0; j < kVec; ++j)
                if (lo + j >= skew && lo + j < end && g + j < capacity && vx.holds(values + g + j, sizeof(U))) values[g + j] = stage[lo + j];
        }
    }
}

template <typename U, int kE>
cudaError_t launch_typed(const void *x, const uint32_t *bitmap, const uint64_t *prefix, uint64_t n, void *y,
                         void *values, uint64_t capacity, cudaStream_t stream)
{
    constexpr int  kWarps   = 4;   // staging area of a CTA below 48 KB for 8-byte elements; 2-byte elements 10 % faster than with 8
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    if (y)
        mask_gather_kernel<U, kE, kWarps, true><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
            static_cast<const U *>(x), bitmap, prefix, n, static_cast<U *>(y), static_cast<U *>(values), capacity);
    else
        mask_gather_kernel<U, kE, kWarps, false><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
            static_cast<const U *>(x), bitmap, prefix, n, nullptr, static_cast<U *>(values), capacity);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_mask_gather(const void *x, const uint32_t *bitmap, const uint64_t *prefix, uint64_t n,
                               int elem_size, void *y, void *values, uint64_t capacity, cudaStream_t stream)
{
    if (elem_size == 8) return launch_typed<uint64_t, 2>(x, bitmap, prefix, n, y, values, capacity, stream);
    return elem_size == 4 ? launch_typed<uint32_t, 4>(x, bitmap, prefix, n, y, values, capacity, stream)
                          : launch_typed<uint16_t, 8>(x, bitmap, prefix, n, y, values, capacity, stream);
}

}  // namespace bt
