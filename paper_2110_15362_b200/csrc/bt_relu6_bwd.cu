// ReLU6 backward from the stash: grad_in[i] = (bit i set and the stashed
// activation is below 6) ? grad_out[i] : +0.  Unlike plain ReLU, the bitmap alone
// does not say whether a unit is saturated (its stashed value is 6), so the
// values are consulted: the decompressor's rank arithmetic (chunk prefix entry +
// popcounts, no communication between warps), a gather of the stashed values of
// the set bits, one comparison each, and a select on the gradient, which moves
// in 16-byte vectors.
//
// One warp, one quarter chunk (1024 elements = 32 bitmap words); a lane owns kE
// consecutive elements per step, i.e. kE consecutive bits of one word.  The
// gradient is fetched kBlk steps at a time, ahead of the gather that depends on
// the stash: two steps for 4- and 8-byte elements (holding the whole quarter
// costs registers and with them occupancy: measured 20 to 45 % slower), all four
// for 2-byte elements (measured faster than two).
#include "bt_internal.cuh"
#include "bt_quarter16.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull = 0xFFFFFFFFu;

template <typename U, int DT, int kE, int kBlk, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
relu6_bwd_kernel(const uint32_t *__restrict__ bitmap, const U *__restrict__ values,
                 const uint64_t *__restrict__ values_offset, const uint64_t *__restrict__ prefix, const U *gout,
                 const uint64_t n, U *gin)   // gin may alias gout
{
    // arena form: the packed values start *values_offset bytes into `values`
    if (values_offset) values = reinterpret_cast<const U *>(reinterpret_cast<const unsigned char *>(values) + *values_offset);
    constexpr int kVec          = 16 / sizeof(U);
    constexpr int kLanesPerWord = 32 / kE;
    constexpr int kWordsPerStep = kE;
    constexpr int kSteps        = 32 / kWordsPerStep;
    static_assert(kE % kVec == 0 && 32 % kE == 0 && kE < 32, "a lane takes whole vectors of one word");
    static_assert(kSteps % kBlk == 0, "whole rounds");

    const uint32_t lane        = threadIdx.x & 31u;
    const uint64_t warp_global = static_cast<uint64_t>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    const uint64_t quarters    = (n + 1023) >> 10;
    if (warp_global >= quarters) return;

    const uint64_t chunk       = warp_global >> 2;
    const uint32_t q           = static_cast<uint32_t>(warp_global & 3u);
    const uint64_t words_total = (n + 31) >> 5;
    const uint64_t w0          = chunk * 128 + 4 * lane;
    const uint64_t e0          = warp_global << 10;

    // kBlk steps of the gradient: these loads do not depend on the stash
    U    g[kBlk][kE];
    auto fetch = [&](const int k0) {
#pragma unroll
        for (int k = 0; k < kBlk; ++k) {
            const uint64_t eo = e0 + static_cast<uint64_t>(k0 + k) * (32 * kE) + lane * kE;
#pragma unroll
            for (int v = 0; v < kE / kVec; ++v) {
                const uint64_t at = eo + v * kVec;
                U             *gv = g[k] + v * kVec;
                if (at + kVec <= n) {
                    const uint4 pack = *reinterpret_cast<const uint4 *>(gout + at);
                    if constexpr (kVec == 2) {
                        gv[0] = pack.x | (static_cast<uint64_t>(pack.y) << 32);
                        gv[1] = pack.z | (static_cast<uint64_t>(pack.w) << 32);
                    } else if constexpr (kVec == 4) {
                        gv[0] = pack.x, gv[1] = pack.y, gv[2] = pack.z, gv[3] = pack.w;
                    } else {
                        gv[0] = static_cast<U>(pack.x), gv[1] = static_cast<U>(pack.x >> 16);
                        gv[2] = static_cast<U>(pack.y), gv[3] = static_cast<U>(pack.y >> 16);
                        gv[4] = static_cast<U>(pack.z), gv[5] = static_cast<U>(pack.z >> 16);
                        gv[6] = static_cast<U>(pack.w), gv[7] = static_cast<U>(pack.w >> 16);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < kVec; ++j) gv[j] = at + j < n ? gout[at + j] : U(0);
                }
            }
        }
    };
    fetch(0);

    const uint4 w4 = load_words4(bitmap, w0, words_total);
    const uint64_t chunk_base = prefix[chunk];

    uint32_t before = lane < 8 * q ? __popc(w4.x) + __popc(w4.y) + __popc(w4.z) + __popc(w4.w) : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(kFull, before, o);

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
    const U *const vp   = values + (chunk_base + before);

    const uint32_t shift = (lane % kLanesPerWord) * kE;
    const Extent   ox    = extent_of(gin, n * sizeof(U));
#pragma unroll
    for (int kk = 0; kk < kSteps; ++kk) {
        const int k = kk % kBlk;                              // row of g
        if (kk != 0 && k == 0) fetch(kk);
        const int      from = kk * kWordsPerStep + lane / kLanesPerWord;
        const uint32_t w    = __shfl_sync(kFull, word, from);
        const uint32_t wex  = __shfl_sync(kFull, excl, from);
        const uint32_t bits = (w >> shift) & ((1u << kE) - 1u);
        uint32_t       off  = wex + __popc(w & ((1u << shift) - 1u));
#pragma unroll
        for (int j = 0; j < kE; ++j) {
            const bool set  = (bits >> j) & 1u;
            const U    v    = set ? vp[off] : U(0);                   // a predicated load, as in the decompressor
            const auto a    = Elem<DT>::widen(v);
            const bool pass = set & (a < static_cast<decltype(a)>(6));   // false for a stashed 6 and for a NaN
            off += set;
            g[k][j] = pass ? g[k][j] : U(0);
        }
        const uint64_t eo = e0 + static_cast<uint64_t>(kk) * (32 * kE) + lane * kE;
#pragma unroll
        for (int v = 0; v < kE / kVec; ++v) {
            const uint64_t at = eo + v * kVec;
            const U       *gv = g[k] + v * kVec;
            if (at + kVec <= n) {
                uint4 pack;
                if constexpr (kVec == 2) {
                    pack = make_uint4(static_cast<uint32_t>(gv[0]), static_cast<uint32_t>(gv[0] >> 32),
                                      static_cast<uint32_t>(gv[1]), static_cast<uint32_t>(gv[1] >> 32));
                } else if constexpr (kVec == 4) {
                    pack = make_uint4(gv[0], gv[1], gv[2], gv[3]);
                } else {
                    pack = make_uint4(gv[0] | (uint32_t(gv[1]) << 16), gv[2] | (uint32_t(gv[3]) << 16),
                                      gv[4] | (uint32_t(gv[5]) << 16), gv[6] | (uint32_t(gv[7]) << 16));
                }
                if (ox.holds(gin + at, 16)) *reinterpret_cast<uint4 *>(gin + at) = pack;
            } else {
#pragma unroll
                for (int j = 0; j < kVec; ++j)
                    if (at + j < n && ox.holds(gin + at + j, sizeof(U))) gin[at + j] = gv[j];
            }
        }
    }
}

// Two packed 2-byte values compared with 6 in their own type: 0xFFFF in the half of a value below 6, else 0 (a NaN
// is not below 6).
template <int DT>
__device__ __forceinline__ uint32_t below_six_mask(const uint32_t pair)
{
    uint32_t m;
    if constexpr (DT == BT_F16) asm("set.lt.u32.f16x2 %0, %1, %2;" : "=r"(m) : "r"(pair), "r"(0x46004600u));
    else asm("set.lt.u32.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(pair), "r"(0x40C040C0u));
    return m;
}

// 2-byte elements: the quarter's packed run staged in shared memory and gathered from there (bt_quarter16.cuh)
// instead of one global gather per value.  The quarter's gradient -- eight 8-byte loads per lane that do not
// depend on the stash -- is requested first, so that it arrives while the run is staged.
template <int DT, int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1536 / (kWarps * 32))   // 40 registers, 12 CTAs per SM: 0.199 -> 0.178 ms against 8 CTAs
relu6_bwd16_kernel(const uint32_t *__restrict__ bitmap, const uint16_t *__restrict__ values,
                   const uint64_t *__restrict__ values_offset, const uint64_t *__restrict__ prefix, const uint16_t *gout,
                   const uint64_t n, uint16_t *gin)   // gin may alias gout
{
    const uint32_t lane        = threadIdx.x & 31u;
    const uint64_t warp_global = static_cast<uint64_t>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    if (warp_global >= ((n + 1023) >> 10)) return;
    const uint64_t e0 = warp_global << 10;
    uint2          g[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint64_t at = e0 + static_cast<uint64_t>(k) * 128 + lane * 4;
        if (at + 4 <= n) {
            g[k] = *reinterpret_cast<const uint2 *>(gout + at);
        } else {
            uint32_t h[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) h[j] = at + j < n ? gout[at + j] : 0u;
            g[k] = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
        }
    }
    q16::Quarter qt;
    if (!q16::stage_quarter<kWarps>(bitmap, values, values_offset, prefix, n, blockIdx.x, qt)) return;
    const Extent ox = extent_of(gin, n * sizeof(uint16_t));
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        // The gradient passes where the bit is set and the stashed value is below 6 (false for a stored 6 and for a
        // NaN).  Elements under a clear bit come out of the expansion as a NaN, so one compare of the packed pair in
        // its own type decides both conditions for two elements: a 16-bit mask of ones per element that passes.
        uint32_t    bits;
        const uint2 v = q16::expand_step<0x7FFFu>(qt, k, lane, bits);
        const uint2 r = make_uint2(g[k].x & below_six_mask<DT>(v.x), g[k].y & below_six_mask<DT>(v.y));
        const uint64_t at = e0 + static_cast<uint64_t>(k) * 128 + lane * 4;
        if (qt.whole || at + 4 <= n) {
            if (ox.holds(gin + at, 8)) *reinterpret_cast<uint2 *>(gin + at) = r;
        } else {
            const uint32_t o[2] = {r.x, r.y};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (at + j < n && ox.holds(gin + at + j, 2)) gin[at + j] = static_cast<uint16_t>(o[j >> 1] >> (16 * (j & 1)));
        }
    }
}

template <int DT>
cudaError_t launch_16(const uint32_t *bitmap, const void *values, const uint64_t *values_offset, const uint64_t *prefix,
                      const void *gout, uint64_t n, void *gin, cudaStream_t stream)
{
    constexpr int  kWarps   = 4;
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    relu6_bwd16_kernel<DT, kWarps><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
        bitmap, static_cast<const uint16_t *>(values), values_offset, prefix, static_cast<const uint16_t *>(gout), n,
        static_cast<uint16_t *>(gin));
    return cudaGetLastError();
}

template <typename U, int DT, int kE, int kBlk>
cudaError_t launch_typed(const uint32_t *bitmap, const void *values, const uint64_t *values_offset, const uint64_t *prefix,
                         const void *gout, uint64_t n, void *gin, cudaStream_t stream)
{
    constexpr int  kWarps   = 4;   // four warps per CTA: 1 to 4 % faster than eight
    const uint64_t quarters = (n + 1023) >> 10;
    const uint64_t grid     = (quarters + kWarps - 1) / kWarps;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    relu6_bwd_kernel<U, DT, kE, kBlk, kWarps><<<static_cast<unsigned>(grid), kWarps * 32, 0, stream>>>(
        bitmap, static_cast<const U *>(values), values_offset, prefix, static_cast<const U *>(gout), n, static_cast<U *>(gin));
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_relu6_bwd(const uint32_t *bitmap, const void *values, const uint64_t *values_offset,
                             const uint64_t *prefix, const void *gout, uint64_t n, int dtype, void *gin,
                             cudaStream_t stream)
{
    switch (dtype) {
    case BT_F64: return launch_typed<uint64_t, BT_F64, 2, 2>(bitmap, values, values_offset, prefix, gout, n, gin, stream);
    case BT_F32: return launch_typed<uint32_t, BT_F32, 4, 2>(bitmap, values, values_offset, prefix, gout, n, gin, stream);
    case BT_F16: return launch_16<BT_F16>(bitmap, values, values_offset, prefix, gout, n, gin, stream);
    default: return launch_16<BT_BF16>(bitmap, values, values_offset, prefix, gout, n, gin, stream);
    }
}

}  // namespace bt
