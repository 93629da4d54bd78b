// 2x2 / stride 2 max pooling with winner codes, and its backward pass from the codes.
//
// The tensor is planes x height x width elements, row-major, height and width even, so the two input rows of
// an output row are adjacent in memory and output row R (counted across all planes) reads input rows 2R and
// 2R + 1.  One thread per output: two loads of an element pair (always aligned: every pair starts at an even
// element index), the framework's comparison rule on the exactly widened values -- a later window element
// replaces the maximum when it is greater or when it is a NaN -- one store of the winner and a 2-bit code of its
// position (2*dy + dx).  Sixteen consecutive outputs belong to sixteen consecutive lanes, which merge their
// codes into one word with four shuffles.  The backward pass reads a gradient and a code per output and writes
// the four window positions as two pair stores: the gradient where the code points, +0 elsewhere.
//
// With the codes kept, neither the pooling layer's input nor an index tensor is needed for its backward pass:
// 2 bits per output instead of 8 bytes per output plus the saved input.
#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull    = 0xFFFFFFFFu;
constexpr int      kThreads = 256;

// a pair of adjacent elements as one register-sized load / store
template <typename U>
struct Pair;
template <>
struct Pair<uint16_t> {
    using T = uint32_t;
    __device__ static uint16_t lo(T p) { return static_cast<uint16_t>(p); }
    __device__ static uint16_t hi(T p) { return static_cast<uint16_t>(p >> 16); }
    __device__ static T make(uint16_t a, uint16_t b) { return a | (static_cast<uint32_t>(b) << 16); }
};
template <>
struct Pair<uint32_t> {
    using T = uint2;
    __device__ static uint32_t lo(T p) { return p.x; }
    __device__ static uint32_t hi(T p) { return p.y; }
    __device__ static T make(uint32_t a, uint32_t b) { return make_uint2(a, b); }
};
template <>
struct Pair<uint64_t> {
    using T = ulonglong2;
    __device__ static uint64_t lo(T p) { return p.x; }
    __device__ static uint64_t hi(T p) { return p.y; }
    __device__ static T make(uint64_t a, uint64_t b) { return make_ulonglong2(a, b); }
};

// I: uint32_t while every element index fits 32 bits (one cheap division per thread), else uint64_t
template <typename U, int DT, typename I>
__global__ void __launch_bounds__(kThreads)
maxpool2x2_fwd_kernel(const U *__restrict__ x, const uint64_t outputs, const I wo, const I width, U *__restrict__ y,
                      uint32_t *__restrict__ codes)
{
    using P             = Pair<U>;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t o64  = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    const bool     live = o64 < outputs;
    uint32_t       code = 0;
    if (live) {
        const I        o   = static_cast<I>(o64);
        const I        row = o / wo;                       // output row, counted across the planes
        const I        col = o - row * wo;
        const uint64_t at  = 2ull * row * width + 2ull * col;
        const typename P::T top = *reinterpret_cast<const typename P::T *>(x + at);
        const typename P::T bot = *reinterpret_cast<const typename P::T *>(x + at + width);
        const U e[4] = {P::lo(top), P::hi(top), P::lo(bot), P::hi(bot)};
        U    best  = e[0];
        auto bestv = Elem<DT>::widen(e[0]);
#pragma unroll
        for (uint32_t k = 1; k < 4; ++k) {
            const auto v    = Elem<DT>::widen(e[k]);
            const bool take = greater_or_nan(v, bestv) != 0;
            best            = take ? e[k] : best;
            bestv           = take ? v : bestv;
            code            = take ? k : code;
        }
        if (extent_of(y, outputs * sizeof(U)).holds(y + o64, sizeof(U))) y[o64] = best;
    }
    if (codes) {
        uint32_t word = code << (2u * (lane & 15u));
#pragma unroll
        for (int d = 8; d > 0; d >>= 1) word |= __shfl_xor_sync(kFull, word, d);
        if (live && (lane & 15u) == 0 && extent_of(codes, 4 * ((outputs + 15) >> 4)).holds(codes + (o64 >> 4), 4)) codes[o64 >> 4] = word;
    }
}

template <typename U, typename I>
__global__ void __launch_bounds__(kThreads)
maxpool2x2_bwd_kernel(const uint32_t *__restrict__ codes, const uint32_t *__restrict__ mask, const U *__restrict__ gout,
                      const uint64_t outputs, const I wo, const I width, U *__restrict__ gin)
{
    // mask (may be NULL): bitmap over the outputs; the gradient of an output whose bit is clear counts as +0
    using P            = Pair<U>;
    const uint64_t o64 = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (o64 >= outputs) return;
    const I        o    = static_cast<I>(o64);
    const I        row  = o / wo;
    const I        col  = o - row * wo;
    const uint64_t at   = 2ull * row * width + 2ull * col;
    const uint32_t k    = (codes[o64 >> 4] >> (2u * (static_cast<uint32_t>(o64) & 15u))) & 3u;
    U              g    = gout[o64];
    if (mask != nullptr && ((mask[o64 >> 5] >> (static_cast<uint32_t>(o64) & 31u)) & 1u) == 0) g = U(0);
    const Extent gx = extent_of(gin, 4 * outputs * sizeof(U));
    if (gx.holds(gin + at, 2 * sizeof(U))) *reinterpret_cast<typename P::T *>(gin + at) = P::make(k == 0 ? g : U(0), k == 1 ? g : U(0));
    if (gx.holds(gin + at + width, 2 * sizeof(U)))
        *reinterpret_cast<typename P::T *>(gin + at + width) = P::make(k == 2 ? g : U(0), k == 3 ? g : U(0));
}

// Vector form for 2- and 4-byte elements whose rows hold whole 16-byte vectors of window pairs (width a multiple of
// 8 resp. 4): a thread takes kOut = 4 resp. 2 adjacent outputs, i.e. one 16-byte load per input row, one 8-byte
// store of the winners and 2 * kOut code bits; 16 / kOut consecutive lanes share a code word.
template <typename U>
__device__ __forceinline__ void unpack16(const uint4 v, U (&e)[16 / sizeof(U)])
{
    if constexpr (sizeof(U) == 4) {
        e[0] = v.x, e[1] = v.y, e[2] = v.z, e[3] = v.w;
    } else {
        e[0] = static_cast<U>(v.x), e[1] = static_cast<U>(v.x >> 16), e[2] = static_cast<U>(v.y), e[3] = static_cast<U>(v.y >> 16);
        e[4] = static_cast<U>(v.z), e[5] = static_cast<U>(v.z >> 16), e[6] = static_cast<U>(v.w), e[7] = static_cast<U>(v.w >> 16);
    }
}
template <typename U>
__device__ __forceinline__ uint4 pack16(const U (&e)[16 / sizeof(U)])
{
    if constexpr (sizeof(U) == 4) return make_uint4(e[0], e[1], e[2], e[3]);
    else
        return make_uint4(e[0] | (uint32_t(e[1]) << 16), e[2] | (uint32_t(e[3]) << 16), e[4] | (uint32_t(e[5]) << 16),
                          e[6] | (uint32_t(e[7]) << 16));
}

template <typename U, int DT, typename I>
__global__ void __launch_bounds__(kThreads)
maxpool2x2_fwd_vec_kernel(const U *__restrict__ x, const uint64_t groups, const I groups_per_row, const I width,
                          U *__restrict__ y, uint32_t *__restrict__ codes)
{
    constexpr int      kOut          = 8 / sizeof(U);          // outputs per thread
    constexpr uint32_t kLanesPerWord = 16 / kOut;
    const uint32_t     lane          = threadIdx.x & 31u;
    const uint64_t     g64           = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    const bool         live          = g64 < groups;
    uint32_t           bits          = 0;
    if (live) {
        const I        g   = static_cast<I>(g64);
        const I        row = g / groups_per_row;
        const I        cg  = g - row * groups_per_row;
        const uint64_t at  = 2ull * row * width + 2ull * kOut * cg;
        U              top[2 * kOut], bot[2 * kOut], win[kOut];
        unpack16<U>(*reinterpret_cast<const uint4 *>(x + at), top);
        unpack16<U>(*reinterpret_cast<const uint4 *>(x + at + width), bot);
#pragma unroll
        for (int j = 0; j < kOut; ++j) {
            const U  e[4]  = {top[2 * j], top[2 * j + 1], bot[2 * j], bot[2 * j + 1]};
            U        best  = e[0];
            auto     bestv = Elem<DT>::widen(e[0]);
            uint32_t code  = 0;
#pragma unroll
            for (uint32_t k = 1; k < 4; ++k) {
                const auto v    = Elem<DT>::widen(e[k]);
                const bool take = greater_or_nan(v, bestv) != 0;
                best            = take ? e[k] : best;
                bestv           = take ? v : bestv;
                code            = take ? k : code;
            }
            win[j] = best;
            bits |= code << (2 * j);
        }
        uint2 pack;
        if constexpr (sizeof(U) == 4) pack = make_uint2(win[0], win[1]);
        else pack = make_uint2(win[0] | (uint32_t(win[1]) << 16), win[2] | (uint32_t(win[3]) << 16));
        if (extent_of(y, groups * kOut * sizeof(U)).holds(y + g64 * kOut, 8)) *reinterpret_cast<uint2 *>(y + g64 * kOut) = pack;
    }
    if (codes) {
        uint32_t word = bits << (2u * kOut * (lane % kLanesPerWord));
#pragma unroll
        for (int d = kLanesPerWord / 2; d > 0; d >>= 1) word |= __shfl_xor_sync(kFull, word, d);
        if (live && (lane % kLanesPerWord) == 0 && extent_of(codes, 4 * ((groups * kOut + 15) >> 4)).holds(codes + ((g64 * kOut) >> 4), 4))
            codes[(g64 * kOut) >> 4] = word;
    }
}

template <typename U, typename I>
__global__ void __launch_bounds__(kThreads)
maxpool2x2_bwd_vec_kernel(const uint32_t *__restrict__ codes, const uint32_t *__restrict__ mask, const U *__restrict__ gout,
                          const uint64_t groups, const I groups_per_row, const I width, U *__restrict__ gin)
{
    constexpr int  kOut = 8 / sizeof(U);
    const uint64_t g64  = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (g64 >= groups) return;
    const I        g    = static_cast<I>(g64);
    const I        row  = g / groups_per_row;
    const I        cg   = g - row * groups_per_row;
    const uint64_t at   = 2ull * row * width + 2ull * kOut * cg;
    const uint64_t o0   = g64 * kOut;
    const uint32_t bits = codes[o0 >> 4] >> (2u * (static_cast<uint32_t>(o0) & 15u));
    // the kOut mask bits of this thread's outputs sit in one word (kOut divides 32)
    const uint32_t live = mask != nullptr ? mask[o0 >> 5] >> (static_cast<uint32_t>(o0) & 31u) : 0xFFFFFFFFu;
    const uint2    gv   = *reinterpret_cast<const uint2 *>(gout + o0);
    U              gr[kOut], top[2 * kOut], bot[2 * kOut];
    if constexpr (sizeof(U) == 4) {
        gr[0] = gv.x, gr[1] = gv.y;
    } else {
        gr[0] = static_cast<U>(gv.x), gr[1] = static_cast<U>(gv.x >> 16), gr[2] = static_cast<U>(gv.y), gr[3] = static_cast<U>(gv.y >> 16);
    }
#pragma unroll
    for (int j = 0; j < kOut; ++j) {
        const uint32_t k = (bits >> (2 * j)) & 3u;
        gr[j]            = (live >> j) & 1u ? gr[j] : U(0);
        top[2 * j]       = k == 0 ? gr[j] : U(0);
        top[2 * j + 1]   = k == 1 ? gr[j] : U(0);
        bot[2 * j]       = k == 2 ? gr[j] : U(0);
        bot[2 * j + 1]   = k == 3 ? gr[j] : U(0);
    }
    const Extent gx = extent_of(gin, 4 * groups * kOut * sizeof(U));
    if (gx.holds(gin + at, 16)) *reinterpret_cast<uint4 *>(gin + at) = pack16<U>(top);
    if (gx.holds(gin + at + width, 16)) *reinterpret_cast<uint4 *>(gin + at + width) = pack16<U>(bot);
}

template <typename U, int DT>
cudaError_t fwd_typed(const void *x, uint64_t outputs, uint64_t wo, uint64_t width, uint64_t elements, void *y, uint32_t *codes,
                      cudaStream_t s)
{
    if constexpr (sizeof(U) <= 4) {
        constexpr uint64_t kOut = 8 / sizeof(U);
        if (width % (2 * kOut) == 0) {
            const uint64_t groups = outputs / kOut, per_row = wo / kOut, vgrid = (groups + kThreads - 1) / kThreads;
            if (vgrid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
            if (elements <= 0xFFFFFFFFull)
                maxpool2x2_fwd_vec_kernel<U, DT, uint32_t><<<static_cast<unsigned>(vgrid), kThreads, 0, s>>>(
                    static_cast<const U *>(x), groups, static_cast<uint32_t>(per_row), static_cast<uint32_t>(width),
                    static_cast<U *>(y), codes);
            else
                maxpool2x2_fwd_vec_kernel<U, DT, uint64_t><<<static_cast<unsigned>(vgrid), kThreads, 0, s>>>(
                    static_cast<const U *>(x), groups, per_row, width, static_cast<U *>(y), codes);
            return cudaGetLastError();
        }
    }
    const uint64_t grid = (outputs + kThreads - 1) / kThreads;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    if (elements <= 0xFFFFFFFFull)
        maxpool2x2_fwd_kernel<U, DT, uint32_t><<<static_cast<unsigned>(grid), kThreads, 0, s>>>(
            static_cast<const U *>(x), outputs, static_cast<uint32_t>(wo), static_cast<uint32_t>(width), static_cast<U *>(y), codes);
    else
        maxpool2x2_fwd_kernel<U, DT, uint64_t><<<static_cast<unsigned>(grid), kThreads, 0, s>>>(
            static_cast<const U *>(x), outputs, wo, width, static_cast<U *>(y), codes);
    return cudaGetLastError();
}

template <typename U>
cudaError_t bwd_typed(const uint32_t *codes, const uint32_t *mask, const void *gout, uint64_t outputs, uint64_t wo,
                      uint64_t width, uint64_t elements, void *gin, cudaStream_t s)
{
    if constexpr (sizeof(U) <= 4) {
        constexpr uint64_t kOut = 8 / sizeof(U);
        if (width % (2 * kOut) == 0) {
            const uint64_t groups = outputs / kOut, per_row = wo / kOut, vgrid = (groups + kThreads - 1) / kThreads;
            if (vgrid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
            if (elements <= 0xFFFFFFFFull)
                maxpool2x2_bwd_vec_kernel<U, uint32_t><<<static_cast<unsigned>(vgrid), kThreads, 0, s>>>(
                    codes, mask, static_cast<const U *>(gout), groups, static_cast<uint32_t>(per_row),
                    static_cast<uint32_t>(width), static_cast<U *>(gin));
            else
                maxpool2x2_bwd_vec_kernel<U, uint64_t><<<static_cast<unsigned>(vgrid), kThreads, 0, s>>>(
                    codes, mask, static_cast<const U *>(gout), groups, per_row, width, static_cast<U *>(gin));
            return cudaGetLastError();
        }
    }
    const uint64_t grid = (outputs + kThreads - 1) / kThreads;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    if (elements <= 0xFFFFFFFFull)
        maxpool2x2_bwd_kernel<U, uint32_t><<<static_cast<unsigned>(grid), kThreads, 0, s>>>(
            codes, mask, static_cast<const U *>(gout), outputs, static_cast<uint32_t>(wo), static_cast<uint32_t>(width),
            static_cast<U *>(gin));
    else
        maxpool2x2_bwd_kernel<U, uint64_t><<<static_cast<unsigned>(grid), kThreads, 0, s>>>(
            codes, mask, static_cast<const U *>(gout), outputs, wo, width, static_cast<U *>(gin));
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_maxpool2x2_fwd(const void *x, uint64_t planes, uint64_t height, uint64_t width, int dtype, void *y,
                                  uint32_t *codes, cudaStream_t s)
{
    const uint64_t wo = width / 2, outputs = planes * (height / 2) * wo, elements = planes * height * width;
    switch (dtype) {
    case BT_F64: return fwd_typed<uint64_t, BT_F64>(x, outputs, wo, width, elements, y, codes, s);
    case BT_F32: return fwd_typed<uint32_t, BT_F32>(x, outputs, wo, width, elements, y, codes, s);
    case BT_F16: return fwd_typed<uint16_t, BT_F16>(x, outputs, wo, width, elements, y, codes, s);
    default: return fwd_typed<uint16_t, BT_BF16>(x, outputs, wo, width, elements, y, codes, s);
    }
}

cudaError_t launch_maxpool2x2_bwd(const uint32_t *codes, const uint32_t *mask, const void *gout, uint64_t planes,
                                  uint64_t height, uint64_t width, int elem_size, void *gin, cudaStream_t s)
{
    const uint64_t wo = width / 2, outputs = planes * (height / 2) * wo, elements = planes * height * width;
    if (elem_size == 8) return bwd_typed<uint64_t>(codes, mask, gout, outputs, wo, width, elements, gin, s);
    return elem_size == 4 ? bwd_typed<uint32_t>(codes, mask, gout, outputs, wo, width, elements, gin, s)
                          : bwd_typed<uint16_t>(codes, mask, gout, outputs, wo, width, elements, gin, s);
}

}  // namespace bt
