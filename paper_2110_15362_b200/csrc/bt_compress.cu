// Algorithm 1 (dense -> bitmap) and its fused forms (ReLU, activation pruning, ReLU6) as ONE pass
// over one tensor or a batch of tensors: a single-pass stream compaction with decoupled look-back.
//
// One CTA, one tile of 32 KB (4096 8-byte, 8192 4-byte or 16384 2-byte elements: whole chunks of the
// prefix array), taken in the order of the block index.  The CTA's eight warps each own a segment of
// the tile:
//
//   - every lane loads its 16-byte vectors of the segment straight into registers (all of them
//     before anything else: these loads are the kernel's bytes in flight) and keeps them there;
//   - a kVec-bit mask per vector of the elements whose pattern is not zero (after the fused forward
//     form, if any).  The masks ARE the bitmap: lanes that share a bitmap byte combine their bits
//     with one or two shuffles, the bytes pass through a small staging area, and lane k stores
//     word k of the segment -- one coalesced store per warp;
//   - the counts of several steps ride in the fields of one register through ONE warp scan (five
//     shuffles); the warps' counts meet in shared memory;
//   - every lane stores its kept elements at its exclusive offset into the tile's staging area in
//     shared memory, with predicated instructions;
//   - meanwhile warp 0 publishes the tile's count and looks back over the tiles before it for its
//     exclusive prefix (below); when it has it, all warps copy the staged run to
//     values[prefix ...] in 16-byte vectors.
//
// Prefix.  Every tile publishes its count in the workspace as soon as it is counted.  The last tile of
// every group of 64 tiles adds up the group's counts and publishes the group's count, the last tile of
// every group of 4096 tiles that of its group (from the 64 group counts below it), and so on.  With
// t = a + 64 b + 4096 c + ... the exclusive prefix of tile t is the sum of a tile counts, b counts of
// groups of 64, c counts of groups of 4096 ...: warp 0 reads them all at once, at most 63 per level, two
// per lane.  No tile waits for another tile's PREFIX, so there is no chain of dependent round trips
// through L2 along the tensor (a look-back over prefixes advances one window of tiles per round trip,
// which at 8 TB/s is too slow for 32 KB tiles): a tile waits only for counts of tiles with a smaller
// block index, which started no later than itself, and by the time it asks nearly all of them are
// out.  The prefix restarts at every tensor of a batch.
//
// Workspace.  It arrives with unspecified contents and is not cleared: a descriptor carries the
// launch's 64-bit tag, half in each of its two words, and a reader takes only descriptors with its
// own launch's tag.
#include <atomic>
#include <chrono>
#include <cstdlib>
#include <type_traits>

#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull     = 0xFFFFFFFFu;
constexpr int      kHdrSeq   = 0;                   // header words (64-bit): launch sequence number,
constexpr int      kHdrAbort = 1;                   //   abort word (== the launch's tag once a wait ran out),
constexpr int      kHdrDone  = 8;                   //   one word per tensor of the launch (== the tag once all its tiles have published)

template <int kJobs>
struct CompressParams {
    CompressCommon c;
    CompressJob    job[kJobs];
};

__device__ __forceinline__ uint64_t now_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

__device__ __forceinline__ void red_add_u64(uint64_t *p, uint64_t v)
{
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// A bijective mixer of 64-bit words (the finaliser of splitmix64).
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

// 16 bytes from global memory that are read once: no line in L1
__device__ __forceinline__ uint4 ldg_vec(const void *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// register type that holds one element: 64 bits for 8-byte elements, 32 bits otherwise
template <typename U>
using Reg = std::conditional_t<sizeof(U) == 8, uint64_t, uint32_t>;

// shared-memory accesses by 32-bit shared address, kept in program order among themselves
__device__ __forceinline__ uint4 lds_vec(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u8(uint32_t addr, uint32_t v) { asm volatile("st.shared.u8 [%0], %1;" ::"r"(addr), "r"(v)); }

// How a warp walks a segment: kVec elements per lane and step (one 16-byte vector), the counts of kPack
// consecutive steps in kFieldBits-wide fields of one register (an inclusive warp sum of a field is at most
// 32 * kVec: 256 needs 9 bits, 128 and 64 fit 8), kLanesPerByte lanes behind one byte of the bitmap.
template <typename U>
struct Vec {
    static constexpr int kVec          = 16 / sizeof(U);
    static constexpr int kFieldBits    = sizeof(U) == 2 ? 16 : 8;
    static constexpr int kPack         = 32 / kFieldBits;
    static constexpr int kLanesPerByte = 8 / kVec;
};

template <typename U>
__device__ __forceinline__ void unpack(const uint4 &q, Reg<U> (&e)[Vec<U>::kVec])
{
    if constexpr (sizeof(U) == 8) {
        e[0] = static_cast<uint64_t>(q.x) | (static_cast<uint64_t>(q.y) << 32);
        e[1] = static_cast<uint64_t>(q.z) | (static_cast<uint64_t>(q.w) << 32);
    } else if constexpr (sizeof(U) == 4) {
        e[0] = q.x, e[1] = q.y, e[2] = q.z, e[3] = q.w;
    } else {
        e[0] = q.x & 0xFFFFu, e[1] = q.x >> 16, e[2] = q.y & 0xFFFFu, e[3] = q.y >> 16;
        e[4] = q.z & 0xFFFFu, e[5] = q.z >> 16, e[6] = q.w & 0xFFFFu, e[7] = q.w >> 16;
    }
}

template <typename U>
__device__ __forceinline__ uint4 repack(const Reg<U> (&e)[Vec<U>::kVec])
{
    if constexpr (sizeof(U) == 8) {
        return make_uint4(static_cast<uint32_t>(e[0]), static_cast<uint32_t>(e[0] >> 32), static_cast<uint32_t>(e[1]),
                          static_cast<uint32_t>(e[1] >> 32));
    } else if constexpr (sizeof(U) == 4) {
        return make_uint4(e[0], e[1], e[2], e[3]);
    } else {
        return make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
    }
}

// m |= bit where the 32-bit word / its low half / its high half / the 64-bit pair is not zero: a compare and a
// predicated OR (written out because the compiler's own form, compare - select - OR, is one instruction longer,
// and these run once per element)
__device__ __forceinline__ void or_if_nz32(uint32_t &m, uint32_t x, uint32_t bit)
{
    asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p or.b32 %0, %0, %2;\n\t}" : "+r"(m) : "r"(x), "r"(bit));
}
__device__ __forceinline__ void or_if_nz_lo16(uint32_t &m, uint32_t x, uint32_t bit)
{
    asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %1, 0xFFFF;\n\tsetp.ne.u32 p, t, 0;\n\t@p or.b32 %0, %0, %2;\n\t}" : "+r"(m) : "r"(x), "r"(bit));
}
__device__ __forceinline__ void or_if_nz_hi16(uint32_t &m, uint32_t x, uint32_t bit)
{
    asm("{\n\t.reg .pred p;\n\tsetp.gt.u32 p, %1, 0xFFFF;\n\t@p or.b32 %0, %0, %2;\n\t}" : "+r"(m) : "r"(x), "r"(bit));
}
__device__ __forceinline__ void or_if_nz64(uint32_t &m, uint32_t lo, uint32_t hi, uint32_t bit)
{
    asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tor.b32 t, %1, %2;\n\tsetp.ne.u32 p, t, 0;\n\t@p or.b32 %0, %0, %3;\n\t}" : "+r"(m) : "r"(lo), "r"(hi), "r"(bit));
}

// the mask of a lane's vector: bit k set where its k-th element is not zero
template <typename U>
__device__ __forceinline__ uint32_t vec_mask(const uint4 &q)
{
    uint32_t m = 0;
    if constexpr (sizeof(U) == 8) {
        or_if_nz64(m, q.x, q.y, 1u), or_if_nz64(m, q.z, q.w, 2u);
    } else if constexpr (sizeof(U) == 4) {
        or_if_nz32(m, q.x, 1u), or_if_nz32(m, q.y, 2u), or_if_nz32(m, q.z, 4u), or_if_nz32(m, q.w, 8u);
    } else {
        or_if_nz_lo16(m, q.x, 1u), or_if_nz_hi16(m, q.x, 2u), or_if_nz_lo16(m, q.y, 4u), or_if_nz_hi16(m, q.y, 8u);
        or_if_nz_lo16(m, q.z, 16u), or_if_nz_hi16(m, q.z, 32u), or_if_nz_lo16(m, q.w, 64u), or_if_nz_hi16(m, q.w, 128u);
    }
    return m;
}

// if (cond) { store the element at addr; addr += its size; } as predicated instructions (a branch per element
// costs more than the element's other work); with kWrap, addr then wraps from `end` back by `ring` bytes
template <bool kWrap>
__device__ __forceinline__ void wrap_addr(uint32_t &addr, const uint32_t end, const uint32_t ring)
{
    if constexpr (kWrap) addr = addr >= end ? addr - ring : addr;
}
template <bool kWrap>
__device__ __forceinline__ void sts32_if(uint32_t &addr, uint32_t x, uint32_t cond, const uint32_t end, const uint32_t ring)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.u32 [%0], %1;\n\t@p add.u32 %0, %0, 4;\n\t}" : "+r"(addr) : "r"(x), "r"(cond));
    wrap_addr<kWrap>(addr, end, ring);
}
template <bool kWrap>
__device__ __forceinline__ void sts64_if(uint32_t &addr, uint32_t lo, uint32_t hi, uint32_t cond, const uint32_t end, const uint32_t ring)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %3, 0;\n\t@p st.shared.v2.u32 [%0], {%1, %2};\n\t@p add.u32 %0, %0, 8;\n\t}" : "+r"(addr) : "r"(lo), "r"(hi), "r"(cond));
    wrap_addr<kWrap>(addr, end, ring);
}
// the two 16-bit elements of a word, each under its own condition
template <bool kWrap>
__device__ __forceinline__ void sts16x2_if(uint32_t &addr, uint32_t x, uint32_t cond_lo, uint32_t cond_hi, const uint32_t end, const uint32_t ring)
{
    if constexpr (!kWrap) {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\t"
            "setp.ne.u32 p, %2, 0;\n\t@p st.shared.u16 [%0], l;\n\t@p add.u32 %0, %0, 2;\n\t"
            "setp.ne.u32 q, %3, 0;\n\t@q st.shared.u16 [%0], h;\n\t@q add.u32 %0, %0, 2;\n\t}"
            : "+r"(addr)
            : "r"(x), "r"(cond_lo), "r"(cond_hi));
    } else {
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.u16 [%0], l;\n\t@p add.u32 %0, %0, 2;\n\t}" : "+r"(addr) : "r"(x), "r"(cond_lo));
        wrap_addr<true>(addr, end, ring);
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.u16 [%0], h;\n\t@p add.u32 %0, %0, 2;\n\t}" : "+r"(addr) : "r"(x), "r"(cond_hi));
        wrap_addr<true>(addr, end, ring);
    }
}

// ---------------------------------------------------------------------------------------------
// The compaction of one segment of kSeg elements by one warp, in four steps that the kernel interleaves with
// its hand-offs.  A lane takes one 16-byte vector per step (element (s * 32 + lane) * kVec + k of the segment
// is its k-th of step s) and keeps it packed in four registers.
template <typename U, int kSeg>
struct Seg {
    using V                              = Vec<U>;
    static constexpr int      kVec       = V::kVec;
    static constexpr int      kPack      = V::kPack;
    static constexpr int      kFB        = V::kFieldBits;
    static constexpr int      kLPB       = V::kLanesPerByte;
    static constexpr int      kSteps     = kSeg / (32 * kVec);
    static constexpr int      kBatches   = kSteps / kPack;
    static constexpr int      kWords     = kSeg / 32;                 // bitmap words of the segment
    static constexpr int      kWordsPerLane = (kWords + 31) / 32;
    static constexpr uint32_t kES        = sizeof(U);
    static constexpr uint32_t kFieldMask = (1u << kFB) - 1u;
    static_assert(kSteps % kPack == 0 && kSteps >= kPack && kWords <= 64, "whole batches of steps; at most two bitmap words per lane");
    static_assert(kLPB == 1 || kPack == 4, "the byte assembly packs four steps");
};

__device__ __forceinline__ void sts_vec(uint32_t addr, const uint4 &v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
}

// (1) first pass over the segment (shared-window address seg_addr): the fused forward form applied in place (and
// written to the dense output), one mask per step (bit k: the lane's k-th element of the step is kept, i.e. its
// pattern is not zero).  Only the masks stay in registers.  `y` points at the segment's first element of the
// dense output, `valid` is how many of the segment's kSeg elements exist (the others are zeros in shared memory).
template <typename U, int FUSED, bool WRITE_Y, int kSeg>
__device__ __forceinline__ void segment_masks(const uint32_t seg_addr, const uint32_t valid, const uint32_t lane, uint32_t (&m)[Seg<U, kSeg>::kSteps],
                                              U *y, const float tau)
{
    using S = Seg<U, kSeg>;
    uint4 q[S::kSteps];
#pragma unroll
    for (int s = 0; s < S::kSteps; ++s) q[s] = lds_vec(seg_addr + (s * 32 + lane) * 16u);
#pragma unroll
    for (int s = 0; s < S::kSteps; ++s) {
        if constexpr (FUSED >= 0) {
            Reg<U> e[S::kVec];
            unpack<U>(q[s], e);
#pragma unroll
            for (int k = 0; k < S::kVec; ++k) e[k] = fused_forward<FUSED>(e[k], tau);
            q[s] = repack<U>(e);
            sts_vec(seg_addr + (s * 32 + lane) * 16u, q[s]);
            if constexpr (WRITE_Y) {
                const uint32_t at = (s * 32 + lane) * S::kVec;                // first element of the vector in the segment
                if (at + S::kVec <= valid) {
                    *reinterpret_cast<uint4 *>(y + at) = q[s];
                } else {
#pragma unroll
                    for (int k = 0; k < S::kVec; ++k)
                        if (at + k < valid) y[at + k] = static_cast<U>(e[k]);
                }
            }
        }
        m[s] = vec_mask<U>(q[s]);
    }
}

// (2) the masks are the bitmap: byte i of the segment's bitmap covers elements 8i .. 8i + 7.  The lanes behind a
// byte combine their bits, the bytes go through a staging area (kSeg / 8 bytes of shared memory at bm_addr), and
// lane k returns with bitmap words k * kWordsPerLane ... of the segment.
template <typename U, int kSeg>
__device__ __forceinline__ void segment_bitmap(const uint32_t (&m)[Seg<U, kSeg>::kSteps], const uint32_t bm_addr, const uint32_t lane,
                                               uint32_t (&word)[Seg<U, kSeg>::kWordsPerLane])
{
    using S = Seg<U, kSeg>;
    __syncwarp();                                   // the words of the segment before this one have been read
#pragma unroll
    for (int b = 0; b < S::kSteps; b += S::kPack) {
        if constexpr (S::kLPB == 1) {
#pragma unroll
            for (int p = 0; p < S::kPack; ++p) sts_u8(bm_addr + (b + p) * 32u + lane, m[b + p]);
        } else {
            // four steps' masks at a byte's distance, shifted to this lane's place in its byte; the lanes behind
            // one byte then hold four finished bytes (one per step) and share the four stores
            uint32_t four = m[b] | (m[b + 1] << 8) | (m[b + 2] << 16) | (m[b + 3] << 24);
            four <<= S::kVec * (lane & (S::kLPB - 1));
#pragma unroll
            for (int o = 1; o < S::kLPB; o <<= 1) four |= __shfl_xor_sync(kFull, four, o);
            if constexpr (S::kLPB == 2) {
                const uint32_t half = (lane & 1u) ? (four >> 16) : four;                 // even lane: steps b, b + 1
                const uint32_t at   = bm_addr + (b + 2u * (lane & 1u)) * 16u + (lane >> 1);
                sts_u8(at, half & 0xFFu);
                sts_u8(at + 16u, (half >> 8) & 0xFFu);
            } else {
                static_assert(S::kLPB == 4, "two or four lanes behind a byte");
                sts_u8(bm_addr + (b + (lane & 3u)) * 8u + (lane >> 2), (four >> (8u * (lane & 3u))) & 0xFFu);
            }
        }
    }
    __syncwarp();
    if constexpr (S::kWordsPerLane == 1) {
        word[0] = 0;
        if (lane < static_cast<uint32_t>(S::kWords)) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(word[0]) : "r"(bm_addr + 4u * lane) : "memory");
    } else {
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(word[0]), "=r"(word[1]) : "r"(bm_addr + 8u * lane) : "memory");
    }
}

// (3a) the lane's own counts, the counts of a batch's steps in the fields of one register; returns the number of
// kept elements of the whole segment (the same in every lane)
template <typename U, int kSeg>
__device__ __forceinline__ uint32_t segment_count(const uint32_t (&m)[Seg<U, kSeg>::kSteps], uint32_t (&packed)[Seg<U, kSeg>::kBatches])
{
    using S = Seg<U, kSeg>;
    uint32_t mine = 0;
#pragma unroll
    for (int b = 0; b < S::kBatches; ++b) {
        packed[b] = 0;
#pragma unroll
        for (int p = 0; p < S::kPack; ++p) {
            const uint32_t c = static_cast<uint32_t>(__popc(m[b * S::kPack + p]));
            packed[b] |= c << (p * S::kFB);
            mine += c;
        }
    }
    return __reduce_add_sync(kFull, mine);
}

// (3b) one warp scan per batch of steps (the counts of a batch's steps ride in the fields of one register), the
// batches' scans side by side.  Leaves the inclusive sums in inc[].
template <typename U, int kSeg>
__device__ __forceinline__ void segment_scan(const uint32_t (&packed)[Seg<U, kSeg>::kBatches], uint32_t (&inc)[Seg<U, kSeg>::kBatches], const uint32_t lane)
{
    using S = Seg<U, kSeg>;
#pragma unroll
    for (int b = 0; b < S::kBatches; ++b) inc[b] = packed[b];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t u[S::kBatches];
#pragma unroll
        for (int b = 0; b < S::kBatches; ++b) u[b] = __shfl_up_sync(kFull, inc[b], o);
#pragma unroll
        for (int b = 0; b < S::kBatches; ++b)
            if (lane >= static_cast<uint32_t>(o)) inc[b] += u[b];
    }
}

// (4) second pass: the segment is packed in place.  Every lane reads its vectors again and stores its kept
// elements at its exclusive offset from the segment's start, with predicated instructions.  The loads of a batch
// of steps are issued before the stores of the batch before it: a store of a batch lands below the batch's end
// and a later batch reads at or above it, so they never meet.
template <typename U, int kSeg>
__device__ __forceinline__ void segment_pack(const uint32_t seg_addr, const uint32_t lane, const uint32_t (&m)[Seg<U, kSeg>::kSteps],
                                             const uint32_t (&inc)[Seg<U, kSeg>::kBatches], const uint32_t (&packed)[Seg<U, kSeg>::kBatches])
{
    using S        = Seg<U, kSeg>;
    uint32_t out = seg_addr;                         // address of the step's first packed slot (warp-uniform)
    uint4    q[S::kPack], qn[S::kPack];
#pragma unroll
    for (int p = 0; p < S::kPack; ++p) q[p] = lds_vec(seg_addr + (p * 32 + lane) * 16u);
#pragma unroll
    for (int b = 0; b < S::kBatches; ++b) {
        if (b + 1 < S::kBatches) {
#pragma unroll
            for (int p = 0; p < S::kPack; ++p) qn[p] = lds_vec(seg_addr + (((b + 1) * S::kPack + p) * 32 + lane) * 16u);
        }
        const uint32_t tot = __shfl_sync(kFull, inc[b], 31);
        const uint32_t exc = inc[b] - packed[b];
#pragma unroll
        for (int p = 0; p < S::kPack; ++p) {
            const uint4    &v  = q[p];
            const uint32_t  mm = m[b * S::kPack + p];
            uint32_t        at = out + S::kES * ((exc >> (p * S::kFB)) & S::kFieldMask);
            if constexpr (sizeof(U) == 8) {
                sts64_if<false>(at, v.x, v.y, mm & 1u, 0, 0), sts64_if<false>(at, v.z, v.w, mm & 2u, 0, 0);
            } else if constexpr (sizeof(U) == 4) {
                sts32_if<false>(at, v.x, mm & 1u, 0, 0), sts32_if<false>(at, v.y, mm & 2u, 0, 0);
                sts32_if<false>(at, v.z, mm & 4u, 0, 0), sts32_if<false>(at, v.w, mm & 8u, 0, 0);
            } else {
                sts16x2_if<false>(at, v.x, mm & 1u, mm & 2u, 0, 0), sts16x2_if<false>(at, v.y, mm & 4u, mm & 8u, 0, 0);
                sts16x2_if<false>(at, v.z, mm & 16u, mm & 32u, 0, 0), sts16x2_if<false>(at, v.w, mm & 64u, mm & 128u, 0, 0);
            }
            out += S::kES * ((tot >> (p * S::kFB)) & S::kFieldMask);
        }
#pragma unroll
        for (int p = 0; p < S::kPack; ++p) q[p] = qn[p];
    }
}

// Down-cast on stash: a binary32 pattern narrowed to binary16 (CAST 1) or bfloat16 (CAST 2), round to nearest
// even by the hardware conversion, every NaN to the one quiet NaN 0x7FFF.  CAST 0 passes the element through.
template <int CAST, typename U>
__device__ __forceinline__ auto narrowed(const U v)
{
    if constexpr (CAST == 0) {
        return v;
    } else {
        static_assert(sizeof(U) == 4, "the narrowing forms take binary32 tensors");
        const float f = __uint_as_float(v);
        uint16_t    h;
        if constexpr (CAST == 1) asm("cvt.rn.f16.f32 %0, %1;" : "=h"(h) : "f"(f));
        else asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(f));
        return (v & 0x7FFFFFFFu) > 0x7F800000u ? static_cast<uint16_t>(0x7FFFu) : h;
    }
}
template <int CAST, typename U>
using Stored = std::conditional_t<CAST == 0, U, uint16_t>;

// The copier warps' share of a run of `cnt` packed values at src[0..cnt), element by element: warp `copier`, lane
// `lane` takes elements copier * 32 + lane + 32 * kCopiers * i; each instruction moves 32 consecutive elements.
template <typename U, int CAST, int kCopiers, bool kGuard>
__device__ __forceinline__ void copy_out_elems(const U *__restrict__ src, const uint32_t first, const uint32_t cnt,
                                               Stored<CAST, U> *__restrict__ out, const uint64_t room)
{
    constexpr uint32_t kStride = 32u * kCopiers;
    uint32_t           j       = first;
    for (; j + 3 * kStride < cnt; j += 4 * kStride) {
        const auto v0 = narrowed<CAST>(src[j]), v1 = narrowed<CAST>(src[j + kStride]), v2 = narrowed<CAST>(src[j + 2 * kStride]),
                   v3 = narrowed<CAST>(src[j + 3 * kStride]);
        if (!kGuard || j < room) out[j] = v0;
        if (!kGuard || j + kStride < room) out[j + kStride] = v1;
        if (!kGuard || j + 2 * kStride < room) out[j + 2 * kStride] = v2;
        if (!kGuard || j + 3 * kStride < room) out[j + 3 * kStride] = v3;
    }
    for (; j < cnt; j += kStride) {
        const auto v = narrowed<CAST>(src[j]);
        if (!kGuard || j < room) out[j] = v;
    }
}

// Words kWS .. kWS + 3 of the eight words {a, b}, shifted right by `bits` (0 or 16) into the next word: the 16-byte
// vector that starts kWS words and bits / 8 bytes into a.
template <int kWS>
__device__ __forceinline__ uint4 window(const uint4 &a, const uint4 &b, const uint32_t bits)
{
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    return make_uint4(__funnelshift_r(w[kWS], w[kWS + 1], bits), __funnelshift_r(w[kWS + 1], w[kWS + 2], bits),
                      __funnelshift_r(w[kWS + 2], w[kWS + 3], bits), __funnelshift_r(w[kWS + 3], w[(kWS + 4) & 7], bits));
}

// The same share in 16-byte vectors: `out` is 16-byte aligned, the run starts `shift` bytes (a multiple of the
// element size, < 16) into the 16-byte shared vector at src_vec.  A lane reads the two shared vectors its output
// vector straddles and stores their window: 32 lanes move 512 bytes per instruction.  nvec whole vectors.
template <int kCopiers, int kWS>
__device__ __forceinline__ void copy_out_vecs_ws(const uint4 *__restrict__ src_vec, const uint32_t bits, const uint32_t first, const uint32_t nvec,
                                                 uint4 *__restrict__ out)
{
    constexpr uint32_t kStride = 32u * kCopiers;
    uint32_t           i       = first;
    for (; i + kStride < nvec; i += 2 * kStride) {
        const uint4 a0 = src_vec[i], b0 = src_vec[i + 1], a1 = src_vec[i + kStride], b1 = src_vec[i + kStride + 1];
        out[i]           = window<kWS>(a0, b0, bits);
        out[i + kStride] = window<kWS>(a1, b1, bits);
    }
    if (i < nvec) {
        const uint4 a0 = src_vec[i], b0 = src_vec[i + 1];
        out[i]         = window<kWS>(a0, b0, bits);
    }
}
template <int kCopiers>
__device__ __forceinline__ void copy_out_vecs(const uint4 *__restrict__ src_vec, const uint32_t shift, const uint32_t first, const uint32_t nvec,
                                              uint4 *__restrict__ out)
{
    constexpr uint32_t kStride = 32u * kCopiers;
    if (shift == 0) {
        for (uint32_t i = first; i < nvec; i += kStride) out[i] = src_vec[i];
        return;
    }
    const uint32_t bits = (shift & 2u) * 8u;
    switch (shift >> 2) {
    case 0: copy_out_vecs_ws<kCopiers, 0>(src_vec, bits, first, nvec, out); break;
    case 1: copy_out_vecs_ws<kCopiers, 1>(src_vec, bits, first, nvec, out); break;
    case 2: copy_out_vecs_ws<kCopiers, 2>(src_vec, bits, first, nvec, out); break;
    default: copy_out_vecs_ws<kCopiers, 3>(src_vec, bits, first, nvec, out); break;
    }
}

// One contiguous piece of a tile's run, `cnt` packed values at src (shared memory), to out[0..cnt) (global memory):
// in 16-byte vectors where nothing stands in the way (values of the tensor's own type, room for all of them), the
// few elements before the first and after the last whole output vector one by one.
template <typename U, int CAST, int kCopiers, bool kGuard>
__device__ __forceinline__ void copy_out_piece(const U *src, const uint32_t cnt, Stored<CAST, U> *out, const uint64_t room,
                                               const uint32_t copier, const uint32_t lane)
{
    const uint32_t mine = copier * 32u + lane;
    if constexpr (CAST != 0 || kGuard) {
        copy_out_elems<U, CAST, kCopiers, kGuard>(src, mine, cnt, out, room);
    } else {
        constexpr uint32_t kVec = 16 / sizeof(U);
        const uint32_t     lead = static_cast<uint32_t>((16u - (reinterpret_cast<uintptr_t>(out) & 15u)) & 15u) / sizeof(U);   // elements before the first aligned output vector
        if (cnt < lead + 2 * kVec) {
            copy_out_elems<U, 0, kCopiers, false>(src, mine, cnt, out, 0);
            return;
        }
        const uint32_t nvec = (cnt - lead) / kVec;
        const uint32_t done = lead + nvec * kVec;
        if (mine < lead) out[mine] = src[mine];
        // the tail goes to the last copier warp, the head to the first
        if (copier == kCopiers - 1 && done + lane < cnt) out[done + lane] = src[done + lane];
        const uintptr_t s0 = reinterpret_cast<uintptr_t>(src + lead);
        copy_out_vecs<kCopiers>(reinterpret_cast<const uint4 *>(s0 & ~static_cast<uintptr_t>(15)), static_cast<uint32_t>(s0 & 15u), mine, nvec,
                                reinterpret_cast<uint4 *>(out + lead));
    }
}


// ---------------------------------------------------------------------------------------------
// A tile's descriptors: kLevels pairs of 64-bit words per tile in the workspace.  A pair holds one 64-bit sum:
//   word 0 = (tag >> 32) << 32 | low half of the sum,   word 1 = (tag & 0xFFFFFFFF) << 32 | high half of the sum
// Both words carry half of the launch's tag: a reader takes the pair only if both halves are those of its own
// launch, so the two words may be written and read separately, and memory this library never wrote matches by
// chance only (2^-64).  Pair 0 of tile t is the tile's own count.  Pair L (L >= 1) is written only by the last
// tile of a group of 64^L tiles (t = 64^L - 1 mod 64^L, counted inside its tensor) and holds the count of that
// whole group.
struct TagHalves {
    uint64_t w0, w1;
    __device__ __forceinline__ explicit TagHalves(uint64_t tag) : w0(tag & 0xFFFFFFFF00000000ull), w1(tag << 32) {}
    __device__ __forceinline__ bool valid(uint64_t d0, uint64_t d1) const { return ((d0 ^ w0) >> 32) == 0 && ((d1 ^ w1) >> 32) == 0; }
    __device__ __forceinline__ static uint64_t value(uint64_t d0, uint64_t d1) { return (d0 & 0xFFFFFFFFull) | (d1 << 32); }
    __device__ __forceinline__ void publish(uint64_t *pair, uint64_t sum) const { st_relaxed_2xu64(pair, w0 | (sum & 0xFFFFFFFFull), w1 | (sum >> 32)); }
};
constexpr int kLevels    = 4;                     // 64^4 tiles of 32 KB: more than a tensor can hold
constexpr int kDescWords = 2 * kLevels;           // 64-bit words per tile

// Raise the abort flag under this launch's tag, move the workspace's sequence number so that the next launch
// cannot take this one's words for its own, and report the timeout in every tensor's status word.
template <int kJobs>
__device__ __noinline__ void raise_timeout(const CompressParams<kJobs> &p, const uint64_t tag)
{
    st_relaxed_u64(p.c.ws_header + kHdrAbort, tag);
    red_add_u64(p.c.ws_header + kHdrSeq, 1ull << 32);
    __threadfence();
    for (uint32_t k = 0; k < p.c.jobs; ++k)
        if (p.job[k].dev_status) *reinterpret_cast<volatile int32_t *>(p.job[k].dev_status) = BT_ERR_TIMEOUT;
}

// Shape of a CTA: 8 warps, a tile of 32 KB whatever the element width (512 8-byte, 1024 4-byte or 2048 2-byte
// elements per warp: one, two or four chunks of the prefix array per tile).  The look-back advances at most one
// window of tiles per round trip to L2, so a tile must be worth that round trip's share of the memory bandwidth;
// kMinBlocks CTAs per SM bound the registers (the loaded vectors of all resident CTAs are the bytes in flight).
template <typename U>
struct TileShape {
    static constexpr int kWarps     = 8;
    static constexpr int kSeg       = 4096 / sizeof(U);
    static constexpr int kTile      = kWarps * kSeg;
    static constexpr int kThreads   = kWarps * 32;
    static constexpr int kMinBlocks = 6;
};

// U: uint64_t, uint32_t or uint16_t (the element's width).
// FUSED: -1 for the plain compressor, else the number of the fused forward form (element type, + 4 for ReLU6).
// CAST: 0, or the 16-bit type the packed binary32 values are narrowed to on their way out (1 binary16, 2 bfloat16).
// kJobs: room for tensors in the kernel's parameters (1, or kMaxBatch for the batched forms).
template <typename U, int FUSED, bool WRITE_Y, int CAST, int kJobs>
__global__ void __launch_bounds__(TileShape<U>::kThreads, TileShape<U>::kMinBlocks)
compress_kernel(const __grid_constant__ CompressParams<kJobs> p)
{
    using T                      = TileShape<U>;
    constexpr int kW             = T::kWarps;
    constexpr int kSeg           = T::kSeg;
    constexpr int kTile          = T::kTile;
    constexpr int kChunksPerTile = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk = BT_CHUNK_ELEMS / kSeg;
    using S                      = Seg<U, kSeg>;
    using V                      = Stored<CAST, U>;

    __shared__ __align__(128) U            s_tile[kTile];              // the tile as it lands; packed in place, segment by segment
    __shared__ __align__(16) unsigned char s_bits[kW][kSeg / 8];       // bitmap bytes of each warp's segment
    __shared__ __align__(8) uint64_t       s_landed;                   // mbarrier: the bulk copy of the tile has landed
    __shared__ uint32_t                    s_wcnt[kW];                 // kept elements of each warp's segment
    __shared__ uint64_t                    s_tag;                      // the launch's tag
    __shared__ uint64_t                    s_excl;                     // the tile's exclusive prefix
    __shared__ uint64_t                    s_arena_c0;                 // arena forms: the cursor as this launch found it
    __shared__ uint32_t                    s_failed;

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;

    // which tile of which tensor: tiles are numbered tensor after tensor, in the order of the block index
    uint32_t k = 0;
    uint64_t t = blockIdx.x;
    if constexpr (kJobs > 1) {
        while (t >= p.job[k].tiles) t -= p.job[k].tiles, ++k;
    }
    const CompressJob &jb    = p.job[k];
    const uint64_t     n     = jb.n;
    const uint64_t     first = t * kTile;                               // the tile's first element
    const uint32_t     have  = n - first < static_cast<uint64_t>(kTile) ? static_cast<uint32_t>(n - first) : static_cast<uint32_t>(kTile);
    const uint64_t     e0    = first + warp * kSeg;                     // first element of this warp's segment
    const uint32_t     valid = have > warp * kSeg ? (have - warp * kSeg < static_cast<uint32_t>(kSeg) ? have - warp * kSeg : static_cast<uint32_t>(kSeg)) : 0u;
    uint64_t *const    desc  = p.c.ws_desc + kDescWords * static_cast<uint64_t>(blockIdx.x);
    const U *const     src   = static_cast<const U *>(jb.src) + first;

    // ---- the tile into shared memory: one bulk copy (whole 16-byte units; the few elements behind them and the
    // zeros of a ragged last tile by ordinary stores).  The first thread also reads the workspace's sequence number
    // (and the arena's cursor): every CTA does so before it publishes anything, and both change only after the last
    // tile of the launch has seen a publication from every tile.
    const uint32_t bytes = (have * static_cast<uint32_t>(sizeof(U))) & ~15u;
    if (tid == 0) {
        mbar_init(&s_landed, 1);
        fence_proxy_async();
        mbar_arrive_expect_tx(&s_landed, bytes);
        if (bytes) bulk_load(s_tile, src, bytes, &s_landed);
        const uint64_t seq = ld_relaxed_u64(p.c.ws_header + kHdrSeq);
        s_arena_c0         = p.c.arena_cursor ? ld_relaxed_u64(p.c.arena_cursor) : 0;
        s_tag              = mix64(p.c.call_tag + seq * 0x9E3779B97F4A7C15ull) | 1ull;
        s_failed           = 0;
    }
    if (have < static_cast<uint32_t>(kTile)) {
        for (uint32_t e = bytes / sizeof(U) + tid; e < static_cast<uint32_t>(kTile); e += T::kThreads) s_tile[e] = e < have ? src[e] : U(0);
    }
    __syncthreads();                                 // the barrier is initialised; the tail is in place
    {
        const uint64_t t0 = now_ns();
        while (!mbar_try_wait(&s_landed, 0)) {
            if (now_ns() - t0 > p.c.wait_ns) {       // cannot happen unless the copy engine is stuck: leave without touching the tile
                if (tid == 0) raise_timeout(p, s_tag);
                return;
            }
        }
    }

    // ---- (1) first pass: masks (and the fused forward form)
    const uint32_t seg_addr = smem_addr(s_tile + warp * kSeg);
    uint32_t       m[S::kSteps];
    segment_masks<U, FUSED, WRITE_Y, kSeg>(seg_addr, valid, lane, m, WRITE_Y ? static_cast<U *>(jb.y) + e0 : nullptr, p.c.tau);

    // ---- (3a) count, and out with the tile's count as early as possible: the tiles behind this one wait for it,
    // and every microsecond it is out before they ask saves them a second round trip to L2
    uint32_t       inc[S::kBatches], packed[S::kBatches];
    const uint32_t cnt = segment_count<U, kSeg>(m, packed);
    if (lane == 0) s_wcnt[warp] = cnt;
    __syncthreads();
    // every warp: where its run goes in the tensor's packed values relative to the tile's, and the tile's count
    uint32_t before = 0, total = 0;
#pragma unroll
    for (int j = 0; j < kW; ++j) {
        const uint32_t c = s_wcnt[j];
        before += j < static_cast<int>(warp) ? c : 0u;
        total += c;
    }
    const TagHalves tag(s_tag);
    if (tid == 0) tag.publish(desc, total);

    // ---- (2) the bitmap
    uint32_t word[S::kWordsPerLane];
    segment_bitmap<U, kSeg>(m, smem_addr(&s_bits[warp][0]), lane, word);
    if (lane * S::kWordsPerLane < static_cast<uint32_t>(S::kWords)) {
        const uint64_t wd = t * (kTile / 32) + warp * S::kWords + lane * S::kWordsPerLane;
#pragma unroll
        for (int j = 0; j < S::kWordsPerLane; ++j)
            if (wd + j < ((n + 31) >> 5)) jb.bitmap[wd + j] = word[j];
    }

    // ---- (3b) the lanes' offsets, (4) second pass: the segment packed in place
    segment_scan<U, kSeg>(packed, inc, lane);
    segment_pack<U, kSeg>(seg_addr, lane, m, inc, packed);

    // ---- warp 0 gathers the tile's exclusive prefix.  With t = a + 64 b + 4096 c + 262144 d (digits of the tile's
    // number inside its tensor) it is the counts of the a tiles before it in its group of 64, of the b groups of 64
    // before that group in their group of 4096, of the c groups of 4096 before that one, and of the d groups of
    // 262144 before that: at most 63 sums per level, two per lane, all read at once.  Nothing here waits for another
    // tile's prefix -- only for counts, and for group counts that the last tile of a group forms from counts.
    if (warp == 0) {
        const uint64_t g0 = static_cast<uint64_t>(blockIdx.x) - t;               // the tensor's first tile
        uint64_t       sum[kLevels];                                             // this lane's share of each level
        bool           got[kLevels][2];
        uint32_t       digit[kLevels];
        {
            uint64_t r = t;
#pragma unroll
            for (int L = 0; L < kLevels; ++L) digit[L] = static_cast<uint32_t>(r & 63u), r >>= 6, sum[L] = 0, got[L][0] = got[L][1] = false;
        }
        // group counts this tile closes: that of level L + 1 if its digits 0 .. L are all 63 -- it goes out as soon as
        // the levels up to L are complete (it must not wait for the higher levels: they wait for other groups' counts,
        // and a count that waits for counts is a chain again)
        uint32_t closes = 0;
#pragma unroll
        for (int L = 0; L + 1 < kLevels; ++L) {
            if (digit[L] != 63u) break;
            closes = L + 1;
        }
        uint32_t published = 0;             // group counts of levels 1 .. published are out
        bool     failed    = false;
        uint32_t polls     = 0;
        uint64_t t_start   = 0;
        for (;;) {
            uint32_t missing = 0;           // bit L: an entry of level L is not there yet
            uint64_t span    = 1;           // tiles in an entry of the level: 64^L
            uint64_t floor_t = t;           // the tile's number with the digits below the level cleared
#pragma unroll
            for (int L = 0; L < kLevels; ++L) {
                floor_t -= static_cast<uint64_t>(digit[L]) * span;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint32_t i = lane + 32u * j;                           // entry i of the level
                    if (i < digit[L] && !got[L][j]) {
                        // the group of 64^L tiles that starts at floor_t + i * span; its count sits with its last tile
                        const uint64_t *d = p.c.ws_desc + kDescWords * (g0 + floor_t + (i + 1) * span - 1) + 2 * L;
                        uint64_t        d0, d1;
                        ld_relaxed_2xu64(d, d0, d1);
                        if (tag.valid(d0, d1)) {
                            got[L][j] = true;
                            sum[L] += TagHalves::value(d0, d1);
                        } else {
                            missing |= 1u << L;
                        }
                    }
                }
                span <<= 6;
            }
            missing = __reduce_or_sync(kFull, missing);
            if (published < closes) {
                uint64_t upto = total;
#pragma unroll
                for (int L = 0; L + 1 < kLevels; ++L) {
                    if (static_cast<uint32_t>(L) >= closes || (missing & ((2u << L) - 1u))) break;      // a level up to L is incomplete
                    upto += warp_sum_u64(sum[L]);
                    if (published == static_cast<uint32_t>(L)) {
                        if (lane == 0) tag.publish(desc + 2 * (L + 1), upto);
                        published = L + 1;
                    }
                }
            }
            if (!missing) break;
            __nanosleep(32);
            if ((++polls & 63u) == 0 || p.c.wait_ns < 1000000ull) {
                if (t_start == 0) t_start = now_ns();
                if (__any_sync(kFull, now_ns() - t_start > p.c.wait_ns || ld_relaxed_u64(p.c.ws_header + kHdrAbort) == s_tag)) {
                    failed = true;
                    break;
                }
            }
        }
        uint64_t excl = 0;
        if (!failed) {
#pragma unroll
            for (int L = 0; L < kLevels; ++L) excl += warp_sum_u64(sum[L]);
        }
        if (lane == 0) {
            if (failed) {
                raise_timeout(p, s_tag);
                s_failed = 1;
            } else {
                s_excl = excl;
            }
        }
        __syncwarp();
        if (!failed) {
            // exclusive count in front of each chunk of the tile
            if (lane < static_cast<uint32_t>(kChunksPerTile)) {
                const uint64_t ch = t * kChunksPerTile + lane;
                uint64_t       at = excl;
                for (uint32_t j = 0; j < lane * kWarpsPerChunk; ++j) at += s_wcnt[j];
                if (ch < (n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS) jb.prefix[ch] = at;
            }
            if (lane == 0 && t == jb.tiles - 1) {
                // the tensor's last tile: the count of the tensor, the status word, the arena's cursor
                const uint64_t incl = excl + total;
                *jb.nnz_out         = incl;
                uint64_t capacity   = jb.capacity;
                bool     fits       = incl <= capacity;
                if (p.c.arena_cursor) {
                    const uint64_t cur = s_arena_c0;
                    capacity           = cur <= p.c.arena_bytes ? (p.c.arena_bytes - cur) / sizeof(V) : 0;
                    fits               = incl <= capacity;
                    if (fits) {
                        *p.c.values_offset_out = cur;
                        *p.c.arena_cursor      = cur + ((incl * sizeof(V) + 15) & ~15ull);
                    }
                }
                if (jb.dev_status) {
                    *reinterpret_cast<volatile int32_t *>(jb.dev_status) = fits ? BT_OK : BT_ERR_CAPACITY;
                    // a CTA that gives up from now on stores its BT_ERR_TIMEOUT after this word; one that gave
                    // up just before is seen here
                    __threadfence();
                    if (ld_relaxed_u64(p.c.ws_header + kHdrAbort) == s_tag) *reinterpret_cast<volatile int32_t *>(jb.dev_status) = BT_ERR_TIMEOUT;
                }
                // Every tile of this tensor has published its count by now (the sums above cover them all).  The
                // tensor's last tile says so in the header; the launch's last tile waits for the other tensors' words,
                // after which every CTA has read the sequence number and the next launch gets another tag.
                __threadfence();
                st_relaxed_u64(p.c.ws_header + kHdrDone + k, s_tag);
                if (k + 1 == p.c.jobs) {
                    bool all = true;
                    for (uint32_t kk = 0; all && kk + 1 < p.c.jobs; ++kk) {
                        const uint64_t t0 = now_ns();
                        while (ld_relaxed_u64(p.c.ws_header + kHdrDone + kk) != s_tag) {
                            if (now_ns() - t0 > p.c.wait_ns) {
                                all = false;
                                break;
                            }
                            __nanosleep(100);
                        }
                    }
                    red_add_u64(p.c.ws_header + kHdrSeq, all ? 1ull : 1ull << 32);
                }
            }
        }
    }
    __syncthreads();
    if (s_failed) return;

    // ---- the staged run to values[exclusive prefix ...]
    V       *vals     = static_cast<V *>(jb.values);
    uint64_t capacity = jb.capacity;
    if (p.c.arena_cursor) {
        const uint64_t cur = s_arena_c0;
        vals               = reinterpret_cast<V *>(static_cast<unsigned char *>(jb.values) + cur);
        capacity           = cur <= p.c.arena_bytes ? (p.c.arena_bytes - cur) / sizeof(V) : 0;
    }
    // every warp copies its own run, which starts its segment
    __syncwarp();
    const uint64_t base = s_excl + before;
    const U *const run  = s_tile + warp * kSeg;
    if (base + cnt <= capacity) {
        copy_out_piece<U, CAST, 1, false>(run, cnt, vals + base, 0, 0, lane);
    } else {
        copy_out_piece<U, CAST, 1, true>(run, cnt, vals + base, base < capacity ? capacity - base : 0, 0, lane);
    }
}

// A value no other call of this process gets: a counter that starts at a salt drawn from the clock and the
// address space, so that words left in recycled memory by another run of the library do not line up either.
uint64_t next_call_tag()
{
    static std::atomic<uint64_t> counter{
        mix64(static_cast<uint64_t>(std::chrono::steady_clock::now().time_since_epoch().count()) ^
              mix64(reinterpret_cast<uintptr_t>(&counter)))};
    return counter.fetch_add(1, std::memory_order_relaxed);
}

// The bound of the kernels' waits; only a test build can change it.
std::atomic<uint64_t> g_wait_ns{kDefaultWaitNs};

template <typename U, int FUSED, bool WRITE_Y, int CAST, int kJobs>
cudaError_t launch_sized(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, cudaStream_t stream)
{
    if (count == 0 || count > static_cast<uint32_t>(kJobs)) return cudaErrorInvalidValue;
    CompressParams<kJobs> p;
    p.c            = c;
    uint64_t tiles = 0;
    for (uint32_t k = 0; k < count; ++k) {
        p.job[k]         = jobs[k];
        const uint64_t t = (jobs[k].n + TileShape<U>::kTile - 1) / TileShape<U>::kTile;
        if (t == 0 || t > 0x7FFFFFFFull) return cudaErrorInvalidValue;
        p.job[k].tiles   = static_cast<uint32_t>(t);
        tiles += t;
    }
    if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;                 // one CTA per tile
    for (uint32_t k = count; k < static_cast<uint32_t>(kJobs); ++k) p.job[k] = CompressJob{};
    p.c.jobs      = count;
    p.c.ws_header = static_cast<uint64_t *>(workspace);
    p.c.ws_desc   = reinterpret_cast<uint64_t *>(static_cast<unsigned char *>(workspace) + kWsHeaderBytes);
    p.c.call_tag  = next_call_tag();
    p.c.wait_ns   = g_wait_ns.load(std::memory_order_relaxed);
    compress_kernel<U, FUSED, WRITE_Y, CAST, kJobs><<<static_cast<unsigned>(tiles), TileShape<U>::kThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

template <typename U, int FUSED, bool WRITE_Y, int CAST = 0>
cudaError_t launch_typed(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, cudaStream_t stream)
{
    // batches (plain and ReLU forms only) run the instantiation with room for kMaxBatch tensors
    constexpr bool kBatchable = CAST == 0 && FUSED < kFusedRelu6;
    if constexpr (kBatchable) {
        if (count > 1) return launch_sized<U, FUSED, WRITE_Y, CAST, kMaxBatch>(c, jobs, count, workspace, stream);
    }
    if (count != 1) return cudaErrorInvalidValue;
    return launch_sized<U, FUSED, WRITE_Y, CAST, 1>(c, jobs, count, workspace, stream);
}

}  // namespace

uint64_t set_compress_wait_ns(uint64_t wait_ns) { return g_wait_ns.exchange(wait_ns, std::memory_order_relaxed); }

cudaError_t launch_compress(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, int dtype,
                            int fused, cudaStream_t stream)
{
    // fused: 0 plain compressor, 1 threshold form (ReLU at tau = 0), 2 ReLU6
    // the dense output is written for all tensors of a launch or for none
    const bool y = jobs[0].y != nullptr;
    for (uint32_t k = 1; k < count; ++k)
        if ((jobs[k].y != nullptr) != y) return cudaErrorInvalidValue;
    if (c.cast != 0) {
        // down-cast on stash: binary32 tensors, plain and threshold forms
        if (dtype != BT_F32 || fused == 2) return cudaErrorInvalidValue;
        const bool h = c.cast == BT_F16;
        if (fused == 0)
            return h ? launch_typed<uint32_t, -1, false, 1>(c, jobs, count, workspace, stream)
                     : launch_typed<uint32_t, -1, false, 2>(c, jobs, count, workspace, stream);
        if (y)
            return h ? launch_typed<uint32_t, BT_F32, true, 1>(c, jobs, count, workspace, stream)
                     : launch_typed<uint32_t, BT_F32, true, 2>(c, jobs, count, workspace, stream);
        return h ? launch_typed<uint32_t, BT_F32, false, 1>(c, jobs, count, workspace, stream)
                 : launch_typed<uint32_t, BT_F32, false, 2>(c, jobs, count, workspace, stream);
    }
    if (fused == 0) {
        return dtype == BT_F64   ? launch_typed<uint64_t, -1, false>(c, jobs, count, workspace, stream)
               : dtype == BT_F32 ? launch_typed<uint32_t, -1, false>(c, jobs, count, workspace, stream)
                                 : launch_typed<uint16_t, -1, false>(c, jobs, count, workspace, stream);
    }
    constexpr int k6 = kFusedRelu6;
    if (fused == 2) {
        switch (dtype) {
        case BT_F64:
            return y ? launch_typed<uint64_t, k6 + BT_F64, true>(c, jobs, count, workspace, stream)
                     : launch_typed<uint64_t, k6 + BT_F64, false>(c, jobs, count, workspace, stream);
        case BT_F32:
            return y ? launch_typed<uint32_t, k6 + BT_F32, true>(c, jobs, count, workspace, stream)
                     : launch_typed<uint32_t, k6 + BT_F32, false>(c, jobs, count, workspace, stream);
        case BT_F16:
            return y ? launch_typed<uint16_t, k6 + BT_F16, true>(c, jobs, count, workspace, stream)
                     : launch_typed<uint16_t, k6 + BT_F16, false>(c, jobs, count, workspace, stream);
        default:
            return y ? launch_typed<uint16_t, k6 + BT_BF16, true>(c, jobs, count, workspace, stream)
                     : launch_typed<uint16_t, k6 + BT_BF16, false>(c, jobs, count, workspace, stream);
        }
    }
    switch (dtype) {
    case BT_F64:
        return y ? launch_typed<uint64_t, BT_F64, true>(c, jobs, count, workspace, stream)
                 : launch_typed<uint64_t, BT_F64, false>(c, jobs, count, workspace, stream);
    case BT_F32:
        return y ? launch_typed<uint32_t, BT_F32, true>(c, jobs, count, workspace, stream)
                 : launch_typed<uint32_t, BT_F32, false>(c, jobs, count, workspace, stream);
    case BT_F16:
        return y ? launch_typed<uint16_t, BT_F16, true>(c, jobs, count, workspace, stream)
                 : launch_typed<uint16_t, BT_F16, false>(c, jobs, count, workspace, stream);
    default:
        return y ? launch_typed<uint16_t, BT_BF16, true>(c, jobs, count, workspace, stream)
                 : launch_typed<uint16_t, BT_BF16, false>(c, jobs, count, workspace, stream);
    }
}

}  // namespace bt
