// Algorithm 1 (dense -> bitmap) and its fused forms (ReLU, activation pruning, ReLU6) as ONE
// compaction pass over one tensor or a batch of tensors: a persistent-CTA stream compaction whose
// prefix sum rides on the wave structure of the grid.
//
// The grid is launched cooperatively with as many CTAs (G) as fit on the device at once, so all of
// them are co-resident.  The tiles of a launch are dealt round robin: tile t of tensor k goes to CTA
// (rot_k + t) mod G, where rot_k continues the deal of the tensor before it, so every CTA gets the
// same share of a batch whatever the tensors' sizes.  Inside a tensor, tiles [jG, (j+1)G) form
// "wave j"; a CTA takes at most one tile of a wave and takes its tiles in order.  The warps of a
// CTA are specialised: one load warp, kWarps compactor warps, two scan warps, kCopiers copier warps.
//
// Compaction.  Compactor warp w owns segment w of the tile.  A lane takes one 16-byte vector of
// the segment per step (kVec consecutive elements), so a warp covers 32 * kVec elements per step:
//
//   - one 16-byte shared load; a kVec-bit mask of the elements whose pattern is not zero (after
//     the fused forward form, if any);
//   - the masks ARE the bitmap: lanes that share a bitmap byte combine their bits with one or two
//     shuffles and store the byte in a small staging area; at the end lane k reads word k of the
//     segment back and the 32 words leave as one coalesced 128-byte store;
//   - the counts of several steps ride in the fields of one register through ONE warp scan (five
//     shuffles) -- 2 steps for 2-byte, 4 steps for wider elements;
//   - every lane stores its surviving elements, in place, at its exclusive offset behind the
//     segment's running output position: the write position never passes the read position, and a
//     batch's loads are issued before the stores of the batch before it.
//
// Prefix.  The exclusive base of tile (tensor k, wave j, virtual CTA v) is
//     sum of the totals of waves 0..j-1 of tensor k  +  sum of the counts of virtual CTAs 0..v-1 in wave j.
// As soon as a tile is counted a scan warp publishes the count in a descriptor and adds it (with a
// 1 in a counter field) to the wave's total with one fire-and-forget reduction.  About one tile
// later -- when every CTA has published that wave -- it reads the v descriptors of its wave and the
// now complete totals of the two waves before it in ONE batch of independent loads, and uses them a
// tile after that.  The two scan warps alternate tiles, so that each has two tiles' time for that
// round trip to L2.  No tile waits on another tile's base: only on counts, which never wait on
// anything but data.
//
// Pipeline.  The warps of a CTA never meet at a CTA-wide barrier after the prologue; a ring slot
// goes round through four mbarriers:
//   full[s]     the bulk copy of the tile has landed         (copy engine -> compactors)
//   counted[s]  every compactor has posted its count         (compactors  -> scan warps)
//   ready[s]    base and segment offsets are in shared       (scan warp   -> copiers)
//   empty[s]    every copier has copied its segments out     (copiers     -> load warp)
// Copier warp c copies its segments' packed values to values[base + offset ...].
//
// Workspace.  It arrives with unspecified contents and is not cleared.  A tile's descriptor carries
// the launch's 64-bit tag in both of its halves, and a reader takes only descriptors with its own
// launch's tag; so counts are published and read from the first tile on.  Only the wave totals,
// being sums, need zeroed words: the last copier warp of every CTA zeroes a share of them and
// writes the launch's tag into the CTA's arrival word; when it has seen all G arrival words it
// declares the grid met.  Until then the scan warps park their contributions to totals in shared
// memory (the copier warp adds them afterwards) and take no total for read.
#include <atomic>
#include <chrono>
#include <cstdlib>
#include <mutex>
#include <type_traits>

#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr uint32_t kFull       = 0xFFFFFFFFu;
constexpr int      kBarWorkers = 1;                   // named barrier of the worker warps (ragged tile only)
constexpr int      kMaxWindows = kMaxGrid / 32;       // descriptor windows of 32 CTAs
constexpr int      kHdrSeq     = 0;                   // header words (64-bit): launch sequence number,
constexpr int      kHdrAbort   = 1;                   //   abort word (== the launch's tag once a wait ran out),
constexpr int      kHdrGo      = 2;                   //   go word (== the launch's tag once every CTA has arrived at the meeting)
constexpr int      kCountShift = 40;                  // wave total word: (tiles added << 40) | sum of counts
constexpr uint32_t kDirect     = 4;                   // waves of a tensor whose bases come from descriptors alone

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

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void red_add_u64(uint64_t *p, uint64_t v)
{
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ uint64_t ld_acquire_u64(const uint64_t *p)
{
    uint64_t v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_release_u64(uint64_t *p, uint64_t v)
{
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
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

// Raise the abort flag (shared, and global under this launch's tag if the CTA got as far as reading it), move
// the workspace's sequence number so that the next launch cannot take this one's words for its own, and report
// the timeout in every tensor's status word.
template <int kJobs>
__device__ __noinline__ void raise_timeout(const CompressParams<kJobs> &p, volatile uint32_t *s_abort, const uint64_t tag)
{
    *s_abort = 1u;
    if (tag) st_relaxed_u64(p.c.ws_header + kHdrAbort, tag);
    red_add_u64(p.c.ws_header + kHdrSeq, 1ull << 32);
    __threadfence();
    for (uint32_t k = 0; k < p.c.jobs; ++k)
        if (p.job[k].dev_status) *reinterpret_cast<volatile int32_t *>(p.job[k].dev_status) = BT_ERR_TIMEOUT;
}

// Bounded wait on an mbarrier phase.  False once the limit passed or the CTA is aborting.  A warp that waits
// sleeps kSleepNs between probes: a probe loop without it takes a third of the SM's issue slots from the warps
// that work (the hardware holds a probing thread only for some tens of cycles), and the clock and the abort
// flag are looked at every 64 probes only.
template <bool kStopOnAbort = true, unsigned kSleepNs = 100>
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *s_abort, const uint64_t limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t probes = 1;; ++probes) {
        __nanosleep(kSleepNs);
        if (mbar_try_wait(bar, parity)) return true;
        if ((probes & 63u) == 0 || limit_ns < 1000000ull) {
            if (t0 == 0) t0 = now_ns();
            if ((kStopOnAbort && *s_abort) || now_ns() - t0 > limit_ns) return false;
        }
    }
}

// The launch's tag as the first scan warp left it in shared memory (bounded wait; 0 if the CTA is aborting).
__device__ __forceinline__ uint64_t wait_tag(volatile uint64_t *s_tag, volatile uint32_t *s_abort, const uint64_t limit_ns)
{
    uint64_t t = *s_tag;
    if (t) return t;
    const uint64_t t0 = now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i) {
            t = *s_tag;
            if (t) return t;
        }
        if (*s_abort || now_ns() - t0 > limit_ns) return 0;
    }
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

// The kept elements of one 16-byte vector, stored one behind the other from `addr` on, which moves past them:
// per element a test of its pattern, a predicated store and a predicated add (a branch per element costs more
// than the element's other work).
template <typename U>
__device__ __forceinline__ void sts_kept(uint32_t &addr, const uint4 &v)
{
    if constexpr (sizeof(U) == 8) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b32 t;\n\t"
            "or.b32 t, %1, %2;\n\tsetp.ne.u32 p, t, 0;\n\t@p st.shared.v2.u32 [%0], {%1, %2};\n\t@p add.u32 %0, %0, 8;\n\t"
            "or.b32 t, %3, %4;\n\tsetp.ne.u32 p, t, 0;\n\t@p st.shared.v2.u32 [%0], {%3, %4};\n\t@p add.u32 %0, %0, 8;\n\t}"
            : "+r"(addr)
            : "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
    } else if constexpr (sizeof(U) == 4) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.u32 p, %1, 0;\n\t@p st.shared.u32 [%0], %1;\n\t@p add.u32 %0, %0, 4;\n\t"
            "setp.ne.u32 p, %2, 0;\n\t@p st.shared.u32 [%0], %2;\n\t@p add.u32 %0, %0, 4;\n\t"
            "setp.ne.u32 p, %3, 0;\n\t@p st.shared.u32 [%0], %3;\n\t@p add.u32 %0, %0, 4;\n\t"
            "setp.ne.u32 p, %4, 0;\n\t@p st.shared.u32 [%0], %4;\n\t@p add.u32 %0, %0, 4;\n\t}"
            : "+r"(addr)
            : "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
    } else {
#define BT_STS_HALVES(X)                                                                                                  \
    "mov.b32 {l, h}, " X ";\n\tand.b32 t, " X ", 0xFFFF;\n\tsetp.ne.u32 p, t, 0;\n\t@p st.shared.u16 [%0], l;\n\t@p add.u32 %0, %0, 2;\n\t" \
    "setp.gt.u32 p, " X ", 0xFFFF;\n\t@p st.shared.u16 [%0], h;\n\t@p add.u32 %0, %0, 2;\n\t"
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b16 l, h;\n\t.reg .b32 t;\n\t" BT_STS_HALVES("%1") BT_STS_HALVES("%2") BT_STS_HALVES("%3") BT_STS_HALVES("%4") "}"
                     : "+r"(addr)
                     : "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
#undef BT_STS_HALVES
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

// (1) the segment into registers, the fused forward form applied, one mask per step (bit k: the lane's k-th
// element of the step is kept, i.e. its pattern is not zero), the dense output written.
template <typename U, int FUSED, bool WRITE_Y, bool kGuardY, int kSeg>
__device__ __forceinline__ void segment_load(const uint32_t seg_addr, const uint32_t lane, uint4 (&q)[Seg<U, kSeg>::kSteps],
                                             uint32_t (&m)[Seg<U, kSeg>::kSteps], U *y, const uint32_t yvalid, const float tau)
{
    using S = Seg<U, kSeg>;
#pragma unroll
    for (int s = 0; s < S::kSteps; ++s) q[s] = lds_vec(seg_addr + lane * 16u + s * 512u);
#pragma unroll
    for (int s = 0; s < S::kSteps; ++s) {
        if constexpr (FUSED >= 0) {
            Reg<U> e[S::kVec];
            unpack<U>(q[s], e);
#pragma unroll
            for (int k = 0; k < S::kVec; ++k) e[k] = fused_forward<FUSED>(e[k], tau);
            q[s] = repack<U>(e);
            if constexpr (WRITE_Y) {
                const uint32_t at = (s * 32 + lane) * S::kVec;                // first element of the vector in the segment
                if (!kGuardY || at + S::kVec <= yvalid) {
                    *reinterpret_cast<uint4 *>(y + at) = q[s];
                } else {
#pragma unroll
                    for (int k = 0; k < S::kVec; ++k)
                        if (at + k < yvalid) y[at + k] = static_cast<U>(e[k]);
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

// (3) one warp scan per batch of steps (the counts of a batch's steps ride in the fields of one register), the
// batches' scans side by side.  Leaves the inclusive sums in inc[], the lane's own counts in packed[]; returns
// the number of kept elements of the segment.
template <typename U, int kSeg>
__device__ __forceinline__ uint32_t segment_scan(const uint32_t (&m)[Seg<U, kSeg>::kSteps], uint32_t (&inc)[Seg<U, kSeg>::kBatches],
                                                 uint32_t (&packed)[Seg<U, kSeg>::kBatches], const uint32_t lane)
{
    using S = Seg<U, kSeg>;
#pragma unroll
    for (int b = 0; b < S::kBatches; ++b) {
        packed[b] = 0;
#pragma unroll
        for (int p = 0; p < S::kPack; ++p) packed[b] |= static_cast<uint32_t>(__popc(m[b * S::kPack + p])) << (p * S::kFB);
        inc[b] = packed[b];
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t u[S::kBatches];
#pragma unroll
        for (int b = 0; b < S::kBatches; ++b) u[b] = __shfl_up_sync(kFull, inc[b], o);
#pragma unroll
        for (int b = 0; b < S::kBatches; ++b)
            if (lane >= static_cast<uint32_t>(o)) inc[b] += u[b];
    }
    uint32_t cnt = 0;
#pragma unroll
    for (int b = 0; b < S::kBatches; ++b) {
        const uint32_t tot = __shfl_sync(kFull, inc[b], 31);
#pragma unroll
        for (int p = 0; p < S::kPack; ++p) cnt += (tot >> (p * S::kFB)) & S::kFieldMask;
    }
    return cnt;
}

// (4) every lane stores its kept elements at its exclusive offset behind `at0`, the shared-window address where
// the segment's packed run starts.
template <typename U, int kSeg>
__device__ __forceinline__ void segment_store(const uint4 (&q)[Seg<U, kSeg>::kSteps], const uint32_t (&inc)[Seg<U, kSeg>::kBatches],
                                              const uint32_t (&packed)[Seg<U, kSeg>::kBatches], const uint32_t at0)
{
    using S        = Seg<U, kSeg>;
    uint32_t out = at0;                              // address of the step's first packed slot (warp-uniform)
#pragma unroll
    for (int b = 0; b < S::kBatches; ++b) {
        const uint32_t tot = __shfl_sync(kFull, inc[b], 31);
        const uint32_t exc = inc[b] - packed[b];
#pragma unroll
        for (int p = 0; p < S::kPack; ++p) {
            uint32_t at = out + S::kES * ((exc >> (p * S::kFB)) & S::kFieldMask);
            sts_kept<U>(at, q[b * S::kPack + p]);
            out += S::kES * ((tot >> (p * S::kFB)) & S::kFieldMask);
        }
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
// The tiles of a launch in the order one CTA takes them: tensor after tensor; inside tensor k the tiles
// v, v + G, v + 2G, ... with v = (cta - rot_k) mod G, the CTA's place in the deal of that tensor.
struct Walk {
    uint32_t k;       // tensor
    uint32_t j;       // wave of the tensor; the tile is v + j * G
    uint32_t v;       // this CTA's virtual index in the tensor
    uint32_t tiles;   // tiles of the tensor
    bool     valid;
    __device__ __forceinline__ uint32_t tile(const uint32_t G) const { return v + j * G; }
};

template <int kJobs>
__device__ __forceinline__ void walk_seek(Walk &w, const CompressParams<kJobs> &p, const uint32_t cta, const uint32_t G)
{
    while (w.k < p.c.jobs) {
        const uint32_t rot = p.job[kJobs == 1 ? 0u : w.k].rot;
        w.tiles            = p.job[kJobs == 1 ? 0u : w.k].tiles;
        w.v                = cta >= rot ? cta - rot : cta + G - rot;
        if (w.v < w.tiles) {
            w.j     = 0;
            w.valid = true;
            return;
        }
        ++w.k;
    }
    w.valid = false;
}
template <int kJobs>
__device__ __forceinline__ void walk_begin(Walk &w, const CompressParams<kJobs> &p, const uint32_t cta, const uint32_t G)
{
    w.k = 0, w.j = 0, w.v = 0, w.tiles = 0;
    walk_seek(w, p, cta, G);
}
template <int kJobs>
__device__ __forceinline__ void walk_next(Walk &w, const CompressParams<kJobs> &p, const uint32_t cta, const uint32_t G)
{
    ++w.j;
    if (static_cast<uint64_t>(w.v) + static_cast<uint64_t>(w.j) * G >= w.tiles) {
        ++w.k;
        walk_seek(w, p, cta, G);
    }
}

// U: uint64_t, uint32_t or uint16_t (the element's width).
// FUSED: -1 for the plain compressor, else the number of the fused forward form (element type, + 4 for ReLU6).
// CAST: 0, or the 16-bit type the copiers narrow the packed binary32 values to (1 binary16, 2 bfloat16).
// kJobs: room for tensors in the kernel's parameters (1, or kMaxBatch for the batched forms).
// kWarps compactor warps, kSeg elements per warp, kStages ring slots, kCopiers copier warps.
template <typename U, int FUSED, bool WRITE_Y, int CAST, int kJobs, int kWarps, int kSeg, int kStages, int kCopiers>
__global__ void __launch_bounds__((kWarps + kCopiers + 3) * 32)
compress_kernel(const __grid_constant__ CompressParams<kJobs> p)
{
    using S                       = Seg<U, kSeg>;
    constexpr int kTile           = kWarps * kSeg;
    constexpr int kChunksPerTile  = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk  = BT_CHUNK_ELEMS / kSeg;
    constexpr int kCompactThreads = kWarps * 32;
    // warp roles
    constexpr int kFirstCopier   = kWarps;
    constexpr int kScanWarp      = kWarps + kCopiers;       // and kScanWarp + 1
    constexpr int kLoadWarp      = kWarps + kCopiers + 2;
    constexpr int kSegsPerCopier = kWarps / kCopiers;
    static_assert(kWarps % kCopiers == 0, "equal shares for the copier warps");
    static_assert(kSeg % 32 == 0 && kSeg <= 1024 && BT_CHUNK_ELEMS % kSeg == 0, "segments tile a chunk");
    static_assert(kTile % BT_CHUNK_ELEMS == 0, "a tile holds whole chunks");
    static_assert(kWarps <= 32, "one lane per warp count");
    // A scan warp makes tile i ready only in its turn for tile i + 2, after that tile has been counted, so
    // tiles i, i + 1 and i + 2 must hold slots at once: three stages are the minimum that cannot deadlock,
    // the fourth keeps the bulk copy of the next tile in flight.
    static_assert(kStages >= 4, "loading, compacting, awaiting its base, copying out");

    extern __shared__ __align__(128) unsigned char smem_raw[];
    U *const tiles = reinterpret_cast<U *>(smem_raw);

    __shared__ __align__(8) uint64_t s_full[kStages];      // the bulk copy has landed            (copy engine -> compactors)
    __shared__ __align__(8) uint64_t s_counted[kStages];   // every compactor posted its count    (compactors -> scan warp)
    __shared__ __align__(8) uint64_t s_ready[kStages];     // base and offsets are in shared      (scan warp -> copiers)
    __shared__ __align__(8) uint64_t s_empty[kStages];     // every copier is done with the slot  (copiers -> load warp)
    __shared__ uint64_t          s_base[kStages];          // exclusive base of the tile in the slot
    __shared__ uint32_t          s_cnt[kStages][kWarps];   // packed count of each segment
    __shared__ uint32_t          s_off[kStages][kWarps];   // exclusive offset of each segment in the tile
    __shared__ uint32_t          s_agg[kStages];           // packed count of the tile
    __shared__ __align__(16) unsigned char s_bits[kWarps][kSeg / 8];   // bitmap bytes of the segment a warp is compacting
    __shared__ volatile uint32_t s_abort;
    __shared__ volatile uint64_t s_tag;                    // this launch's tag once the first scan warp has it, else 0
    __shared__ volatile uint32_t s_met;                    // the grid has met: wave totals may be added to and read
    // Contributions to wave totals held back until then, and the total words they belong to.  This CTA's i-th tile
    // can be counted before the meeting is over only while i <= kStages (tile kStages + 1 needs the slot of tile 1,
    // whose base may need a total), so kStages + 1 slots, indexed by i modulo that, never collide.
    constexpr uint32_t kHeld = kStages + 1;
    __shared__ unsigned long long s_held[kHeld];
    __shared__ uint32_t          s_held_word[kHeld];
    __shared__ uint64_t          s_arena_c0;               // arena forms: the cursor as this launch found it

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    // broadcast from lane 0 so that the compiler knows the role branches below are warp-uniform
    const uint32_t warp    = __shfl_sync(kFull, tid >> 5, 0);
    const uint32_t G       = gridDim.x;
    const uint32_t cta     = blockIdx.x;
    const uint64_t wait_ns = p.c.wait_ns;
    // The first kDirect waves of a tensor take the counts of the waves before them straight from the descriptors, so
    // totals (and with them the zeroing and the meeting) are needed only by tensors of more waves than that; and
    // without totals the last tile's base of one tensor holds a count from every CTA: no meeting.
    bool meet = p.c.jobs > 1;
    for (uint32_t k = 0; k < p.c.jobs; ++k) meet = meet || p.job[k].tiles > kDirect * G;

    if (tid == 0) {
        // Read before the barrier below: the kernel's one update of the cursor follows the last tile's base,
        // which needs a publication from every CTA, and a CTA publishes only after this barrier.
        s_arena_c0 = p.c.arena_cursor ? *reinterpret_cast<const volatile uint64_t *>(p.c.arena_cursor) : 0;
        s_abort    = 0;
        s_tag      = 0;
        s_met      = 0;
        for (uint32_t k = 0; k < kHeld; ++k) s_held[k] = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&s_full[s], 1);
            mbar_init(&s_counted[s], kWarps);
            mbar_init(&s_ready[s], 1);
            mbar_init(&s_empty[s], kCopiers);
        }
        fence_proxy_async();
    }
    __syncthreads();

    if (warp == kLoadWarp) {
        // ------------------------------------------------------------ load warp (one lane)
        if (lane == 0) {
            bool     ok     = true;
            uint32_t issued = 0;
            Walk     w;
            walk_begin(w, p, cta, G);
            for (uint32_t it = 0; ok && w.valid; ++it, walk_next(w, p, cta, G)) {
                if (it >= static_cast<uint32_t>(kStages)) {
                    ok = mbar_wait(&s_empty[it % kStages], ((it / kStages) - 1) & 1u, &s_abort, wait_ns);
                    if (!ok) break;
                }
                // Start-up pacing: at most two bulk copies outstanding per SM while the ring fills for the first
                // time, as in steady state, where a copy is issued only as a slot frees.  Requesting the whole ring
                // at once puts 33 MB in front of every other memory operation of the launch's first microseconds.
                if (it >= 2u && it < static_cast<uint32_t>(kStages)) mbar_wait<false>(&s_full[(it - 2u) % kStages], 0, &s_abort, wait_ns);
                // bulk copy of the tile into its ring slot
                const uint32_t s     = it % kStages;
                const U *const src   = static_cast<const U *>(p.job[kJobs == 1 ? 0u : w.k].src);
                const uint64_t first = static_cast<uint64_t>(w.tile(G)) * kTile;
                const uint64_t left  = p.job[kJobs == 1 ? 0u : w.k].n - first;
                const uint32_t valid = left < static_cast<uint64_t>(kTile) ? static_cast<uint32_t>(left) : kTile;
                const uint32_t bytes = (valid * static_cast<uint32_t>(sizeof(U))) & ~15u;   // whole 16-byte units
                fence_proxy_async();                       // the copiers' and compactors' accesses to the slot come first
                mbar_arrive_expect_tx(&s_full[s], bytes);  // bytes == 0 simply completes the phase
                if (bytes) bulk_load(tiles + static_cast<size_t>(s) * kTile, src + first, bytes, &s_full[s]);
                issued = it + 1;
            }
            // This lane stays until every bulk copy it issued has landed, whatever the other warps do (they may
            // leave early once a bounded wait has run out somewhere): the CTA never retires with a copy into its
            // shared memory in flight.  Only the last kStages copies can still be pending; each wait is bounded.
            for (uint32_t it = issued > static_cast<uint32_t>(kStages) ? issued - kStages : 0; it < issued; ++it)
                mbar_wait<false>(&s_full[it % kStages], (it / kStages) & 1u, &s_abort, 20000000ull);
        }
        return;
    }

    if (warp == kScanWarp || warp == kScanWarp + 1) {
        // ------------------------------------------------------------ scan warps
        // Two warps share the scan: warp q takes this CTA's tiles q, q + 2, q + 4, ... (counted in the order the
        // CTA takes them).  A warp's turn for tile i is
        //   (a) wait until the compactors have counted tile i, publish the count,
        //   (c) finish tile i - 2 (its own previous tile) from the loads of its previous turn and hand it
        //       to the copiers,
        //   (b) wait until tile i + 1 is counted -- about one tile later, when every CTA has published
        //       the wave of tile i -- and issue, in ONE batch of independent loads, the reads of the descriptors
        //       of that wave and of the totals of the two waves before it.
        // The loads of (b) are used a whole tile later, in (c) of the next turn, so the round trip to L2
        // (1.3 us under load, longer than one tile) never stalls a turn for long: a turn has two tiles' time.
        const uint32_t  q          = warp - kScanWarp;
        uint64_t *const wave_total = p.c.ws_total;
        uint64_t *const desc       = p.c.ws_desc;
        bool            failed     = false;

        // number of tiles this CTA takes
        uint32_t my_tiles = 0;
        for (uint32_t k = 0; k < p.c.jobs; ++k) {
            const uint32_t rot = p.job[k].rot, t = p.job[k].tiles;
            const uint32_t v   = cta >= rot ? cta - rot : cta + G - rot;
            if (v < t) my_tiles += (t - v + G - 1) / G;
        }
        const uint32_t last_i = my_tiles - 1;       // every CTA has a tile: the grid is no larger than the tile count

        // The tag of this launch.  One warp reads the sequence number; it changes only once every CTA has arrived
        // at the meeting, which a CTA does after this read.
        uint64_t tag = 0;
        if (q == 0) {
            if (lane == 0) {
                const uint64_t seq = ld_relaxed_u64(p.c.ws_header + kHdrSeq);
                tag                = mix64(p.c.call_tag + seq * 0x9E3779B97F4A7C15ull) | 1ull;
                s_tag              = tag;
            }
        } else if (lane == 0) {
            tag = wait_tag(&s_tag, &s_abort, wait_ns);
        }
        tag = __shfl_sync(kFull, tag, 0);
        if (tag == 0) {
            if (lane == 0) raise_timeout(p, &s_abort, 0);
            return;
        }
        const uint64_t tag_w0 = tag & 0xFFFFFFFF00000000ull, tag_w1 = tag << 32;
        auto valid = [&](const uint64_t w0, const uint64_t w1) {
            return ((w0 ^ tag_w0) >> 32) == 0 && ((w1 ^ tag_w1) >> 32) == 0 && static_cast<uint32_t>(w0) == static_cast<uint32_t>(w1);
        };

        // Wave totals are sums made by reductions, so their words must be zero first, and the grid must have met
        // after the zeroing before anyone adds or reads.  That meeting is a copier warp's job (below): until it is
        // over, a scan warp parks its contribution in shared memory and goes on -- the tagged descriptors need no
        // clearing, so counts are published and read without waiting for the meeting.
        auto add_to_total = [&](const uint32_t i, const uint32_t word_index, const unsigned long long contribution) {   // lane 0 only
            if (s_met) {
                red_add_u64(wave_total + word_index, contribution);
                return;
            }
            const uint32_t slot = i % kHeld;
            s_held_word[slot]   = word_index;
            __threadfence_block();
            atomicExch(&s_held[slot], contribution);
            __threadfence_block();
            if (s_met) {
                // the meeting ended meanwhile: whoever takes the parked value out adds it
                const unsigned long long v = atomicExch(&s_held[slot], 0ull);
                if (v) red_add_u64(wave_total + word_index, v);
            }
        };

        // d0[k], d1[k], lane l <-> descriptor of virtual CTA l + 32k of the wave of this warp's previous tile;
        // w1, w2: total words of the one and the two waves before it (0: not read yet)
        uint64_t d0[kMaxWindows], d1[kMaxWindows], w1 = 0, w2 = 0;
#pragma unroll
        for (int k = 0; k < kMaxWindows; ++k) d0[k] = tag_w0, d1[k] = tag_w1;

        Walk cur;                                   // this warp's tile of the turn
        walk_begin(cur, p, cta, G);
        if (q == 1 && cur.valid) walk_next(cur, p, cta, G);
        uint32_t pk = 0, pj = 0, pv = 0;            // this warp's previous tile: tensor, wave, virtual CTA
        uint64_t p_direct = 0;                      //   and, for a wave < kDirect, the counts of all the waves before it
        uint64_t waves_before = 0;                  // sum of the counts of the waves before the previous tile (of its tensor)

        for (uint32_t i = q; !failed && i <= last_i + 2; i += 2) {
            const bool has = i <= last_i;
            if (has) {
                // ---- (a)
                const uint32_t s = i % kStages;
                if (!mbar_wait(&s_counted[s], (i / kStages) & 1u, &s_abort, wait_ns)) {
                    failed = true;
                    break;
                }
                const uint32_t c   = lane < kWarps ? s_cnt[s][lane] : 0u;
                uint32_t       inc = c;
#pragma unroll
                for (int o = 1; o < kWarps; o <<= 1) {
                    const uint32_t u = __shfl_up_sync(kFull, inc, o);
                    if (lane >= static_cast<uint32_t>(o)) inc += u;
                }
                const uint32_t agg = __shfl_sync(kFull, inc, kWarps - 1);
                if (lane == 0) {
                    st_relaxed_2xu64(desc + 2 * (static_cast<uint64_t>(p.job[kJobs == 1 ? 0u : cur.k].desc0) + cur.tile(G)), tag_w0 | agg, tag_w1 | agg);
                    s_agg[s] = agg;
                }
                if (lane < kWarps) s_off[s][lane] = inc - c;
                if (cur.tiles > kDirect * G && lane == 0) add_to_total(i, p.job[kJobs == 1 ? 0u : cur.k].total0 + cur.j, (1ull << kCountShift) + agg);
            }
            if (i >= 2) {
                // ---- (c): this warp's previous tile, (pk, pj, pv)
                const CompressJob &jb    = p.job[kJobs == 1 ? 0u : pk];
                uint32_t           polls = 0;
                uint64_t           t0    = 0;
                for (;;) {
                    bool missing = pj >= kDirect && ((w1 >> kCountShift) != G || (w2 >> kCountShift) != G);
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k) missing |= !valid(d0[k], d1[k]);
                    if (!__any_sync(kFull, missing)) break;
                    __nanosleep(100);
                    if ((++polls & 255u) == 0 || wait_ns < 1000000ull) {
                        if (t0 == 0) t0 = now_ns();
                        if (__any_sync(kFull, (now_ns() - t0 > wait_ns) || ld_relaxed_u64(p.c.ws_header + kHdrAbort) == tag)) {
                            failed = true;
                            break;
                        }
                    }
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k)
                        if (!valid(d0[k], d1[k]))
                            ld_relaxed_2xu64(desc + 2 * (static_cast<uint64_t>(jb.desc0) + static_cast<uint64_t>(pj) * G + lane + 32u * k), d0[k], d1[k]);
                    if (s_met && pj >= kDirect) {        // a total counts only once every CTA has zeroed its share
                        if ((w1 >> kCountShift) != G) w1 = ld_relaxed_u64(wave_total + jb.total0 + (pj - 1));
                        if ((w2 >> kCountShift) != G) w2 = ld_relaxed_u64(wave_total + jb.total0 + (pj - 2));
                    }
                }
                if (failed) break;
                uint64_t part = 0;
#pragma unroll
                for (int k = 0; k < kMaxWindows; ++k) part += static_cast<uint32_t>(d0[k]);
                // the waves in front of the tile: those in front of this warp's tile before it, if that was wave
                // pj - 2 of the same tensor, and the one or two waves read for this turn
                // (a wave < kDirect brings the sum with it; the tile of this warp before a wave >= kDirect is of the same tensor)
                waves_before = pj < kDirect ? p_direct : waves_before + (w1 & ((1ull << kCountShift) - 1)) + (w2 & ((1ull << kCountShift) - 1));
                const uint64_t base = waves_before + warp_sum_u64(part);
                const uint32_t ps   = (i - 2) % kStages;
                const uint64_t pt   = pv + static_cast<uint64_t>(pj) * G;
                // exclusive count in front of each chunk of that tile
                if (lane < kWarps && (lane % kWarpsPerChunk) == 0) {
                    const uint64_t ch = pt * kChunksPerTile + lane / kWarpsPerChunk;
                    if (ch < (jb.n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS) jb.prefix[ch] = base + s_off[ps][lane];
                }
                if (pt == jb.tiles - 1 && lane == 0) {
                    const uint64_t nnz = base + s_agg[ps];
                    *jb.nnz_out        = nnz;
                    __threadfence();
                    const bool aborted  = ld_relaxed_u64(p.c.ws_header + kHdrAbort) == tag;
                    uint64_t   capacity = jb.capacity;
                    if (p.c.arena_cursor) {
                        // arena form: the room left behind the cursor; the cursor moves only when everything fitted
                        const uint64_t c0 = s_arena_c0;
                        capacity          = c0 <= p.c.arena_bytes ? (p.c.arena_bytes - c0) / sizeof(Stored<CAST, U>) : 0;
                        if (!aborted && nnz <= capacity) {
                            *p.c.values_offset_out = c0;
                            *p.c.arena_cursor      = c0 + ((nnz * sizeof(Stored<CAST, U>) + 15) & ~15ull);
                        }
                    }
                    // without a meeting: every CTA has published its count by now, so every CTA has read the sequence
                    // number, and the next launch on this workspace gets another tag
                    if (!meet) red_add_u64(p.c.ws_header + kHdrSeq, 1ull);
                    if (jb.dev_status) {
                        *reinterpret_cast<volatile int32_t *>(jb.dev_status) = aborted ? BT_ERR_TIMEOUT : (nnz > capacity ? BT_ERR_CAPACITY : BT_OK);
                        // a CTA that gives up from now on stores its BT_ERR_TIMEOUT after this word; one that gave
                        // up just before is seen here
                        __threadfence();
                        if (!aborted && ld_relaxed_u64(p.c.ws_header + kHdrAbort) == tag)
                            *reinterpret_cast<volatile int32_t *>(jb.dev_status) = BT_ERR_TIMEOUT;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    s_base[ps] = base;
                    mbar_arrive(&s_ready[ps]);                       // the copiers may take the tile
                }
            }
            if (has) {
                // ---- (b): a tile later (when the other scan warp's next tile is counted, if there is one)
                if (i + 1 > last_i) {
                    // This CTA's last tile: no next tile to wait for.  A short pause gives the other counts of the
                    // wave time to land, so that the reads below usually succeed at once instead of costing a second
                    // round trip.
                    __nanosleep(300);
                } else if (!mbar_wait(&s_counted[(i + 1) % kStages], ((i + 1) / kStages) & 1u, &s_abort, wait_ns)) {
                    failed = true;
                    break;
                }
                const uint64_t d_first = static_cast<uint64_t>(p.job[kJobs == 1 ? 0u : cur.k].desc0) + static_cast<uint64_t>(cur.j) * G;
#pragma unroll
                for (int k = 0; k < kMaxWindows; ++k) {
                    const uint32_t b = lane + 32u * k;
                    if (b < cur.v) ld_relaxed_2xu64(desc + 2 * (d_first + b), d0[k], d1[k]);
                    else d0[k] = tag_w0, d1[k] = tag_w1;             // not in front of this CTA: a valid count of 0
                }
                const bool met = s_met != 0;
                w1 = (cur.j >= kDirect && met) ? ld_relaxed_u64(wave_total + p.job[kJobs == 1 ? 0u : cur.k].total0 + (cur.j - 1)) : 0ull;
                w2 = (cur.j >= kDirect && met) ? ld_relaxed_u64(wave_total + p.job[kJobs == 1 ? 0u : cur.k].total0 + (cur.j - 2)) : 0ull;
                p_direct = 0;
                if (cur.j > 0 && cur.j < kDirect) {
                    // one of a tensor's first waves: the counts of all tiles of the waves before it, read here and now
                    // (they were published a tile ago and more; what is not there yet is asked for again)
                    const uint64_t t_first = static_cast<uint64_t>(p.job[kJobs == 1 ? 0u : cur.k].desc0);
                    uint64_t       sum     = 0;
                    for (uint32_t jj = 0; jj < cur.j && !failed; ++jj) {
                        bool     got[kMaxWindows];
#pragma unroll
                        for (int k = 0; k < kMaxWindows; ++k) got[k] = lane + 32u * k >= G;
                        uint32_t tries = 0;
                        uint64_t t_start = 0;
                        for (;;) {
                            bool miss = false;
#pragma unroll
                            for (int k = 0; k < kMaxWindows; ++k) {
                                if (!got[k]) {
                                    uint64_t x0, x1;
                                    ld_relaxed_2xu64(desc + 2 * (t_first + static_cast<uint64_t>(jj) * G + lane + 32u * k), x0, x1);
                                    if (valid(x0, x1)) got[k] = true, sum += static_cast<uint32_t>(x0);
                                    else miss = true;
                                }
                            }
                            if (!__any_sync(kFull, miss)) break;
                            __nanosleep(100);
                            if ((++tries & 255u) == 0 || wait_ns < 1000000ull) {
                                if (t_start == 0) t_start = now_ns();
                                if (__any_sync(kFull, (now_ns() - t_start > wait_ns) || ld_relaxed_u64(p.c.ws_header + kHdrAbort) == tag)) {
                                    failed = true;
                                    break;
                                }
                            }
                        }
                    }
                    p_direct = warp_sum_u64(sum);
                }
                pk = cur.k, pj = cur.j, pv = cur.v;
                walk_next(cur, p, cta, G);
                if (cur.valid) walk_next(cur, p, cta, G);
            }
        }
        if (failed && lane == 0) raise_timeout(p, &s_abort, tag);
        return;
    }

    if (warp >= kFirstCopier) {
        // ------------------------------------------------------------ copier warps
        const uint32_t copier = warp - kFirstCopier;
        using V               = Stored<CAST, U>;
        if (copier == kCopiers - 1 && meet) {
            // The meeting: this warp has nothing to copy for the first microseconds.  It zeroes this CTA's share of
            // the wave totals and writes the launch's tag into this CTA's arrival word.  CTA 0 waits (bounded) until
            // all G arrival words carry the tag -- every CTA has then zeroed its share, and has read the sequence
            // number, which CTA 0 now moves on -- and writes the tag into the "go" word; the others wait for that
            // word (one poller and one word per CTA: every CTA polling every arrival word makes a hot spot in L2
            // that takes microseconds to cool).  Then the warp adds what the scan warps have parked meanwhile.
            uint64_t *const wave_total = p.c.ws_total;
            uint64_t *const arrive     = p.c.ws_header + kWsArriveWord;
            uint64_t        tag        = 0;
            if (lane == 0) tag = wait_tag(&s_tag, &s_abort, wait_ns);
            tag     = __shfl_sync(kFull, tag, 0);
            bool ok = tag != 0;
            if (ok) {
                for (uint32_t i = cta * 32 + lane; i < p.c.ws_totals; i += G * 32) wave_total[i] = 0;
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    st_release_u64(arrive + cta, tag);
                }
                const uint64_t t0 = now_ns();
                if (cta == 0) {
                    bool here[kMaxWindows];
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k) here[k] = lane + 32u * k >= G;
                    for (;;) {
                        bool missing = false;
#pragma unroll
                        for (int k = 0; k < kMaxWindows; ++k) {
                            if (!here[k]) here[k] = ld_acquire_u64(arrive + lane + 32u * k) == tag;
                            missing |= !here[k];
                        }
                        if (!__any_sync(kFull, missing)) break;
                        if (__any_sync(kFull, s_abort != 0 || now_ns() - t0 > wait_ns)) {
                            ok = false;
                            break;
                        }
                    }
                    if (ok && lane == 0) {
                        __threadfence();
                        st_release_u64(p.c.ws_header + kHdrGo, tag);
                        red_add_u64(p.c.ws_header + kHdrSeq, 1ull);      // every CTA has read it: the next launch gets another tag
                    }
                } else {
                    if (lane == 0) {
                        while (ld_acquire_u64(p.c.ws_header + kHdrGo) != tag) {
                            if (s_abort != 0 || now_ns() - t0 > wait_ns) {
                                ok = false;
                                break;
                            }
                            __nanosleep(64);
                        }
                    }
                    ok = __shfl_sync(kFull, ok ? 1 : 0, 0) != 0;
                }
            }
            if (lane == 0) {
                if (ok) {
                    __threadfence();
                    s_met = 1;
                    __threadfence_block();
                    for (uint32_t k = 0; k < kHeld; ++k) {
                        const unsigned long long v = atomicExch(&s_held[k], 0ull);
                        if (v) red_add_u64(wave_total + s_held_word[k], v);
                    }
                } else {
                    raise_timeout(p, &s_abort, tag);
                }
            }
            __syncwarp();
        }
        Walk w;
        walk_begin(w, p, cta, G);
        for (uint32_t it = 0; w.valid; ++it, walk_next(w, p, cta, G)) {
            const uint32_t s = it % kStages;
            if (!mbar_wait(&s_ready[s], (it / kStages) & 1u, &s_abort, wait_ns)) break;
            V       *vals     = static_cast<V *>(p.job[kJobs == 1 ? 0u : w.k].values);
            uint64_t capacity = p.job[kJobs == 1 ? 0u : w.k].capacity;
            if (p.c.arena_cursor) {
                const uint64_t c0 = s_arena_c0;
                vals              = reinterpret_cast<V *>(static_cast<unsigned char *>(p.job[kJobs == 1 ? 0u : w.k].values) + c0);
                capacity          = c0 <= p.c.arena_bytes ? (p.c.arena_bytes - c0) / sizeof(V) : 0;
            }
            const uint64_t base = s_base[s];
#pragma unroll
            for (int qq = 0; qq < kSegsPerCopier; ++qq) {
                const uint32_t seg  = copier * kSegsPerCopier + qq;
                const U *const pseg = tiles + static_cast<size_t>(s) * kTile + seg * kSeg;
                const uint32_t cnt  = s_cnt[s][seg];
                const uint64_t dst  = base + s_off[s][seg];
                if (dst + cnt <= capacity)
                    copy_out_piece<U, CAST, 1, false>(pseg, cnt, vals + dst, 0, 0, lane);
                else
                    copy_out_piece<U, CAST, 1, true>(pseg, cnt, vals + dst, dst < capacity ? capacity - dst : 0, 0, lane);
            }
            __syncwarp();
            asm volatile("" ::: "memory");        // the copy-out stays above the release of the slot
            if (lane == 0) mbar_arrive(&s_empty[s]);
        }
        return;
    }

    // ---------------------------------------------------------------- compactor warps
    const uint32_t bm_addr = smem_addr(&s_bits[warp][0]);
    Walk           w;
    walk_begin(w, p, cta, G);
    for (uint32_t it = 0; w.valid; ++it, walk_next(w, p, cta, G)) {
        const CompressJob &jb    = p.job[kJobs == 1 ? 0u : w.k];
        const uint64_t     n     = jb.n;
        const uint64_t     t64   = w.tile(G);
        const uint32_t     s     = it % kStages;
        U *const           tile  = tiles + static_cast<size_t>(s) * kTile;
        const uint64_t     first = t64 * kTile;
        if (!mbar_wait(&s_full[s], (it / kStages) & 1u, &s_abort, wait_ns)) {
            if (lane == 0) raise_timeout(p, &s_abort, s_tag);
            break;
        }
        if (n - first < static_cast<uint64_t>(kTile)) {
            // ragged last tile: fetch what the 16-byte granular bulk copy left out, zero the rest
            const U *const src     = static_cast<const U *>(jb.src);
            const uint32_t have    = static_cast<uint32_t>(n - first);
            const uint32_t by_bulk = ((have * static_cast<uint32_t>(sizeof(U))) & ~15u) / sizeof(U);
            for (uint32_t e = by_bulk + tid; e < static_cast<uint32_t>(kTile); e += kCompactThreads)
                tile[e] = (e < have) ? src[first + e] : U(0);
            asm volatile("bar.sync %0, %1;" ::"n"(kBarWorkers), "n"(kCompactThreads) : "memory");
        }

        // ---- this warp's segment: into registers, counted, packed in place
        const uint64_t e0     = first + warp * kSeg;                 // first element of the segment
        uint32_t       yvalid = 0;
        U             *y      = nullptr;
        if constexpr (WRITE_Y) {
            y      = static_cast<U *>(jb.y) + e0;
            yvalid = e0 + kSeg <= n ? static_cast<uint32_t>(kSeg) : (e0 < n ? static_cast<uint32_t>(n - e0) : 0u);
        }
        const uint32_t seg_addr = smem_addr(tile + warp * kSeg);
        uint4          q[S::kSteps];
        uint32_t       m[S::kSteps];
        if (!WRITE_Y || yvalid == static_cast<uint32_t>(kSeg))   // all but a ragged last tile: no bounds checks on y
            segment_load<U, FUSED, WRITE_Y, false, kSeg>(seg_addr, lane, q, m, y, yvalid, p.c.tau);
        else
            segment_load<U, FUSED, WRITE_Y, true, kSeg>(seg_addr, lane, q, m, y, yvalid, p.c.tau);
        uint32_t       inc[S::kBatches], packed[S::kBatches];
        const uint32_t cnt = segment_scan<U, kSeg>(m, inc, packed, lane);
        // the whole segment is in registers: the packed values may overwrite it from its start
        segment_store<U, kSeg>(q, inc, packed, seg_addr);
        __syncwarp();
        if (lane == 0) {
            s_cnt[s][warp] = cnt;
            mbar_arrive(&s_counted[s]);                   // hand the count to the scan warp
        }
        // the bitmap, behind the count: nobody waits for it
        uint32_t word[S::kWordsPerLane];
        segment_bitmap<U, kSeg>(m, bm_addr, lane, word);
        if (lane * S::kWordsPerLane < static_cast<uint32_t>(S::kWords)) {
            const uint64_t wd = t64 * (kTile / 32) + warp * S::kWords + lane * S::kWordsPerLane;
#pragma unroll
            for (int k = 0; k < S::kWordsPerLane; ++k)
                if (wd + k < ((n + 31) >> 5)) jb.bitmap[wd + k] = word[k];
        }
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

// The calling thread's limit on the CTAs of one compress launch (0: none).  A cooperative launch needs all its
// CTAs resident at once and a CTA of this kernel fills an SM, so two launches of more than half the SMs each run
// one after the other even on different streams; a caller that keeps several launches in flight gives each a
// share of the SMs.
thread_local uint32_t t_max_ctas = 0;

// The bound of the kernels' waits; only a test build can change it.
std::atomic<uint64_t> g_wait_ns{kDefaultWaitNs};

// Launch shape of one kernel instantiation on one device: the opt-in shared
// memory size is set and the number of co-resident CTAs is looked up once.
struct LaunchShape {
    std::mutex lock;
    int        grid_of_device[64] = {};
    template <typename Kernel>
    cudaError_t max_grid(Kernel kernel, int threads, size_t smem, int &grid)
    {
        int         dev = 0;
        cudaError_t e   = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> g(lock);
        if (grid_of_device[dev] == 0) {
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
            if (e != cudaSuccess) return e;
            int sms = 0, per_sm = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return e;
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
            if (e != cudaSuccess) return e;
            if (per_sm < 1 || sms < 1) return cudaErrorLaunchOutOfResources;
            grid_of_device[dev] = sms * per_sm;
        }
        grid = grid_of_device[dev];
        return cudaSuccess;
    }
};

template <typename U, int FUSED, bool WRITE_Y, int CAST, int kJobs, int kWarps, int kSeg, int kStages, int kCopiers>
cudaError_t launch_shaped(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, cudaStream_t stream)
{
    constexpr int    kTile    = kWarps * kSeg;
    constexpr int    kThreads = (kWarps + kCopiers + 3) * 32;
    constexpr size_t kSmem    = static_cast<size_t>(kStages) * kTile * sizeof(U);
    static LaunchShape shape;   // one per instantiation
    auto kernel = compress_kernel<U, FUSED, WRITE_Y, CAST, kJobs, kWarps, kSeg, kStages, kCopiers>;
    if (count == 0 || count > static_cast<uint32_t>(kJobs)) return cudaErrorInvalidValue;

    CompressParams<kJobs> p;
    p.c             = c;
    uint64_t tiles  = 0;
    for (uint32_t k = 0; k < count; ++k) {
        p.job[k]            = jobs[k];
        const uint64_t t    = (jobs[k].n + kTile - 1) / kTile;
        if (t == 0 || t > 0xFFFFFFFFull) return cudaErrorInvalidValue;
        p.job[k].tiles      = static_cast<uint32_t>(t);
        tiles += t;
    }
    if (tiles > 0xFFFFFFFFull) return cudaErrorInvalidValue;
    for (uint32_t k = count; k < static_cast<uint32_t>(kJobs); ++k) p.job[k] = CompressJob{};

    int         max_grid = 0;
    cudaError_t e        = shape.max_grid(kernel, kThreads, kSmem, max_grid);
    if (e != cudaSuccess) return e;
    if (max_grid > static_cast<int>(kMaxGrid)) max_grid = kMaxGrid;
    if (t_max_ctas != 0 && static_cast<uint32_t>(max_grid) > t_max_ctas) max_grid = static_cast<int>(t_max_ctas);
    const uint32_t grid = tiles < static_cast<uint64_t>(max_grid) ? static_cast<uint32_t>(tiles) : static_cast<uint32_t>(max_grid);

    // the deal: tile t of tensor k goes to CTA (rot_k + t) mod grid; wave totals and descriptors tensor after tensor
    uint64_t dealt = 0, totals = 0;
    for (uint32_t k = 0; k < count; ++k) {
        p.job[k].rot    = static_cast<uint32_t>(dealt % grid);
        p.job[k].total0 = static_cast<uint32_t>(totals);
        p.job[k].desc0  = static_cast<uint32_t>(dealt);
        dealt += p.job[k].tiles;
        totals += (p.job[k].tiles + grid - 1) / grid;
    }
    p.c.jobs      = count;
    p.c.ws_totals = static_cast<uint32_t>((totals + 1) & ~1ull);     // an even number of total words keeps the descriptors 16-byte aligned
    p.c.ws_header = static_cast<uint64_t *>(workspace);
    p.c.ws_total  = reinterpret_cast<uint64_t *>(static_cast<unsigned char *>(workspace) + kWsHeaderBytes);
    p.c.ws_desc   = p.c.ws_total + p.c.ws_totals;
    p.c.call_tag  = next_call_tag();
    p.c.wait_ns   = g_wait_ns.load(std::memory_order_relaxed);
    // cooperative launch: the runtime guarantees that all `grid` CTAs are resident together
    void *params[] = {&p};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(kThreads), params, kSmem, stream);
}

template <typename U, int FUSED, bool WRITE_Y, int CAST = 0>
cudaError_t launch_typed(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, cudaStream_t stream)
{
    // One CTA per SM, the ring takes nearly all of its shared memory.
    //   8-byte elements: 8 compactor warps x 512 elements (32 KB tiles), 8 copiers, 7 stages;
    //   4-byte elements: 8 compactor warps x 1024 elements (32 KB tiles), 8 copiers, 7 stages;
    //   2-byte elements: 16 compactor warps x 1024 elements (32 KB tiles), 8 copiers, 6 stages.
    // Batches (plain and ReLU forms only) run the instantiation with room for kMaxBatch tensors.
    constexpr bool kBatchable = CAST == 0 && FUSED < kFusedRelu6;
    if constexpr (kBatchable) {
        if (count > 1) {
            if constexpr (sizeof(U) == 8) return launch_shaped<U, FUSED, WRITE_Y, CAST, kMaxBatch, 8, 512, 7, 8>(c, jobs, count, workspace, stream);
            else if constexpr (sizeof(U) == 4) return launch_shaped<U, FUSED, WRITE_Y, CAST, kMaxBatch, 8, 1024, 7, 8>(c, jobs, count, workspace, stream);
            else return launch_shaped<U, FUSED, WRITE_Y, CAST, kMaxBatch, 16, 1024, 6, 8>(c, jobs, count, workspace, stream);
        }
    }
    if (count != 1) return cudaErrorInvalidValue;
    if constexpr (sizeof(U) == 8) return launch_shaped<U, FUSED, WRITE_Y, CAST, 1, 8, 512, 7, 8>(c, jobs, count, workspace, stream);
    else if constexpr (sizeof(U) == 4) return launch_shaped<U, FUSED, WRITE_Y, CAST, 1, 8, 1024, 7, 8>(c, jobs, count, workspace, stream);
    else return launch_shaped<U, FUSED, WRITE_Y, CAST, 1, 16, 1024, 6, 8>(c, jobs, count, workspace, stream);
}

}  // namespace

uint32_t set_compress_max_ctas(uint32_t max_ctas)
{
    const uint32_t before = t_max_ctas;
    t_max_ctas            = max_ctas;
    return before;
}

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
