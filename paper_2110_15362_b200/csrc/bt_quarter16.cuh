// The quarter-chunk walk over a stash of 2-byte values, shared by the restore (bt_decompress.cu) and the ReLU6
// backward (bt_relu6_bwd.cu).
//
// The generic kernels gather every stashed value with one global load and a 64-bit address computation per
// element, which makes a 2-byte element cost as many instructions as a 4-byte one.  Here a warp first brings its
// quarter's packed run (at most 1024 values) into shared memory with one bulk copy -- the run starts wherever its
// rank puts it: the 16-byte vectors that cover it are copied whole, the last one element by element so that
// nothing behind the caller's values is read -- and the gather reads shared memory: a test of the element's bit,
// a 2-byte shared load, a select, a predicated 32-bit add.
#pragma once

#include "bt_internal.cuh"

namespace bt {
namespace q16 {

constexpr uint32_t kFull = 0xFFFFFFFFu;

__device__ __forceinline__ uint4 ldg_vec_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Four consecutive elements under the four low bits of `bits`: for every set bit the next 2-byte value at shared
// address `a` (which moves on), kFill for a clear bit; packed two to a word.
template <uint32_t kFill = 0>
__device__ __forceinline__ uint2 expand4_u16(uint32_t a, const uint32_t bits)
{
    uint2 r;
#define BT_PAIR(OUT, B0, B1)                                                                                         \
    "and.b32 t, %3, " #B0 ";\n\tsetp.ne.u32 p, t, 0;\n\tld.shared.u16 lo, [%2];\n\tselp.b32 lo, lo, %4, p;\n\t@p add.u32 %2, %2, 2;\n\t" \
    "and.b32 t, %3, " #B1 ";\n\tsetp.ne.u32 p, t, 0;\n\tld.shared.u16 hi, [%2];\n\tselp.b32 hi, hi, %4, p;\n\t@p add.u32 %2, %2, 2;\n\t" \
    "prmt.b32 " OUT ", lo, hi, 0x5410;\n\t"
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 t, lo, hi;\n\t" BT_PAIR("%0", 1, 2) BT_PAIR("%1", 4, 8) "}" : "=r"(r.x), "=r"(r.y), "+r"(a) : "r"(bits), "n"(kFill));
#undef BT_PAIR
    return r;
}

// Bounded wait for a warp's own bulk copy (phase 0 of its mbarrier): false if it has not landed within the limit.
constexpr uint64_t kLandLimitNs = 2000000000ull, kLandLastNs = 20000000ull;
__device__ __forceinline__ bool landed(uint64_t *bar, const uint64_t limit_ns)
{
    uint64_t t0 = 0;
    for (uint32_t probes = 1; !mbar_try_wait(bar, 0); ++probes) {
        if ((probes & 63u) == 0) {
            uint64_t now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) return false;
        }
    }
    return true;
}

// What a warp knows about its quarter once the run is staged.
struct Quarter {
    uint32_t word;      // lane l: bitmap word l of the quarter
    uint32_t excl;      // lane l: set bits of the quarter in front of word l
    uint32_t run;       // shared address of the quarter's first value
    uint64_t e0;        // index of the quarter's first element
    bool     whole;     // all 1024 elements exist
};

// Reads the chunk's bitmap words and prefix entry, ranks the quarter's words and stages its packed run.  False if
// this warp has no quarter.  `block`: index of the CTA among those that work on the tensor.
template <int kWarps>
__device__ __forceinline__ bool stage_quarter(const uint32_t *__restrict__ bitmap, const uint16_t *values,
                                              const uint64_t *__restrict__ values_offset, const uint64_t *__restrict__ prefix,
                                              const uint64_t n, const uint64_t block, Quarter &qt)
{
    // a quarter's run (at most 1024 values) behind up to 14 bytes of its first vector, whole vectors
    __shared__ __align__(16) unsigned char s_run[kWarps][2048 + 32];
    __shared__ __align__(8) uint64_t       s_landed[kWarps];   // the warp's bulk copy has landed

    const uint32_t lane        = threadIdx.x & 31u;
    const uint32_t wic         = threadIdx.x >> 5;
    const uint64_t warp_global = block * kWarps + wic;
    const uint64_t quarters    = (n + 1023) >> 10;
    if (warp_global >= quarters) return false;
    if (lane == 0) {
        mbar_init(&s_landed[wic], 1);
        fence_proxy_async();
    }
    __syncwarp();

    const uint64_t chunk       = warp_global >> 2;
    const uint32_t q           = static_cast<uint32_t>(warp_global & 3u);
    const uint64_t words_total = (n + 31) >> 5;
    const uint64_t w0          = chunk * 128 + 4 * lane;   // this lane's four words of the chunk

    // the chunk's 128 words (zero past the end of the bitmap) and its prefix entry: independent loads
    const uint4    c4         = load_words4(bitmap, w0, words_total);
    const uint64_t chunk_base = prefix[chunk];
    if (values_offset) values = reinterpret_cast<const uint16_t *>(reinterpret_cast<const unsigned char *>(values) + *values_offset);

    // non-zeros of the chunk in front of this quarter
    uint32_t before = lane < 8 * q ? __popc(c4.x) + __popc(c4.y) + __popc(c4.z) + __popc(c4.w) : 0u;
    before          = __reduce_add_sync(kFull, before);
    // lane l takes word l of its own quarter: component l & 3 of lane 8q + (l >> 2)
    const int      from_lane = 8 * q + (lane >> 2);
    const uint32_t x0 = __shfl_sync(kFull, c4.x, from_lane), x1 = __shfl_sync(kFull, c4.y, from_lane);
    const uint32_t x2 = __shfl_sync(kFull, c4.z, from_lane), x3 = __shfl_sync(kFull, c4.w, from_lane);
    const uint32_t word = (lane & 2u) ? ((lane & 1u) ? x3 : x2) : ((lane & 1u) ? x1 : x0);
    uint32_t       incl = __popc(word);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(kFull, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += u;
    }
    const uint32_t excl = incl - __popc(word);
    const uint32_t cnt  = __shfl_sync(kFull, incl, 31);      // values of this quarter

    // ---- the run into shared memory: one bulk copy per warp.  The copy engine writes shared memory by itself;
    // brought in through registers (16-byte loads, then 16-byte shared stores) the same bytes pass the L1 data pipe
    // twice, and that pipe is what bounds these kernels (85 % busy): 0.129 -> 0.113 ms for the restore of the
    // 392 MiB tensor.  The copy covers the whole 16-byte vectors of the run; the elements of the last, partial
    // vector are fetched one by one so that nothing behind the caller's values is read.
    const uint16_t *const src   = values + (chunk_base + before);
    const uint32_t        shift = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src) & 15u);         // bytes
    const uint32_t        bytes = shift + 2u * cnt;                                                      // of the staging area in use
    const uint32_t        stage = smem_addr(&s_run[wic][0]);
    if (cnt) {
        const uint4 *const gv   = reinterpret_cast<const uint4 *>(reinterpret_cast<const unsigned char *>(src) - shift);
        const uint32_t     full = bytes >> 4;                                                            // whole vectors
        if (full && lane == 0) {
            mbar_arrive_expect_tx(&s_landed[wic], 16u * full);
            bulk_load(&s_run[wic][0], gv, 16u * full, &s_landed[wic]);
        }
        const uint32_t tail0 = full * 16u > shift ? full * 16u : shift;
        for (uint32_t b = tail0 + 2u * lane; b < bytes; b += 64u)
            s_run[wic][b] = reinterpret_cast<const unsigned char *>(gv)[b], s_run[wic][b + 1] = reinterpret_cast<const unsigned char *>(gv)[b + 1];
        // Not seen so far: the copy engine has not delivered within two seconds.  The calls built on this have no
        // status word; the warp gives the copy a last, short time (so that the CTA does not retire with a copy into
        // its shared memory in flight) and leaves its quarter of the output unwritten.
        if (full && !landed(&s_landed[wic], kLandLimitNs)) {
            landed(&s_landed[wic], kLandLastNs);
            return false;
        }
    }
    __syncwarp();
    qt.word  = word;
    qt.excl  = excl;
    qt.run   = stage + shift;
    qt.e0    = warp_global << 10;
    qt.whole = qt.e0 + 1024 <= n;
    return true;
}

// Step k (0..7) of the expansion: the lane's four consecutive elements e0 + 128k + 4 lane .. + 3, packed two to a
// word, kFill (+0 unless the caller asks otherwise) where the bit is clear; `bits` receives the four bits (low nibble).  (With 8 elements per lane the 32
// lanes of one shared load reach over 256 bytes of the run and every load takes two passes: 0.131 ms instead of
// 0.126 on 205 M elements; with 2 per lane the shuffles and stores double: 0.153 ms.)
template <uint32_t kFill = 0>
__device__ __forceinline__ uint2 expand_step(const Quarter &qt, const int k, const uint32_t lane, uint32_t &bits)
{
    const int      from = k * 4 + (lane >> 3);
    const uint32_t w    = __shfl_sync(kFull, qt.word, from);
    const uint32_t wex  = __shfl_sync(kFull, qt.excl, from);
    const uint32_t sh   = (lane & 7u) * 4u;
    const uint32_t off  = wex + __popc(w & ((1u << sh) - 1u));
    bits                = w >> sh;
    return expand4_u16<kFill>(qt.run + 2u * off, bits);
}

}  // namespace q16
}  // namespace bt
