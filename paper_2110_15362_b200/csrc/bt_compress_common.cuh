// What the single-tensor and the batched compress kernels share: constants of the workspace protocol, small PTX
// wrappers, the bounded mbarrier wait, the in-place compaction of one segment by one warp, the copy-out of a
// packed segment, and the host-side launch shape.
#pragma once

#include <mutex>
#include <type_traits>

#include "bt_internal.cuh"

namespace bt {

// A value no other call of this process gets (bt_compress.cu).
uint64_t next_call_tag();
// The calling thread's limit on the CTAs of one compress launch, 0: none (bt_compress.cu).
uint32_t compress_max_ctas();
// The bound of the kernels' waits in nanoseconds; only a test build can change it (bt_compress.cu).
uint64_t compress_wait_ns();

namespace cmp {

constexpr uint32_t kFull       = 0xFFFFFFFFu;
constexpr int      kMaxWindows = 5;                   // the grid never exceeds 32 * kMaxWindows CTAs
constexpr int      kHdrSeq     = 0;                   // header words (64-bit): launch sequence number,
constexpr int      kHdrAbort   = 1;                   //   abort word (== the launch's tag once a wait ran out)
constexpr int      kCountShift = 40;                  // wave total word: (tiles added << 40) | sum of counts


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

// Raise the abort flag (shared, and global under this launch's tag if a scan warp got as far as reading it),
// move the workspace's sequence number so that the next launch cannot take this one's words for its own, and
// report the timeout.
static __device__ __noinline__ void raise_timeout(uint64_t *ws_header, int32_t *dev_status, volatile uint32_t *s_abort,
                                           const uint64_t tag)
{
    *s_abort = 1u;
    if (tag) st_relaxed_u64(ws_header + kHdrAbort, tag);
    red_add_u64(ws_header + kHdrSeq, 1ull << 32);
    __threadfence();
    if (dev_status) *reinterpret_cast<volatile int32_t *>(dev_status) = BT_ERR_TIMEOUT;
}

// A limit below this is kept to the nanosecond (see mbar_wait_strict).  Only the test build of the library
// (-DBT_TEST_HOOKS) can set such a limit, and only that build carries the code for it: the product's waits
// are the same instructions with or without it.
constexpr uint64_t kStrictLimitNs = 1000;
#ifdef BT_TEST_HOOKS
constexpr bool kTestHooks = true;
#else
constexpr bool kTestHooks = false;
#endif

// The wait under a limit of less than a microsecond, which only a test build of the library can set: probes that
// return at once (a try_wait may itself suspend the thread for longer than such a limit), the clock read after
// every probe.  A phase that is not complete at the first probe and does not complete within the limit fails.
static __device__ __noinline__ bool mbar_wait_strict(uint64_t *bar, const uint32_t parity, const uint64_t limit_ns)
{
    const uint64_t t0 = now_ns();
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(smem_addr(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
        if (now_ns() - t0 > limit_ns) return false;
    }
}

// Bounded wait on an mbarrier phase.  False once the limit passed or the CTA is aborting.  The limit is checked
// every 32 probes, each of which may suspend the thread for a while: exact enough for the product's two seconds.
template <bool kStopOnAbort = true>
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *s_abort, const uint64_t limit_ns)
{
    if (kTestHooks && limit_ns < kStrictLimitNs) return mbar_wait_strict(bar, parity, limit_ns);
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if ((kStopOnAbort && *s_abort) || now_ns() - t0 > limit_ns) return false;
    }
}

// shared-memory accesses by 32-bit shared address, kept in program order among themselves
// register type that holds one element: 64 bits for 8-byte elements, 32 bits otherwise
template <typename U>
using Reg = std::conditional_t<sizeof(U) == 8, uint64_t, uint32_t>;

template <typename U>
__device__ __forceinline__ Reg<U> lds_elem(uint32_t addr)
{
    Reg<U> v;
    if constexpr (sizeof(U) == 8) asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr));
    else if constexpr (sizeof(U) == 4) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    else asm volatile("ld.shared.s16 %0, [%1];" : "=r"(v) : "r"(addr));   // sign-extended
    return v;
}

// ---------------------------------------------------------------------------------------------
// One warp compacts its segment of kSteps * 32 elements in place.  Returns the number of packed
// values; lane k leaves with the ballot of step k, which is bitmap word k of the segment, in `word`
// (kept in registers through a tree of selects: a store to shared memory per step costs more).
// `y` (fused form with dense output) points at the segment's first element of the dense ReLU
// output, `yvalid` is how many of them exist.  seg_addr is a shared-window address.
//
// The loads of a batch of 8 steps are issued before the stores of the batch before it: a store of
// step k lands below element 32(k+1) and a later batch reads at or above it, so they never meet.
//
// Which pipe an instruction runs on decides the speed of this loop: with 2-byte elements the kernel is bound by
// the SM's integer/logic pipe (73 % busy, the top stall reason "math pipe throttle"), which the compare, the
// mask of the ballot, the address arithmetic and the selects of a step all queue at.  So what can be a
// multiply-add is one (those run on the FMA pipe): the ballot bits below the lane are b * 2^(32 - lane) instead
// of b & lanemask_lt, addresses are rank * size + base with the size in a register the compiler cannot see
// through, and lane k takes ballot k as a sum of ballots times 0/1 factors instead of through a tree of selects.
// On the 392 MiB bf16 tensor: 0.1485 -> 0.139 ms plain, 0.165 -> 0.138 ms fused (with the compare below).
template <typename U, int RELU_DT, bool WRITE_Y, bool kGuardY, int kSteps>
__device__ __forceinline__ uint32_t compact_segment(const uint32_t seg_addr, uint32_t &word, const uint32_t lane,
                                                    U *y, const uint32_t yvalid, const float tau, const Extent yx)
{
    constexpr int      kBatch = 8;
    static_assert(kSteps % kBatch == 0 && kSteps <= 32, "whole batches; one bitmap word per lane");
    constexpr uint32_t kES    = sizeof(U);
    const uint32_t     in0    = seg_addr + lane * kES;
    uint32_t           out    = seg_addr;               // address of the next free packed slot
    Reg<U>             v[kBatch], vn[kBatch];
    const uint32_t     below  = lane ? (1u << (32u - lane)) : 0u;   // b * below: the ballot bits of the lanes below, at the top
    uint32_t           size, pick[kBatch];              // element size; pick[j] = 1 on the lanes that keep ballot j of a batch
    asm volatile("mov.u32 %0, %1;" : "=r"(size) : "n"(kES));
#pragma unroll
    for (int j = 0; j < kBatch; ++j) asm volatile("mov.u32 %0, %1;" : "=r"(pick[j]) : "r"((lane & 7u) == static_cast<uint32_t>(j) ? 1u : 0u));
    word = 0;
#pragma unroll
    for (int j = 0; j < kBatch; ++j) v[j] = lds_elem<U>(in0 + j * 32 * kES);
#pragma unroll
    for (int kb = 0; kb < kSteps; kb += kBatch) {
        if (kb + kBatch < kSteps) {
#pragma unroll
            for (int j = 0; j < kBatch; ++j) vn[j] = lds_elem<U>(in0 + (kb + kBatch + j) * 32 * kES);
        }
        uint32_t w = 0;
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            Reg<U> x = v[j];
            bool   nz;
            if constexpr (RELU_DT >= kFusedReluHalf) {
                nz = relu_keeps_half<RELU_DT & 3>(x);        // a kept element is never the zero pattern
                if constexpr (RELU_DT >= kFusedRelu6Half) x = relu6_saturates_half<RELU_DT & 3>(x) ? Elem<RELU_DT & 3>::kSix : x;
                if constexpr (WRITE_Y) {
                    const uint32_t e = (kb + j) * 32 + lane;
                    if ((!kGuardY || e < yvalid) && yx.holds(y + e, sizeof(U))) y[e] = nz ? static_cast<U>(x) : U(0);
                }
            } else {
                if constexpr (RELU_DT >= 0) {
                    x = fused_forward<RELU_DT>(x, tau);
                    if constexpr (WRITE_Y) {
                        const uint32_t e = (kb + j) * 32 + lane;
                        if ((!kGuardY || e < yvalid) && yx.holds(y + e, sizeof(U))) y[e] = static_cast<U>(x);
                    }
                }
                nz = x != Reg<U>(0);
            }
            const uint32_t b = __ballot_sync(kFull, nz);
            uint32_t       lower, at;
            asm("mul.lo.u32 %0, %1, %2;" : "=r"(lower) : "r"(b), "r"(below));
            asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(at) : "r"(__popc(lower)), "r"(size), "r"(out));
            if (nz) {
                if constexpr (kES == 8) asm volatile("st.shared.u64 [%0], %1;" ::"r"(at), "l"(x));
                else if constexpr (kES == 4) asm volatile("st.shared.u32 [%0], %1;" ::"r"(at), "r"(x));
                else asm volatile("st.shared.u16 [%0], %1;" ::"r"(at), "h"(static_cast<uint16_t>(x)));
            }
            asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(out) : "r"(__popc(b)), "r"(size));
            asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(w) : "r"(b), "r"(pick[j]));
        }
        word = (lane >> 3) == static_cast<uint32_t>(kb / 8) ? w : word;     // lane kb + j keeps ballot j of this batch
#pragma unroll
        for (int j = 0; j < kBatch; ++j) v[j] = vn[j];
    }
    return (out - seg_addr) / kES;
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

// One warp copies the `cnt` packed slots of its segment to out[0..cnt): contiguous, coalesced.
template <typename U, int CAST, bool kGuard>
__device__ __forceinline__ void copy_out_segment(const U *__restrict__ seg, const uint32_t lane, const uint32_t cnt,
                                                 Stored<CAST, U> *__restrict__ out, const uint64_t room, const Extent vx)
{
    // (Pairing narrowed values into 4-byte stores was measured and is no faster: at half zeros the narrowing
    // forms run at the speed of the compaction, not of the copy-out.)
    uint32_t j = lane;
    for (; j + 96 < cnt; j += 128) {
        const auto v0 = narrowed<CAST>(seg[j]), v1 = narrowed<CAST>(seg[j + 32]), v2 = narrowed<CAST>(seg[j + 64]),
                   v3 = narrowed<CAST>(seg[j + 96]);
        if ((!kGuard || j < room) && vx.holds(out + j, sizeof(*out))) out[j] = v0;
        if ((!kGuard || j + 32 < room) && vx.holds(out + j + 32, sizeof(*out))) out[j + 32] = v1;
        if ((!kGuard || j + 64 < room) && vx.holds(out + j + 64, sizeof(*out))) out[j + 64] = v2;
        if ((!kGuard || j + 96 < room) && vx.holds(out + j + 96, sizeof(*out))) out[j + 96] = v3;
    }
    for (; j < cnt; j += 32) {
        const auto v = narrowed<CAST>(seg[j]);
        if ((!kGuard || j < room) && vx.holds(out + j, sizeof(*out))) out[j] = v;
    }
}

// The copy-out of a packed run of 2-byte values through the copy engine.  A lane-by-lane copy costs a shared load
// and a 2-byte global store per survivor on the port the compactors' votes, counts and stores also queue at; a
// bulk copy reads shared memory by itself.  It wants source and destination on 16-byte boundaries, and the
// destination is wherever the run's rank puts it: so the up to 7 values in front of the destination's first
// boundary and the up to 7 behind its last one leave as single elements, and the rest is first moved down inside
// the segment by that many elements (two 16-byte loads, four funnel shifts, one 16-byte store per 8 values;
// loads of a round before its stores, rounds in rising order, so nothing is overwritten before it is read).
// The caller waits for the copy engine's reads (bulk_store_wait_read) before it releases the slot.
constexpr bool kBulkCopyOut16 = true;

__device__ __forceinline__ void bulk_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

__device__ __forceinline__ void copy_out_run16(uint16_t *seg, const uint32_t lane, const uint32_t cnt, uint16_t *out,
                                               const Extent vx)
{
    const uint32_t sa = smem_addr(seg);
    uint32_t       h  = (static_cast<uint32_t>(16u - (reinterpret_cast<uintptr_t>(out) & 15u)) & 15u) >> 1;
    h                 = h < cnt ? h : cnt;                       // values in front of the first boundary
    const uint32_t vecs = (cnt - h) >> 3;                        // whole 16-byte units behind them
    const uint32_t tail = h + 8u * vecs;                         // first of the values behind the last unit
    // the ragged ends: lanes 0..6 the head, lanes 8..14 the tail; read now, the move below overwrites the head
    const bool     is_head = lane < h, is_tail = lane >= 8u && tail + (lane - 8u) < cnt;
    const uint32_t ei      = is_head ? lane : tail + (lane - 8u);
    uint16_t       edge    = 0;
    if (is_head || is_tail) edge = seg[ei];
    if (vecs) {
        if (h) {
            __syncwarp();
            const uint32_t sh = (h & 1u) * 16u;
            for (uint32_t v0 = 0; v0 < vecs; v0 += 32) {
                const uint32_t v  = v0 + lane;
                const uint32_t at = sa + 16u * v;
                uint32_t       w0 = 0, w1 = 0, w2 = 0, w3 = 0, w4 = 0, w5 = 0, w6 = 0, w7 = 0;
                if (v < vecs) {
                    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(at));
                    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w4), "=r"(w5), "=r"(w6), "=r"(w7) : "r"(at + 16u));
                }
                __syncwarp();
                if (v < vecs) {
                    uint32_t o0, o1, o2, o3;
                    switch (h >> 1) {                              // the same for the whole warp
                    case 0: o0 = __funnelshift_r(w0, w1, sh), o1 = __funnelshift_r(w1, w2, sh), o2 = __funnelshift_r(w2, w3, sh), o3 = __funnelshift_r(w3, w4, sh); break;
                    case 1: o0 = __funnelshift_r(w1, w2, sh), o1 = __funnelshift_r(w2, w3, sh), o2 = __funnelshift_r(w3, w4, sh), o3 = __funnelshift_r(w4, w5, sh); break;
                    case 2: o0 = __funnelshift_r(w2, w3, sh), o1 = __funnelshift_r(w3, w4, sh), o2 = __funnelshift_r(w4, w5, sh), o3 = __funnelshift_r(w5, w6, sh); break;
                    default: o0 = __funnelshift_r(w3, w4, sh), o1 = __funnelshift_r(w4, w5, sh), o2 = __funnelshift_r(w5, w6, sh), o3 = __funnelshift_r(w6, w7, sh); break;
                    }
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(at), "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                }
            }
            fence_proxy_async();                                  // the moved values, before the copy engine reads them
        }
        __syncwarp();
        if (lane == 0 && vx.holds(out + h, 16u * vecs)) {
            fence_proxy_async();                                  // the compactors' stores (ordered before this by the mbarriers)
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(out + h), "r"(sa), "r"(16u * vecs) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
    if ((is_head || is_tail) && vx.holds(out + ei, 2)) out[ei] = edge;
}

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


}  // namespace cmp
}  // namespace bt
