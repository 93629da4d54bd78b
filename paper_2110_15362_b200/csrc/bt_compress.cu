// Algorithm 1 (dense -> bitmap) and its ReLU-fused form as ONE compaction pass:
// a persistent-CTA stream compaction with a single-pass scan (decoupled
// look-back over per-tile descriptors).
//
// Per CTA: tiles are handed out by an atomic ticket (so a tile's predecessors
// always belong to CTAs that are already running), staged into shared memory
// by 1-D bulk async copies through a ring of kStages buffers, and each warp
// owns 1024 consecutive elements of the tile = 32 bitmap words:
//
//   step k of a warp:  lane l reads element 32k+l from shared memory;
//                      ballot(non-zero) IS bitmap word k (LSB first);
//                      popc(ballot & lanemask_lt) is the lane's rank;
//                      non-zero lanes write the element back IN PLACE at
//                      [run + rank] of the warp's own segment (always at or
//                      before the position being read, so nothing unread is
//                      overwritten).
//
// After 32 steps lane k holds word k (one coalesced 128-byte bitmap store) and
// the segment's first `run` slots hold the packed values.  Warp 0 then scans
// the warp counts, publishes the tile aggregate, looks back for the tile's
// exclusive base, writes the chunk prefix entries, and every warp copies its
// packed slots out to values[base + warp offset ...], contiguous per warp.
#include <mutex>

#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr int      kWarpElems = 1024;                 // 32 steps x 32 lanes
constexpr uint32_t kFull      = 0xFFFFFFFFu;
constexpr uint64_t kWaitNs    = 2000000000ull;        // bound of every in-kernel wait: 2 s

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

// Raise the abort flag (shared and global) and report the timeout.
__device__ __noinline__ void raise_timeout(const CompressArgs &a, volatile uint32_t *s_abort)
{
    *s_abort = 1u;
    st_relaxed_u32(a.ws_header + 1, 1u);
    __threadfence();
    if (a.dev_status) *reinterpret_cast<volatile int32_t *>(a.dev_status) = BT_ERR_TIMEOUT;
}

// Bounded wait for a bulk copy to land.  False once the limit passed or another CTA aborted.
__device__ __forceinline__ bool wait_full(uint64_t *bar, uint32_t parity, const CompressArgs &a)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (now_ns() - t0 > kWaitNs) return false;
    }
}

// Decoupled look-back by one warp: exclusive prefix of tile t (t > 0).
// Each poll reads the 32 predecessors t-1-lane; a window with an inclusive
// entry ends the walk, otherwise its aggregates are added and the window moves
// back by 32.  Entries before tile 0 count as "inclusive 0".
__device__ __forceinline__ bool look_back(const CompressArgs &a, uint32_t t, uint32_t lane, uint64_t &base_out)
{
    uint64_t base = 0;
    int64_t  idx  = static_cast<int64_t>(t) - 1 - lane;
    uint64_t t0   = 0;
    uint32_t polls = 0;
    for (;;) {
        uint64_t d = (idx >= 0) ? ld_relaxed_u64(a.ws_desc + idx) : kStateInclusive;
        if (__any_sync(kFull, (d & 3u) == kStateInvalid)) {
            // not all 32 predecessors have published yet: poll again, bounded
            if (++polls > 16) {
                __nanosleep(64);
                if ((polls & 255u) == 0) {
                    if (t0 == 0) t0 = now_ns();
                    const bool give_up = (now_ns() - t0 > kWaitNs) || ld_relaxed_u32(a.ws_header + 1) != 0;
                    if (__any_sync(kFull, give_up)) return false;
                }
            }
            continue;
        }
        const uint32_t incl = __ballot_sync(kFull, (d & 3u) == kStateInclusive);
        uint64_t       v    = d >> 2;
        if (incl) {
            const uint32_t first = __ffs(incl) - 1;   // nearest predecessor holding an inclusive prefix
            if (lane > first) v = 0;
            base_out = base + warp_sum_u64(v);
            return true;
        }
        base += warp_sum_u64(v);
        idx -= 32;
    }
}

// U: uint32_t (4-byte elements) or uint16_t (2-byte elements).
// RELU_DT: -1 for the plain compressor, else the element type whose ReLU is fused in.
template <typename U, int RELU_DT, bool WRITE_Y, int kWarps, int kStages>
__global__ void __launch_bounds__(kWarps * 32) compress_kernel(const CompressArgs a, const uint32_t num_tiles)
{
    constexpr int kThreads       = kWarps * 32;
    constexpr int kTile          = kWarps * kWarpElems;
    constexpr int kChunksPerTile = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk = BT_CHUNK_ELEMS / kWarpElems;
    static_assert(kTile % BT_CHUNK_ELEMS == 0, "a tile holds whole chunks");

    extern __shared__ __align__(128) unsigned char smem_raw[];
    U *const tiles = reinterpret_cast<U *>(smem_raw);

    __shared__ __align__(8) uint64_t s_full[kStages];
    __shared__ uint32_t          s_tile[kStages];   // tile held (or being loaded) by each stage
    __shared__ uint32_t          s_done[kStages];   // warps that finished copying a stage out
    __shared__ uint32_t          s_next;            // ticket for the next refill
    __shared__ uint32_t          s_warp_cnt[kWarps];
    __shared__ uint32_t          s_warp_off[kWarps];
    __shared__ uint64_t          s_base;
    __shared__ volatile uint32_t s_abort;

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;
    const uint32_t lt   = lanemask_lt();
    const U *const src  = static_cast<const U *>(a.src);
    U *const       vals = static_cast<U *>(a.values);
    const uint64_t words_total  = (a.n + 31) >> 5;
    const uint64_t chunks_total = (a.n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS;

    // Issue the bulk load of tile t into stage s (one thread).
    auto issue_load = [&](uint32_t s, uint32_t t) {
        const uint64_t first = static_cast<uint64_t>(t) * kTile;
        const uint64_t left  = a.n - first;
        const uint32_t valid = left < static_cast<uint64_t>(kTile) ? static_cast<uint32_t>(left) : kTile;
        const uint32_t bytes = (valid * static_cast<uint32_t>(sizeof(U))) & ~15u;   // whole 16-byte units
        fence_proxy_async();                       // earlier generic accesses to this stage come first
        mbar_arrive_expect_tx(&s_full[s], bytes);  // bytes == 0 simply completes the phase
        if (bytes) bulk_load(tiles + static_cast<size_t>(s) * kTile, src + first, bytes, &s_full[s]);
    };

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&s_full[s], 1);
            s_done[s] = 0;
        }
        fence_proxy_async();
        for (int s = 0; s < kStages; ++s) {
            const uint32_t t = atomicAdd(a.ws_header, 1u);
            s_tile[s] = t;
            if (t < num_tiles) issue_load(s, t);
        }
    }
    __syncthreads();

    for (uint32_t it = 0;; ++it) {
        const uint32_t s = it % kStages;
        const uint32_t t = s_tile[s];
        if (t >= num_tiles) break;
        const uint32_t parity = (it / kStages) & 1u;
        U *const       tile   = tiles + static_cast<size_t>(s) * kTile;
        const uint64_t first  = static_cast<uint64_t>(t) * kTile;

        // ticket for the refill of this stage, asked for now and used after the copy-out
        uint32_t ticket = 0;
        if (tid == 0) ticket = atomicAdd(a.ws_header, 1u);

        if (!wait_full(&s_full[s], parity, a)) raise_timeout(a, &s_abort);

        if (a.n - first < static_cast<uint64_t>(kTile)) {
            // ragged last tile: fetch what the 16-byte granular bulk copy left out, zero the rest
            const uint32_t valid   = static_cast<uint32_t>(a.n - first);
            const uint32_t by_bulk = ((valid * static_cast<uint32_t>(sizeof(U))) & ~15u) / sizeof(U);
            for (uint32_t e = by_bulk + tid; e < static_cast<uint32_t>(kTile); e += kThreads)
                tile[e] = (e < valid) ? src[first + e] : U(0);
            __syncthreads();
        }

        // ---- per-warp in-place compaction of 1024 elements
        U *const seg    = tile + warp * kWarpElems;
        uint32_t run    = 0;
        uint32_t myword = 0;
#pragma unroll 1
        for (int kb = 0; kb < 32; kb += 8) {
            uint32_t v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = seg[(kb + j) * 32 + lane];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t x = v[j];
                if constexpr (RELU_DT >= 0) {
                    x = ReluKeep<RELU_DT>::keep(x) ? x : 0u;
                    if constexpr (WRITE_Y) {
                        const uint64_t g = first + warp * kWarpElems + (kb + j) * 32 + lane;
                        if (g < a.n) static_cast<U *>(a.y)[g] = static_cast<U>(x);
                    }
                }
                const bool     p = x != 0u;
                const uint32_t b = __ballot_sync(kFull, p);
                if (lane == static_cast<uint32_t>(kb + j)) myword = b;
                if (p) seg[run + __popc(b & lt)] = static_cast<U>(x);
                run += __popc(b);
            }
        }
        {
            const uint64_t w = static_cast<uint64_t>(t) * (kTile / 32) + warp * 32 + lane;
            if (w < words_total) a.bitmap[w] = myword;
        }
        if (lane == 0) s_warp_cnt[warp] = run;
        __syncthreads();   // B1: warp counts visible; every lane's packed slots written

        if (warp == 0 && !s_abort) {   // a CTA whose load never landed publishes nothing
            // scan of the warp counts
            const uint32_t c   = lane < kWarps ? s_warp_cnt[lane] : 0u;
            uint32_t       inc = c;
#pragma unroll
            for (int o = 1; o < kWarps; o <<= 1) {
                const uint32_t u = __shfl_up_sync(kFull, inc, o);
                if (lane >= static_cast<uint32_t>(o)) inc += u;
            }
            const uint32_t agg = __shfl_sync(kFull, inc, kWarps - 1);
            uint64_t       base = 0;
            bool           ok   = true;
            if (t == 0) {
                if (lane == 0) st_relaxed_u64(a.ws_desc, (static_cast<uint64_t>(agg) << 2) | kStateInclusive);
            } else {
                if (lane == 0) st_relaxed_u64(a.ws_desc + t, (static_cast<uint64_t>(agg) << 2) | kStateAggregate);
                ok = look_back(a, t, lane, base);
                if (ok && lane == 0)
                    st_relaxed_u64(a.ws_desc + t, ((base + agg) << 2) | kStateInclusive);
            }
            if (!ok) {
                if (lane == 0) raise_timeout(a, &s_abort);
            } else {
                if (lane < kWarps) s_warp_off[lane] = inc - c;
                if (lane == 0) {
                    s_base = base;
                    s_next = ticket;
                }
                // exclusive count in front of each chunk of this tile
                if (lane < kWarps && (lane % kWarpsPerChunk) == 0) {
                    const uint64_t ch = static_cast<uint64_t>(t) * kChunksPerTile + lane / kWarpsPerChunk;
                    if (ch < chunks_total) a.prefix[ch] = base + (inc - c);
                }
                if (t == num_tiles - 1 && lane == 0) {
                    const uint64_t nnz = base + agg;
                    *a.nnz_out = nnz;
                    __threadfence();
                    const bool aborted = ld_relaxed_u32(a.ws_header + 1) != 0;
                    if (a.dev_status)
                        *a.dev_status = aborted ? BT_ERR_TIMEOUT : (nnz > a.capacity ? BT_ERR_CAPACITY : BT_OK);
                }
            }
        }
        __syncthreads();   // B2: base and warp offsets visible
        if (s_abort) {
            // leaving early: first let this CTA's bulk copies still in flight land (bounded)
            for (uint32_t d = 1; d < static_cast<uint32_t>(kStages); ++d) {
                const uint32_t it2 = it + d;
                if (s_tile[it2 % kStages] < num_tiles) wait_full(&s_full[it2 % kStages], (it2 / kStages) & 1u, a);
            }
            return;
        }

        // ---- copy this warp's packed slots out, contiguous in values[]
        {
            const uint64_t dst = s_base + s_warp_off[warp];
            for (uint32_t j = lane; j < run; j += 32)
                if (dst + j < a.capacity) vals[dst + j] = seg[j];
        }
        __syncwarp();
        if (lane == 0) {
            __threadfence_block();
            if (atomicAdd(&s_done[s], 1u) == kWarps - 1) {
                // last warp out of this stage refills it
                __threadfence_block();
                s_done[s]       = 0;
                const uint32_t nt = s_next;
                s_tile[s]       = nt;
                if (nt < num_tiles) issue_load(s, nt);
            }
        }
    }
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

template <typename U, int RELU_DT, bool WRITE_Y>
cudaError_t launch_typed(const CompressArgs &a, cudaStream_t stream)
{
    constexpr int kWarps  = 8;
    constexpr int kStages = 3;
    constexpr int kTile   = kWarps * kWarpElems;
    constexpr size_t kSmem = static_cast<size_t>(kStages) * kTile * sizeof(U);
    static LaunchShape shape;   // one per instantiation
    auto kernel = compress_kernel<U, RELU_DT, WRITE_Y, kWarps, kStages>;

    const uint32_t num_tiles = static_cast<uint32_t>((a.n + kTile - 1) / kTile);
    int            max_grid  = 0;
    cudaError_t    e         = shape.max_grid(kernel, kWarps * 32, kSmem, max_grid);
    if (e != cudaSuccess) return e;
    // ticket, abort flag and the descriptors start at zero
    e = cudaMemsetAsync(a.ws_header, 0, kWsHeaderBytes + 8 * static_cast<size_t>(num_tiles), stream);
    if (e != cudaSuccess) return e;
    const uint32_t grid = num_tiles < static_cast<uint32_t>(max_grid) ? num_tiles : static_cast<uint32_t>(max_grid);
    kernel<<<grid, kWarps * 32, kSmem, stream>>>(a, num_tiles);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_compress(const CompressArgs &a, int dtype, bool relu, cudaStream_t stream)
{
    const bool y = a.y != nullptr;
    if (!relu) {
        return dtype == BT_F32 ? launch_typed<uint32_t, -1, false>(a, stream)
                               : launch_typed<uint16_t, -1, false>(a, stream);
    }
    switch (dtype) {
    case BT_F32:
        return y ? launch_typed<uint32_t, BT_F32, true>(a, stream) : launch_typed<uint32_t, BT_F32, false>(a, stream);
    case BT_F16:
        return y ? launch_typed<uint16_t, BT_F16, true>(a, stream) : launch_typed<uint16_t, BT_F16, false>(a, stream);
    default:
        return y ? launch_typed<uint16_t, BT_BF16, true>(a, stream)
                 : launch_typed<uint16_t, BT_BF16, false>(a, stream);
    }
}

}  // namespace bt
