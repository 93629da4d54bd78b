// Algorithm 1 (dense -> bitmap) and its ReLU-fused form as ONE compaction pass:
// a persistent-CTA stream compaction with a single-pass scan (decoupled
// look-back over per-tile descriptors).
//
// A CTA is kWarps worker warps plus one scan warp.  The grid is launched
// cooperatively with exactly as many CTAs as fit on the device at once, so all
// of them are co-resident, and CTA b takes tiles b, b+G, b+2G, ... : the CTAs
// move through the tensor in waves and a tile's predecessors are always being
// worked on.  Tiles are staged into shared memory by 1-D bulk async copies
// through a ring of kStages buffers.  Each worker warp owns 1024 consecutive
// elements of the tile = 32 bitmap words:
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
// the segment's first `run` slots hold the packed values.  The scan warp takes
// the 8 warp counts of tile i, publishes the tile aggregate, looks back for the
// tile's exclusive base and writes the chunk prefix entries WHILE the workers
// already compact tile i+1; the workers copy tile i's packed slots out to
// values[base + warp offset ...] one iteration later, so the look-back latency
// hides behind the next tile's compaction and no tile's count waits on another
// tile's copy-out.
#include <cstdlib>
#include <mutex>

#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr int      kWarpElems = 1024;                 // 32 steps x 32 lanes
constexpr uint32_t kFull      = 0xFFFFFFFFu;
constexpr uint64_t kWaitNs    = 2000000000ull;        // bound of every in-kernel wait: 2 s

// named barriers (0 is __syncthreads)
constexpr int kBarCounts = 1;   // +parity: workers arrive, scan warp waits: warp counts of a tile are in shared memory
constexpr int kBarBase   = 3;   // +parity: scan warp arrives, workers wait: base and warp offsets of a tile are ready
constexpr int kBarWorkers = 5;  // workers only

__device__ __forceinline__ void bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int threads)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

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
__device__ __noinline__ void raise_timeout(uint32_t *ws_header, int32_t *dev_status, volatile uint32_t *s_abort)
{
    *s_abort = 1u;
    st_relaxed_u32(ws_header + 1, 1u);
    __threadfence();
    if (dev_status) *reinterpret_cast<volatile int32_t *>(dev_status) = BT_ERR_TIMEOUT;
}

// Bounded wait for a bulk copy to land.  False once the limit passed.
__device__ __forceinline__ bool wait_full(uint64_t *bar, uint32_t parity)
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
// Persistent CTAs move through the tiles in waves, so the nearest tile that
// already holds an inclusive prefix can be a whole wave (hundreds of tiles)
// back.  The walk therefore loads kLookWindows windows of 32 predecessors at
// once (independent loads, one round trip) and consumes them nearest first: a
// window with an inclusive entry ends the walk, a window of aggregates is
// added; a window with an unpublished entry is polled on its own until it is
// complete.  Entries before tile 0 count as "inclusive 0".
constexpr int kLookWindows = 8;

__device__ __forceinline__ bool look_back(const uint64_t *desc, const uint32_t *abort_flag, uint32_t t,
                                          uint32_t lane, uint64_t &base_out)
{
    uint64_t part = 0;                                    // this lane's share of the sum
    int64_t  top  = static_cast<int64_t>(t) - 1;          // nearest predecessor not yet consumed
    for (;;) {
        uint64_t d[kLookWindows];
#pragma unroll
        for (int j = 0; j < kLookWindows; ++j) {
            const int64_t idx = top - lane - 32 * j;
            d[j] = (idx >= 0) ? ld_relaxed_u64(desc + idx) : kStateInclusive;
        }
#pragma unroll
        for (int j = 0; j < kLookWindows; ++j) {
            uint64_t dj    = d[j];
            uint32_t polls = 0;
            uint64_t t0    = 0;
            while (__any_sync(kFull, (dj & 3u) == kStateInvalid)) {
                if (++polls > 4) {
                    __nanosleep(20);
                    if ((polls & 255u) == 0) {
                        if (t0 == 0) t0 = now_ns();
                        const bool give_up = (now_ns() - t0 > kWaitNs) || ld_relaxed_u32(abort_flag) != 0;
                        if (__any_sync(kFull, give_up)) return false;
                    }
                }
                const int64_t idx = top - lane;
                dj = (idx >= 0) ? ld_relaxed_u64(desc + idx) : kStateInclusive;
            }
            const uint32_t incl = __ballot_sync(kFull, (dj & 3u) == kStateInclusive);
            if (incl) {
                const uint32_t first = __ffs(incl) - 1;   // nearest predecessor holding an inclusive prefix
                if (lane <= first) part += dj >> 2;
                base_out = warp_sum_u64(part);
                return true;
            }
            part += dj >> 2;
            top -= 32;
        }
    }
}

// U: uint32_t (4-byte elements) or uint16_t (2-byte elements).
// RELU_DT: -1 for the plain compressor, else the element type whose ReLU is fused in.
template <typename U, int RELU_DT, bool WRITE_Y, int kWarps, int kStages>
__global__ void __launch_bounds__(kWarps * 32 + 32) compress_kernel(const CompressArgs a, const uint32_t num_tiles)
{
    constexpr int kWorkerThreads = kWarps * 32;
    constexpr int kThreads       = kWorkerThreads + 32;
    constexpr int kTile          = kWarps * kWarpElems;
    constexpr int kChunksPerTile = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk = BT_CHUNK_ELEMS / kWarpElems;
    static_assert(kTile % BT_CHUNK_ELEMS == 0, "a tile holds whole chunks");
    static_assert(kStages >= 3, "one stage compacting, one awaiting copy-out, at least one loading");

    extern __shared__ __align__(128) unsigned char smem_raw[];
    U *const tiles = reinterpret_cast<U *>(smem_raw);

    __shared__ __align__(8) uint64_t s_full[kStages];
    __shared__ uint32_t          s_done[kStages];      // warps that finished copying a stage out
    __shared__ uint32_t          s_cnt[2][kWarps];     // by tile parity: packed count of each warp
    __shared__ uint32_t          s_off[2][kWarps];     //                 exclusive offset of each warp in the tile
    __shared__ uint64_t          s_base[2];            //                 exclusive base of the tile
    __shared__ volatile uint32_t s_abort;

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;
    const U *const src  = static_cast<const U *>(a.src);
    const uint64_t n    = a.n;

    // Issue the bulk load of tile t into stage s (one thread).
    auto issue_load = [&](uint32_t s, uint32_t t) {
        const uint64_t first = static_cast<uint64_t>(t) * kTile;
        const uint64_t left  = n - first;
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
            const uint64_t t = blockIdx.x + static_cast<uint64_t>(s) * gridDim.x;
            if (t < num_tiles) issue_load(s, static_cast<uint32_t>(t));
        }
    }
    __syncthreads();
    // tile of iteration `it` of this CTA (64-bit so that running past the end cannot wrap)
    auto tile_of = [&](uint32_t it) { return blockIdx.x + static_cast<uint64_t>(it) * gridDim.x; };

    if (warp == kWarps) {
        // ------------------------------------------------------------ scan warp
        uint64_t *const desc         = a.ws_desc;
        const uint64_t  chunks_total = (n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS;
        for (uint32_t it = 0;; ++it) {
            const uint64_t t64 = tile_of(it);
            if (t64 >= num_tiles) return;
            const uint32_t t   = static_cast<uint32_t>(t64);
            const uint32_t par = it & 1u;

            bar_sync(kBarCounts + par, kThreads);             // warp counts of tile `it` are in
            if (s_abort) {                                    // a load never landed: publish nothing
                bar_arrive(kBarBase + par, kThreads);
                return;
            }
            const uint32_t c   = lane < kWarps ? s_cnt[par][lane] : 0u;
            uint32_t       inc = c;
#pragma unroll
            for (int o = 1; o < kWarps; o <<= 1) {
                const uint32_t u = __shfl_up_sync(kFull, inc, o);
                if (lane >= static_cast<uint32_t>(o)) inc += u;
            }
            const uint32_t agg  = __shfl_sync(kFull, inc, kWarps - 1);
            uint64_t       base = 0;
            bool           ok   = true;
            if (t == 0) {
                if (lane == 0) st_relaxed_u64(desc, (static_cast<uint64_t>(agg) << 2) | kStateInclusive);
            } else {
                if (lane == 0) st_relaxed_u64(desc + t, (static_cast<uint64_t>(agg) << 2) | kStateAggregate);
                ok = look_back(desc, a.ws_header + 1, t, lane, base);
                if (ok && lane == 0) st_relaxed_u64(desc + t, ((base + agg) << 2) | kStateInclusive);
            }
            if (!ok) {
                if (lane == 0) raise_timeout(a.ws_header, a.dev_status, &s_abort);
                __syncwarp();
                bar_arrive(kBarBase + par, kThreads);
                return;
            }
            if (lane < kWarps) s_off[par][lane] = inc - c;
            if (lane == 0) s_base[par] = base;
            bar_arrive(kBarBase + par, kThreads);             // workers may copy tile `it` out

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

    // ---------------------------------------------------------------- worker warps
    const uint32_t lt           = lanemask_lt();
    U *const       vals         = static_cast<U *>(a.values);
    const uint64_t words_total  = (n + 31) >> 5;
    const uint64_t capacity     = a.capacity;
    uint32_t       prev_run     = 0;       // packed count of this warp in the previous tile

    for (uint32_t it = 0;; ++it) {
        const uint32_t s     = it % kStages;
        const uint64_t t64   = tile_of(it);
        const bool     valid = t64 < num_tiles;
        const uint32_t t     = static_cast<uint32_t>(t64);
        const uint32_t par   = it & 1u;
        uint32_t       run   = 0;

        if (valid) {
            U *const       tile  = tiles + static_cast<size_t>(s) * kTile;
            const uint64_t first = static_cast<uint64_t>(t) * kTile;
            if (!wait_full(&s_full[s], (it / kStages) & 1u)) raise_timeout(a.ws_header, a.dev_status, &s_abort);

            if (n - first < static_cast<uint64_t>(kTile)) {
                // ragged last tile: fetch what the 16-byte granular bulk copy left out, zero the rest
                const uint32_t have    = static_cast<uint32_t>(n - first);
                const uint32_t by_bulk = ((have * static_cast<uint32_t>(sizeof(U))) & ~15u) / sizeof(U);
                for (uint32_t e = by_bulk + tid; e < static_cast<uint32_t>(kTile); e += kWorkerThreads)
                    tile[e] = (e < have) ? src[first + e] : U(0);
                bar_sync(kBarWorkers, kWorkerThreads);
            }

            // ---- per-warp in-place compaction of 1024 elements
            U *const seg    = tile + warp * kWarpElems;
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
                            if (g < n) static_cast<U *>(a.y)[g] = static_cast<U>(x);
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
            if (lane == 0) s_cnt[par][warp] = run;
            __syncwarp();
            bar_arrive(kBarCounts + par, kThreads);           // hand the counts to the scan warp
        }

        if (it > 0) {
            // ---- copy the previous tile's packed slots out, contiguous in values[]
            const uint32_t pp = par ^ 1u;
            const uint32_t ps = (it - 1) % kStages;
            bar_sync(kBarBase + pp, kThreads);                // its base and warp offsets are ready
            if (s_abort) {
                // leaving early: one warp first lets this CTA's bulk copies still in flight land (bounded)
                if (warp == 0)
                    for (uint32_t d = 1; d + 1 < static_cast<uint32_t>(kStages); ++d) {
                        const uint32_t it2 = it + d;
                        if (tile_of(it2) < num_tiles) wait_full(&s_full[it2 % kStages], (it2 / kStages) & 1u);
                    }
                return;
            }
            const U *const pseg = tiles + static_cast<size_t>(ps) * kTile + warp * kWarpElems;
            const uint64_t dst  = s_base[pp] + s_off[pp][warp];
            for (uint32_t j = lane; j < prev_run; j += 32)
                if (dst + j < capacity) vals[dst + j] = pseg[j];
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                if (atomicAdd(&s_done[ps], 1u) == kWarps - 1) {
                    // last warp out of this stage refills it with the tile it holds kStages iterations on
                    __threadfence_block();
                    s_done[ps]        = 0;
                    const uint64_t nt = tile_of(it - 1 + kStages);
                    if (nt < num_tiles) issue_load(ps, static_cast<uint32_t>(nt));
                }
            }
        }
        if (!valid) return;
        prev_run = run;
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

template <typename U, int RELU_DT, bool WRITE_Y, int kWarps, int kStages>
cudaError_t launch_shaped(const CompressArgs &a, cudaStream_t stream)
{
    constexpr int kTile   = kWarps * kWarpElems;
    constexpr int kThreads = kWarps * 32 + 32;
    constexpr size_t kSmem = static_cast<size_t>(kStages) * kTile * sizeof(U);
    static LaunchShape shape;   // one per instantiation
    auto kernel = compress_kernel<U, RELU_DT, WRITE_Y, kWarps, kStages>;

    const uint32_t num_tiles = static_cast<uint32_t>((a.n + kTile - 1) / kTile);
    int            max_grid  = 0;
    cudaError_t    e         = shape.max_grid(kernel, kThreads, kSmem, max_grid);
    if (e != cudaSuccess) return e;
    // abort flag and the descriptors start at zero
    e = cudaMemsetAsync(a.ws_header, 0, kWsHeaderBytes + 8 * static_cast<size_t>(num_tiles), stream);
    if (e != cudaSuccess) return e;
    const uint32_t grid = num_tiles < static_cast<uint32_t>(max_grid) ? num_tiles : static_cast<uint32_t>(max_grid);
    // cooperative launch: the runtime guarantees that all `grid` CTAs are resident together
    CompressArgs args = a;
    uint32_t     nt   = num_tiles;
    void *params[] = {&args, &nt};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(kThreads), params, kSmem,
                                       stream);
}

template <typename U, int RELU_DT, bool WRITE_Y>
cudaError_t launch_typed(const CompressArgs &a, cudaStream_t stream)
{
    static const int cfg = [] { const char *e = getenv("BT_CFG"); return e ? atoi(e) : 0; }();
    switch (cfg) {
    case 1: return launch_shaped<U, RELU_DT, WRITE_Y, 4, 4>(a, stream);
    case 2: return launch_shaped<U, RELU_DT, WRITE_Y, 4, 5>(a, stream);
    case 3: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 3>(a, stream);
    case 4: return launch_shaped<U, RELU_DT, WRITE_Y, 4, 3>(a, stream);
    case 5: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 6>(a, stream);
    default: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 4>(a, stream);
    }
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
