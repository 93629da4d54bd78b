// Algorithm 1 (dense -> bitmap) and its ReLU-fused form as ONE compaction pass:
// a persistent-CTA stream compaction whose prefix sum rides on the wave
// structure of the grid.
//
// The grid is launched cooperatively with exactly as many CTAs (G) as fit on
// the device at once, so all of them are co-resident, and CTA b takes tiles
// b, b+G, b+2G, ...: iteration j of every CTA together forms "wave j", G
// consecutive tiles.  A CTA is kWarps worker warps plus one scan warp.  Tiles
// are staged into shared memory by 1-D bulk async copies through a ring of
// kStages buffers.  Each worker warp owns 1024 consecutive elements of the tile
// = 32 bitmap words:
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
// the segment's first `run` slots hold the packed values.
//
// Prefix.  The exclusive base of tile (wave j, CTA b) is
//     sum of the totals of waves 0..j-1  +  sum of the counts of CTAs 0..b-1 in wave j.
// As soon as a tile is compacted its scan warp publishes the tile count in a
// descriptor and adds it (with a 1 in a counter field) to the wave's total with
// one fire-and-forget reduction.  One iteration later -- when every CTA has
// long published wave j -- it reads the b descriptors of its own wave and the
// now complete total of wave j-1 in ONE batch of independent loads, and uses
// them an iteration after that, so the round trip to L2 hides behind the
// compaction of the following tiles.  No tile waits on another tile's base:
// only on counts, which never wait on anything but the data.
//
// The warps of a CTA never meet at a CTA-wide barrier; they hand work over
// through mbarriers:
//   full[s]     the bulk copy into stage s has landed            (copy engine -> workers)
//   counted[s]  every worker has posted its packed count         (workers -> scan warp)
//   ready[s]    base and warp offsets of the tile are in shared  (scan warp -> workers)
// Each worker copies its packed slots of a tile out to values[base + warp
// offset ...] kLag iterations after compacting it; the last worker warp out of
// a stage refills it.
#include <cstdlib>
#include <mutex>

#include "bt_internal.cuh"

namespace bt {
namespace {

constexpr int      kWarpElems  = 1024;                // 32 steps x 32 lanes
constexpr uint32_t kFull       = 0xFFFFFFFFu;
constexpr uint64_t kWaitNs     = 2000000000ull;       // bound of every in-kernel wait: 2 s
constexpr int      kBarWorkers = 1;                   // named barrier of the worker warps (ragged tile only)
constexpr int      kMaxWindows = 10;                  // the grid never exceeds 32 * kMaxWindows CTAs
constexpr int      kCountShift = 40;                  // wave total word: (tiles added << 40) | sum of counts

#ifdef BT_PROFILE
#define PROF_T(var) const long long var = clock64()
#define PROF_ADD(slot, val) prof[slot] += (unsigned long long)(val)
__device__ unsigned long long *g_dbg     = nullptr;   // timeline buffer: [4 iterations][grid][8]
__device__ unsigned int        g_dbg_it0 = 0;
#define DBG_MARK(iter, slot, val)                                                                             \
    do {                                                                                                       \
        if (g_dbg && (iter) >= g_dbg_it0 && (iter) < g_dbg_it0 + 4)                                            \
            g_dbg[(((iter) - g_dbg_it0) * (size_t)gridDim.x + blockIdx.x) * 8 + (slot)] = (val);               \
    } while (0)
#else
#define PROF_T(var)
#define PROF_ADD(slot, val)
#define DBG_MARK(iter, slot, val)
#endif

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

// Raise the abort flag (shared and global) and report the timeout.
__device__ __noinline__ void raise_timeout(uint32_t *ws_header, int32_t *dev_status, volatile uint32_t *s_abort)
{
    *s_abort = 1u;
    st_relaxed_u32(ws_header + 1, 1u);
    __threadfence();
    if (dev_status) *reinterpret_cast<volatile int32_t *>(dev_status) = BT_ERR_TIMEOUT;
}

// Bounded wait on an mbarrier phase.  False once the limit passed or the CTA is aborting.
template <bool kStopOnAbort = true>
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *s_abort,
                                          uint64_t limit_ns = kWaitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = now_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if ((kStopOnAbort && *s_abort) || now_ns() - t0 > limit_ns) return false;
    }
}

// What the scan warp holds in flight for one tile: the descriptors of the lower CTAs of the
// tile's wave (lane l, window k <-> CTA l + 32k) and the total word of the previous wave.
struct PendingScan {
    uint64_t d[kMaxWindows];
    uint64_t prev_wave;
};

// U: uint32_t (4-byte elements) or uint16_t (2-byte elements).
// RELU_DT: -1 for the plain compressor, else the element type whose ReLU is fused in.
// kLag: how many iterations the copy-out of a tile trails its compaction (>= 2: the scan of a
// tile is issued one iteration and finished two iterations after the tile was counted).
template <typename U, int RELU_DT, bool WRITE_Y, int kWarps, int kStages, int kLag>
__global__ void __launch_bounds__(kWarps * 32 + 32) compress_kernel(const CompressArgs a, const uint32_t num_tiles)
{
    constexpr int kTile          = kWarps * kWarpElems;
    constexpr int kChunksPerTile = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk = BT_CHUNK_ELEMS / kWarpElems;
    constexpr int kScanWarp      = kWarps;          // warp index of the scan warp
    constexpr int kWorkerThreads = kWarps * 32;
    static_assert(kTile % BT_CHUNK_ELEMS == 0, "a tile holds whole chunks");
    static_assert(kWarps <= 32, "one lane per warp count");
    static_assert(kLag >= 2, "a tile's base is known two iterations after its count");
    static_assert(kStages >= kLag + 2, "one stage compacting, kLag awaiting copy-out, at least one loading");

    extern __shared__ __align__(128) unsigned char smem_raw[];
    U *const tiles = reinterpret_cast<U *>(smem_raw);

    __shared__ __align__(8) uint64_t s_full[kStages];
    __shared__ __align__(8) uint64_t s_counted[kStages];
    __shared__ __align__(8) uint64_t s_ready[kStages];
    __shared__ uint64_t          s_base[kStages];          // exclusive base of the tile in the stage
    __shared__ uint32_t          s_cnt[kStages][kWarps];   // packed count of each warp
    __shared__ uint32_t          s_off[kStages][kWarps];   // exclusive offset of each warp in the tile
    __shared__ uint32_t          s_done[kStages];          // warps that finished copying the stage out
    __shared__ volatile uint32_t s_abort;

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;
    const uint32_t G    = gridDim.x;
    const uint32_t cta  = blockIdx.x;
    const U *const src  = static_cast<const U *>(a.src);
    const uint64_t n    = a.n;
#ifdef BT_PROFILE
    unsigned long long prof[16] = {};
#endif

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
    // tile of iteration `it` of this CTA (64-bit so that running past the end cannot wrap)
    auto tile_of = [&](uint32_t it) { return cta + static_cast<uint64_t>(it) * G; };

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&s_full[s], 1);
            mbar_init(&s_counted[s], kWarps);
            mbar_init(&s_ready[s], 1);
            s_done[s] = 0;
        }
        fence_proxy_async();
        for (int s = 0; s < kStages; ++s)
            if (tile_of(s) < num_tiles) issue_load(s, static_cast<uint32_t>(tile_of(s)));
    }
    __syncthreads();

    if (warp == kScanWarp) {
        // ------------------------------------------------------------ scan warp
        uint64_t *const wave_total   = a.ws_desc;                  // one word per wave
        uint64_t *const desc         = a.ws_desc + a.ws_waves;     // one word per tile: (count << 1) | 1
        const uint64_t  chunks_total = (n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS;
        const uint32_t *abort_flag   = a.ws_header + 1;

        uint64_t    waves_before = 0;     // sum of the totals of all waves before the pending tile's wave
        PendingScan pend;                 // loads in flight for the pending tile (iteration it - 1)
        uint32_t    pend_agg = 0, pend_chunk_off = 0;   // of the pending tile: its count; this lane's chunk offset
        bool        failed = false;

        // Start the scan of tile (wave j, this CTA): one batch of independent loads.
        auto start_scan = [&](uint32_t j) {
#pragma unroll
            for (int k = 0; k < kMaxWindows; ++k) {
                const uint32_t b = lane + 32u * k;
                pend.d[k] = (b < cta) ? ld_relaxed_u64(desc + static_cast<uint64_t>(j) * G + b) : 1ull;
            }
            pend.prev_wave = (j > 0) ? ld_relaxed_u64(wave_total + (j - 1)) : (static_cast<uint64_t>(G) << kCountShift);
        };
        // Finish it: everything normally arrived long ago; entries that had not been published
        // when the batch was issued are polled (bounded).  Publishes base and offsets to the workers.
        auto finish_scan = [&](uint32_t j) -> bool {
            uint64_t part  = 0;
            uint32_t polls = 0;
            uint64_t t0    = 0;
#pragma unroll
            for (int k = 0; k < kMaxWindows; ++k) {
                const uint32_t b = lane + 32u * k;
                while (__any_sync(kFull, (pend.d[k] & 1ull) == 0)) {
                    PROF_ADD(11, 1);
                    __nanosleep(100);
                    if ((++polls & 255u) == 0) {
                        if (t0 == 0) t0 = now_ns();
                        const bool give_up = (now_ns() - t0 > kWaitNs) || ld_relaxed_u32(abort_flag) != 0;
                        if (__any_sync(kFull, give_up)) return false;
                    }
                    if ((pend.d[k] & 1ull) == 0) pend.d[k] = ld_relaxed_u64(desc + static_cast<uint64_t>(j) * G + b);
                }
                part += pend.d[k] >> 1;
            }
            while ((pend.prev_wave >> kCountShift) != G) {           // uniform: every lane loaded the same word
                PROF_ADD(12, 1);
                __nanosleep(100);
                if ((++polls & 255u) == 0) {
                    if (t0 == 0) t0 = now_ns();
                    if ((now_ns() - t0 > kWaitNs) || ld_relaxed_u32(abort_flag) != 0) return false;
                }
                pend.prev_wave = ld_relaxed_u64(wave_total + (j - 1));
            }
            if (j > 0) waves_before += pend.prev_wave & ((1ull << kCountShift) - 1);
            const uint64_t base = waves_before + warp_sum_u64(part);
            const uint32_t s    = j % kStages;
            const uint64_t t    = tile_of(j);
            if (lane == 0) s_base[s] = base;
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_ready[s]);                 // workers may copy the tile out
            // exclusive count in front of each chunk of this tile
            if (lane < kWarps && (lane % kWarpsPerChunk) == 0) {
                const uint64_t ch = t * kChunksPerTile + lane / kWarpsPerChunk;
                if (ch < chunks_total) a.prefix[ch] = base + pend_chunk_off;
            }
            if (t == num_tiles - 1 && lane == 0) {
                const uint64_t nnz = base + pend_agg;
                *a.nnz_out = nnz;
                __threadfence();
                const bool aborted = ld_relaxed_u32(abort_flag) != 0;
                if (a.dev_status)
                    *a.dev_status = aborted ? BT_ERR_TIMEOUT : (nnz > a.capacity ? BT_ERR_CAPACITY : BT_OK);
            }
            return true;
        };

        uint32_t it = 0;
        for (;; ++it) {
            const uint64_t t64 = tile_of(it);
            if (t64 >= num_tiles) break;
            const uint32_t s = it % kStages;

            PROF_T(c0);
            if (!mbar_wait(&s_counted[s], (it / kStages) & 1u, &s_abort)) {
                failed = true;
                break;
            }
            PROF_T(c1);
            if (lane == 0) DBG_MARK(it, 4, now_ns());
            const uint32_t c   = lane < kWarps ? s_cnt[s][lane] : 0u;
            uint32_t       inc = c;
#pragma unroll
            for (int o = 1; o < kWarps; o <<= 1) {
                const uint32_t u = __shfl_up_sync(kFull, inc, o);
                if (lane >= static_cast<uint32_t>(o)) inc += u;
            }
            const uint32_t agg = __shfl_sync(kFull, inc, kWarps - 1);
            if (lane == 0) {
                st_relaxed_u64(desc + t64, (static_cast<uint64_t>(agg) << 1) | 1ull);
                red_add_u64(wave_total + it, (1ull << kCountShift) + agg);
            }
            if (lane < kWarps) s_off[s][lane] = inc - c;

            // the tile counted one iteration ago: its loads have been in flight since then
            if (it > 0 && !finish_scan(it - 1)) {
                failed = true;
                break;
            }
            if (lane == 0) DBG_MARK(it, 5, now_ns());
            pend_agg       = agg;
            pend_chunk_off = inc - c;
            start_scan(it);
            PROF_T(c2);
            PROF_ADD(8, c1 - c0);
            PROF_ADD(9, c2 - c1);
        }
        if (!failed && it > 0 && !finish_scan(it - 1)) failed = true;
        if (failed && lane == 0) raise_timeout(a.ws_header, a.dev_status, &s_abort);
#ifdef BT_PROFILE
        if (lane == 0)
            for (int k = 8; k < 13; ++k) atomicAdd(reinterpret_cast<unsigned long long *>(a.ws_header) + 8 + k, prof[k]);
#endif
        return;
    }

    // ---------------------------------------------------------------- worker warps
    const uint32_t lt          = lanemask_lt();
    U *const       vals        = static_cast<U *>(a.values);
    const uint64_t words_total = (n + 31) >> 5;
    const uint64_t capacity    = a.capacity;

    for (uint32_t it = 0;; ++it) {
        const uint32_t s   = it % kStages;
        const uint64_t t64 = tile_of(it);

        if (t64 < num_tiles) {
            const uint32_t t     = static_cast<uint32_t>(t64);
            U *const       tile  = tiles + static_cast<size_t>(s) * kTile;
            const uint64_t first = t64 * kTile;
            PROF_T(c0);
            if (!mbar_wait(&s_full[s], (it / kStages) & 1u, &s_abort)) {
                if (lane == 0) raise_timeout(a.ws_header, a.dev_status, &s_abort);
                break;
            }
            PROF_T(c1);
            if (tid == 0) DBG_MARK(it, 0, now_ns());
            if (n - first < static_cast<uint64_t>(kTile)) {
                // ragged last tile: fetch what the 16-byte granular bulk copy left out, zero the rest
                const uint32_t have    = static_cast<uint32_t>(n - first);
                const uint32_t by_bulk = ((have * static_cast<uint32_t>(sizeof(U))) & ~15u) / sizeof(U);
                for (uint32_t e = by_bulk + tid; e < static_cast<uint32_t>(kTile); e += kWorkerThreads)
                    tile[e] = (e < have) ? src[first + e] : U(0);
                asm volatile("bar.sync %0, %1;" ::"n"(kBarWorkers), "n"(kWorkerThreads) : "memory");
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
            if (lane == 0) {
                s_cnt[s][warp] = run;
                mbar_arrive(&s_counted[s]);                   // hand the count to the scan warp
            }
            PROF_T(c2);
            if (tid == 0) DBG_MARK(it, 1, now_ns());
            PROF_ADD(0, c1 - c0);
            PROF_ADD(1, c2 - c1);
        }

        if (it >= static_cast<uint32_t>(kLag)) {
            // ---- copy the packed slots of the tile compacted kLag iterations ago out, contiguous in values[]
            const uint32_t pit = it - kLag;
            if (tile_of(pit) >= num_tiles) {
#ifdef BT_PROFILE
                if (lane == 0 && warp == 0)
                    for (int k = 0; k < 4; ++k)
                        atomicAdd(reinterpret_cast<unsigned long long *>(a.ws_header) + 8 + k, prof[k]);
#endif
                return;                                        // every tile of this CTA is out
            }
            const uint32_t ps = pit % kStages;
            PROF_T(c3);
            if (!mbar_wait(&s_ready[ps], (pit / kStages) & 1u, &s_abort)) break;
            PROF_T(c4);
            if (tid == 0) DBG_MARK(pit, 2, now_ns());
            const U *const pseg = tiles + static_cast<size_t>(ps) * kTile + warp * kWarpElems;
            const uint32_t cnt  = s_cnt[ps][warp];
            const uint64_t dst  = s_base[ps] + s_off[ps][warp];
            if (dst + cnt <= capacity) {
                for (uint32_t j = lane; j < cnt; j += 32) vals[dst + j] = pseg[j];
            } else {
                for (uint32_t j = lane; j < cnt; j += 32)
                    if (dst + j < capacity) vals[dst + j] = pseg[j];
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                if (atomicAdd(&s_done[ps], 1u) == kWarps - 1) {
                    // last warp out of this stage refills it with the tile it holds kStages iterations on
                    __threadfence_block();
                    s_done[ps]        = 0;
                    const uint64_t nt = tile_of(pit + kStages);
                    if (nt < num_tiles) issue_load(ps, static_cast<uint32_t>(nt));
                }
            }
            PROF_T(c5);
            if (tid == 0) DBG_MARK(pit, 3, now_ns());
            PROF_ADD(2, c4 - c3);
            PROF_ADD(3, c5 - c4);
        }
    }

    // ---- only reached when a bounded wait ran out: before leaving, warp 0 lets the bulk copies
    // that may still be in flight into this CTA's shared memory land (bounded, short)
    if (warp == 0)
        for (int s = 0; s < kStages; ++s) {
            mbar_wait<false>(&s_full[s], 0, &s_abort, 20000000ull);
            mbar_wait<false>(&s_full[s], 1, &s_abort, 20000000ull);
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

template <typename U, int RELU_DT, bool WRITE_Y, int kWarps, int kStages, int kLag>
cudaError_t launch_shaped(const CompressArgs &a, cudaStream_t stream)
{
    constexpr int kTile    = kWarps * kWarpElems;
    constexpr int kThreads = kWarps * 32 + 32;
    constexpr size_t kSmem = static_cast<size_t>(kStages) * kTile * sizeof(U);
    static LaunchShape shape;   // one per instantiation
    auto kernel = compress_kernel<U, RELU_DT, WRITE_Y, kWarps, kStages, kLag>;

    const uint32_t num_tiles = static_cast<uint32_t>((a.n + kTile - 1) / kTile);
    int            max_grid  = 0;
    cudaError_t    e         = shape.max_grid(kernel, kThreads, kSmem, max_grid);
    if (e != cudaSuccess) return e;
    if (max_grid > 32 * kMaxWindows) max_grid = 32 * kMaxWindows;
    const uint32_t grid  = num_tiles < static_cast<uint32_t>(max_grid) ? num_tiles : static_cast<uint32_t>(max_grid);
    const uint32_t waves = (num_tiles + grid - 1) / grid;
    // abort flag, wave totals and tile descriptors start at zero
    e = cudaMemsetAsync(a.ws_header, 0, kWsHeaderBytes + 8 * (static_cast<size_t>(num_tiles) + waves), stream);
    if (e != cudaSuccess) return e;
    // cooperative launch: the runtime guarantees that all `grid` CTAs are resident together
    CompressArgs args = a;
    args.ws_waves     = waves;
    uint32_t     nt   = num_tiles;
    void *params[] = {&args, &nt};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(kThreads), params, kSmem,
                                       stream);
}

template <typename U, int RELU_DT, bool WRITE_Y>
cudaError_t launch_typed(const CompressArgs &a, cudaStream_t stream)
{
    static const int cfg = [] { const char *e = getenv("BT_CFG"); return e ? atoi(e) : 0; }();
    constexpr int B = sizeof(U) == 4 ? 1 : 2;   // 16-bit tiles are half the bytes: room for twice the stages
    switch (cfg) {
    case 1: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 6 * B, 2>(a, stream);      // 1 CTA/SM, 3 loading
    case 2: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 6 * B, 3>(a, stream);      // 1 CTA/SM, lag 3
    case 3: return launch_shaped<U, RELU_DT, WRITE_Y, 4, 6 * B, 2>(a, stream);      // 2 CTAs/SM
    case 4: return launch_shaped<U, RELU_DT, WRITE_Y, 4, 4 * B, 2>(a, stream);      // 3 CTAs/SM
    case 5: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 7 * B, 2>(a, stream);      // 1 CTA/SM, 4 loading
    case 6: return launch_shaped<U, RELU_DT, WRITE_Y, 4, 7 * B, 3>(a, stream);      // 2 CTAs/SM, lag 3
    default: return launch_shaped<U, RELU_DT, WRITE_Y, 8, 5 * B, 2>(a, stream);     // 1 CTA/SM, 2 loading
    }
}

}  // namespace

#ifdef BT_PROFILE
extern "C" int bt_debug_set_buffer(void *buf, unsigned int it0)
{
    unsigned long long *p = static_cast<unsigned long long *>(buf);
    if (cudaMemcpyToSymbol(g_dbg, &p, sizeof(p)) != cudaSuccess) return 1;
    return cudaMemcpyToSymbol(g_dbg_it0, &it0, sizeof(it0)) != cudaSuccess;
}
#endif

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
