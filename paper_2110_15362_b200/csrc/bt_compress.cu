// Algorithm 1 (dense -> bitmap) and its fused forms (ReLU, activation pruning) as ONE
// compaction pass: a persistent-CTA stream compaction whose prefix sum rides on the
// wave structure of the grid.
//
// The grid is launched cooperatively with exactly as many CTAs (G) as fit on
// the device at once, so all of them are co-resident, and CTA b takes tiles
// b, b+G, b+2G, ...: iteration j of every CTA together forms "wave j", G
// consecutive tiles.  The warps of a CTA are specialised: one load warp,
// kWarps compactor warps, two scan warps, kCopiers copier warps.
//
// Compaction.  Compactor warp w owns segment w (1024 elements) of the tile:
//
//   step k:  lane l reads element 32k+l (conflict-free shared load);
//            ballot(non-zero) IS bitmap word k (LSB first), kept by lane k;
//            the number of ballot bits below the lane is the lane's rank;
//            non-zero lanes store the element at [run + rank] of the same
//            segment -- in place: the write position never passes the read
//            position, and a batch's loads are issued before the previous
//            batch's stores;
//            run += popc(ballot).
//
// After 32 steps the segment's first `run` entries hold the packed values and
// lane k holds bitmap word k: one coalesced 128-byte bitmap store per warp.
//
// Prefix.  The exclusive base of tile (wave j, CTA b) is
//     sum of the totals of waves 0..j-1  +  sum of the counts of CTAs 0..b-1 in wave j.
// As soon as a tile is counted a scan warp publishes the count in a descriptor
// and adds it (with a 1 in a counter field) to the wave's total with one
// fire-and-forget reduction.  About one tile later -- when every CTA has
// published wave j -- it reads the b descriptors of its wave and the now
// complete totals of the waves before it in ONE batch of independent loads,
// and uses them a tile after that.  The two scan warps alternate tiles, so
// that each has two tiles' time for that round trip to L2.  No tile waits on
// another tile's base: only on counts, which never wait on anything but data.
//
// Pipeline.  The warps of a CTA never meet at a CTA-wide barrier after the
// prologue; a ring slot goes round through four mbarriers:
//   full[s]     the bulk copy of the tile has landed         (copy engine -> compactors)
//   counted[s]  every compactor has posted its count         (compactors  -> scan warps)
//   ready[s]    base and segment offsets are in shared       (scan warp   -> copiers)
//   empty[s]    every copier has copied its segments out     (copiers     -> load warp)
// Copier warp c copies its segments' packed values to values[base + offset ...]
// (2-byte values through the copy engine, in 16-byte units: copy_out_run16).
// With a ring of 7 tiles the load warp runs several tiles ahead of the
// compactors and the compactors several tiles ahead of the copiers, so nobody
// waits for a round trip to L2 or to HBM.
//
// Workspace.  It arrives with unspecified contents and is not cleared.  A tile's
// descriptor carries the launch's 64-bit tag in both of its halves, and a reader
// takes only descriptors with its own launch's tag; so counts are published and
// read from the first tile on.  Only the wave totals, being sums, need zeroed
// words: in the prologue every CTA zeroes a share of them and the grid meets
// once (cooperative_groups::this_grid().sync()), the first two bulk copies
// already on their way; nothing reads or adds to a total before that meeting.
// A launch of one wave has no totals and no meeting.
#include <cooperative_groups.h>

#include <atomic>
#include <chrono>

#include "bt_compress_common.cuh"

namespace bt {
namespace {

using namespace cmp;

// U: uint32_t (4-byte elements) or uint16_t (2-byte elements).
// RELU_DT: -1 for the plain compressor, else the number of the fused forward form (element type, + 4 for ReLU6).
// CAST: 0, or the 16-bit type the copiers narrow the packed binary32 values to (1 binary16, 2 bfloat16).
// A tile is kWarps segments of kSeg elements; kCompactors compactor warps take the CTA's segments in turn
// (segment g of the CTA's stream of tiles goes to warp g mod kCompactors; with kCompactors == kWarps warp w
// simply owns segment w of every tile), kCopiers copier warps, kStages ring slots.
template <typename U, int RELU_DT, bool WRITE_Y, int CAST, int kWarps, int kSeg, int kStages, int kCopiers, int kCompactors = kWarps>
__global__ void __launch_bounds__((kCompactors + kCopiers + 3) * 32) compress_kernel(const CompressArgs a, const uint32_t num_tiles)
{
    constexpr int kTile          = kWarps * kSeg;
    constexpr int kSteps         = kSeg / 32;
    constexpr int kChunksPerTile = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk = BT_CHUNK_ELEMS / kSeg;
    // warp roles
    constexpr int kFirstCopier = kCompactors;
    constexpr int kScanWarp    = kCompactors + kCopiers;  // and kScanWarp + 1
    constexpr int kLoadWarp    = kCompactors + kCopiers + 2;
    constexpr int kSegsPerCopier = kWarps / kCopiers;
    static_assert(kWarps % kCopiers == 0, "equal shares for the copier warps");
    static_assert(kSeg % 32 == 0 && kSeg <= 1024 && BT_CHUNK_ELEMS % kSeg == 0, "segments tile a chunk");
    static_assert(kTile % BT_CHUNK_ELEMS == 0, "a tile holds whole chunks");
    static_assert(kWarps <= 32, "one lane per warp count");
    // A scan warp makes tile j ready only in its turn for tile j + 2, after that tile has been counted, so
    // tiles j, j + 1 and j + 2 must hold slots at once: three stages are the minimum that cannot deadlock,
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
    __shared__ volatile uint32_t s_abort;
    __shared__ volatile uint64_t s_tag;                    // this launch's tag once a scan warp has it, else 0
    __shared__ uint64_t          s_arena_c0;               // arena forms: the cursor as this launch found it

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    // broadcast from lane 0 so that the compiler knows the role branches below are warp-uniform and may keep
    // warp-uniform values (ballots, their counts, the running output position) on the uniform datapath
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);
    const uint32_t G    = gridDim.x;
    const uint32_t cta  = blockIdx.x;
    const U *const src  = static_cast<const U *>(a.src);
    const uint64_t n    = a.n;
    const uint64_t wait_ns = a.wait_ns;          // bound of every wait below

    // tile of iteration `it` of this CTA (64-bit so that running past the end cannot wrap)
    auto tile_of = [&](uint32_t it) { return cta + static_cast<uint64_t>(it) * G; };

    if (tid == 0) {
        // Read before the barrier below: the kernel's one update of the cursor follows the last tile's base,
        // which needs a publication from every CTA, and a CTA publishes only after this barrier.
        s_arena_c0 = a.arena_cursor ? *reinterpret_cast<const volatile uint64_t *>(a.arena_cursor) : 0;
        s_abort    = 0;
        s_tag      = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&s_full[s], 1);
            mbar_init(&s_counted[s], kWarps);
            mbar_init(&s_ready[s], 1);
            mbar_init(&s_empty[s], kCopiers);
        }
        fence_proxy_async();
    }
    __syncthreads();

    // bulk copy of tile `it` of this CTA into its ring slot (issued by lane 0 of the load warp)
    auto issue_load = [&](const uint32_t it) {
        const uint32_t s     = it % kStages;
        const uint64_t first = tile_of(it) * kTile;
        const uint64_t left  = n - first;
        const uint32_t valid = left < static_cast<uint64_t>(kTile) ? static_cast<uint32_t>(left) : kTile;
        const uint32_t bytes = (valid * static_cast<uint32_t>(sizeof(U))) & ~15u;   // whole 16-byte units
        fence_proxy_async();                       // the copiers' and compactors' accesses to the slot come first
        mbar_arrive_expect_tx(&s_full[s], bytes);  // bytes == 0 simply completes the phase
        if (bytes) bulk_load(tiles + static_cast<size_t>(s) * kTile, src + first, bytes, &s_full[s]);
    };

    // More than one wave: the wave totals are sums made by reductions, so their words must be zero before the first
    // count is added.  Every CTA zeroes a share and the grid meets once, here, before any warp takes up its role;
    // the first two bulk copies are on their way meanwhile, so the meeting costs a launch next to nothing.
    const bool     multi  = num_tiles > G;
    // the part of the workspace behind its header, as large as the size query promises the caller
    const Extent   wsx    = extent_of(a.ws_desc, compress_workspace_bytes((n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS) - kWsHeaderBytes);
    uint32_t       it_pre = 0;                    // bulk copies issued before the meeting
    if (multi) {
        if (warp == kLoadWarp && lane == 0) {
            for (; it_pre < 2u && tile_of(it_pre) < num_tiles; ++it_pre) issue_load(it_pre);
        }
        for (uint32_t i = cta * blockDim.x + tid; i < a.ws_waves; i += G * blockDim.x)
            if (wsx.holds(a.ws_desc + i, 8)) a.ws_desc[i] = 0;
        cooperative_groups::this_grid().sync();
    }

    if (warp == kLoadWarp) {
        // ------------------------------------------------------------ load warp (one lane)
        if (lane == 0) {
            bool     ok     = true;
            uint32_t issued = it_pre;
            for (uint32_t it = it_pre; ok; ++it) {
                if (tile_of(it) >= num_tiles) break;
                if (it >= static_cast<uint32_t>(kStages)) {
                    ok = mbar_wait(&s_empty[it % kStages], ((it / kStages) - 1) & 1u, &s_abort, wait_ns);
                    if (!ok) break;
                }
                // Start-up pacing: at most two bulk copies outstanding per SM while the ring fills for the first
                // time, as in steady state, where a copy is issued only as a slot frees.  Requesting the whole ring
                // at once puts 33 MB in front of every other memory operation of the first microseconds -- the
                // grid meeting and the first reads of the counts then take 5 us and more instead of 1.3, and the
                // ring runs full waiting for the first base (a 26 MB layer: 34.1 -> 31.3 us per call).
                if (it >= 2u && it < static_cast<uint32_t>(kStages)) mbar_wait<false>(&s_full[(it - 2u) % kStages], 0, &s_abort, wait_ns);
                issue_load(it);
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
        // Two warps share the scan: warp p takes this CTA's tiles p, p + 2, p + 4, ...  A warp's turn for
        // tile j is
        //   (a) wait until the compactors have counted tile j, publish the count,
        //   (c) finish tile j - 2 (its own previous tile) from the loads of its previous turn and hand it
        //       to the copiers,
        //   (b) wait until tile j + 1 is counted -- about one tile later, when every CTA has published
        //       wave j -- and issue, in ONE batch of independent loads, the reads of the descriptors of
        //       wave j and of the totals of waves j - 1 and j - 2.
        // The loads of (b) are used a whole tile later, in (c) of the next turn, so the round trip to L2
        // (1.3 us under load, longer than one tile) never stalls a turn for long: a turn has two tiles' time.
        // (One warp doing every tile cannot hide that round trip however deep its software pipeline is:
        // its loads of consecutive tiles retire through the same scoreboard.)
        const uint32_t  p            = warp - kScanWarp;
        uint64_t *const wave_total   = a.ws_desc;                  // one word per wave
        uint64_t *const desc         = a.ws_desc + a.ws_waves;     // two words per tile
        const uint64_t  chunks_total = (n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS;
        const uint32_t  last_it      = static_cast<uint32_t>((num_tiles - 1 - cta) / G);   // this CTA's last iteration
        uint64_t        waves_before = 0;    // sum of the totals of the waves before this warp's previous tile
        bool            failed       = false;

        // The tag of this launch.  Both scan warps read the same sequence number: it changes only once every CTA
        // has published all its counts, or two seconds into a failure.
        uint64_t seq = 0;
        if (lane == 0) seq = ld_relaxed_u64(a.ws_header + kHdrSeq);
        seq                   = __shfl_sync(kFull, seq, 0);
        const uint64_t tag    = mix64(a.call_tag + seq * 0x9E3779B97F4A7C15ull) | 1ull;
        const uint64_t tag_w0 = tag & 0xFFFFFFFF00000000ull, tag_w1 = tag << 32;
        if (p == 0 && lane == 0) s_tag = tag;
        auto valid = [&](const uint64_t w0, const uint64_t w1) {
            return ((w0 ^ tag_w0) >> 32) == 0 && ((w1 ^ tag_w1) >> 32) == 0 && static_cast<uint32_t>(w0) == static_cast<uint32_t>(w1);
        };

        // d0[k], d1[k], lane l <-> descriptor of CTA l + 32k of the wave of this warp's previous tile;
        // w1, w2: total words of the one and the two waves before it
        uint64_t d0[kMaxWindows], d1[kMaxWindows], w1 = 0, w2 = 0;
#pragma unroll
        for (int k = 0; k < kMaxWindows; ++k) d0[k] = tag_w0, d1[k] = tag_w1;

        for (uint32_t j = p; !failed && j <= last_it + 2; j += 2) {
            if (j <= last_it) {
                // ---- (a)
                const uint32_t s = j % kStages;
                if (!mbar_wait(&s_counted[s], (j / kStages) & 1u, &s_abort, wait_ns)) {
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
                    if (wsx.holds(desc + 2 * tile_of(j), 16)) st_relaxed_2xu64(desc + 2 * tile_of(j), tag_w0 | agg, tag_w1 | agg);
                    s_agg[s] = agg;
                }
                if (lane < kWarps) s_off[s][lane] = inc - c;
                if (multi && lane == 0 && wsx.holds(wave_total + j, 8)) red_add_u64(wave_total + j, (1ull << kCountShift) + agg);
            }
            if (j >= 2) {
                // ---- (c): tile j - 2 <= last_it
                const uint32_t f     = j - 2;
                uint32_t       polls = 0;
                uint64_t       t0    = 0;
                for (;;) {
                    bool missing = (f > 0 && (w1 >> kCountShift) != G) || (f > 1 && (w2 >> kCountShift) != G);
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k) missing |= !valid(d0[k], d1[k]);
                    if (!__any_sync(kFull, missing)) break;
                    __nanosleep(100);
                    if ((++polls & 255u) == 0 || (kTestHooks && wait_ns < kStrictLimitNs)) {
                        if (t0 == 0) t0 = now_ns();
                        if (__any_sync(kFull, (now_ns() - t0 > wait_ns) || ld_relaxed_u64(a.ws_header + kHdrAbort) == tag)) {
                            failed = true;
                            break;
                        }
                    }
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k)
                        if (!valid(d0[k], d1[k]))
                            ld_relaxed_2xu64(desc + 2 * (static_cast<uint64_t>(f) * G + lane + 32u * k), d0[k], d1[k]);
                    if (f > 0 && (w1 >> kCountShift) != G) w1 = ld_relaxed_u64(wave_total + (f - 1));
                    if (f > 1 && (w2 >> kCountShift) != G) w2 = ld_relaxed_u64(wave_total + (f - 2));
                }
                if (failed) break;
                uint64_t part = 0;
#pragma unroll
                for (int k = 0; k < kMaxWindows; ++k) part += static_cast<uint32_t>(d0[k]);
                // the waves in front of tile f: those in front of tile f - 2, and waves f - 2 and f - 1
                waves_before += (w1 & ((1ull << kCountShift) - 1)) + (w2 & ((1ull << kCountShift) - 1));
                const uint64_t base = waves_before + warp_sum_u64(part);
                const uint32_t ps   = f % kStages;
                const uint64_t pt   = tile_of(f);
                // exclusive count in front of each chunk of that tile
                if (lane < kWarps && (lane % kWarpsPerChunk) == 0) {
                    const uint64_t ch = pt * kChunksPerTile + lane / kWarpsPerChunk;
                    if (ch < chunks_total && extent_of(a.prefix, 8 * chunks_total).holds(a.prefix + ch, 8)) a.prefix[ch] = base + s_off[ps][lane];
                }
                if (pt == num_tiles - 1 && lane == 0) {
                    const uint64_t nnz = base + s_agg[ps];
                    *a.nnz_out = nnz;
                    __threadfence();
                    const bool aborted = ld_relaxed_u64(a.ws_header + kHdrAbort) == tag;
                    uint64_t capacity = a.capacity;
                    if (a.arena_cursor) {
                        // arena form: the room left behind the cursor; the cursor moves only when everything fitted
                        const uint64_t c0 = s_arena_c0;
                        capacity          = c0 <= a.arena_bytes ? (a.arena_bytes - c0) / sizeof(Stored<CAST, U>) : 0;
                        if (!aborted && nnz <= capacity) {
                            *a.values_offset_out = c0;
                            *a.arena_cursor      = c0 + ((nnz * sizeof(Stored<CAST, U>) + 15) & ~15ull);
                        }
                    }
                    if (a.dev_status)
                        *a.dev_status = aborted ? BT_ERR_TIMEOUT : (nnz > capacity ? BT_ERR_CAPACITY : BT_OK);
                    // every CTA has published all its counts by now, so every CTA has read the sequence number:
                    // the next launch on this workspace gets another tag
                    red_add_u64(a.ws_header + kHdrSeq, 1ull);
                }
                __syncwarp();
                if (lane == 0) {
                    s_base[ps] = base;
                    mbar_arrive(&s_ready[ps]);                       // the copiers may take the tile
                }
            }
            if (j <= last_it) {
                // ---- (b): a tile later (when the other scan warp's next tile is counted, if there is one)
                if (j + 1 > last_it) {
                    // This CTA's last tile: no next tile to wait for.  A short pause gives the other counts of the
                    // wave time to land, so that the reads below usually succeed at once instead of costing a second
                    // round trip (cold ResNet-shaped forward passes: -5 %; reading at once and polling was slower).
                    __nanosleep(300);
                } else if (!mbar_wait(&s_counted[(j + 1) % kStages], ((j + 1) / kStages) & 1u, &s_abort, wait_ns)) {
                    failed = true;
                    break;
                }
#pragma unroll
                for (int k = 0; k < kMaxWindows; ++k) {
                    const uint32_t b = lane + 32u * k;
                    if (b < cta) ld_relaxed_2xu64(desc + 2 * (static_cast<uint64_t>(j) * G + b), d0[k], d1[k]);
                    else d0[k] = tag_w0, d1[k] = tag_w1;             // not in front of this CTA: a valid count of 0
                }
                w1 = (j > 0) ? ld_relaxed_u64(wave_total + (j - 1)) : 0ull;
                w2 = (j > 1) ? ld_relaxed_u64(wave_total + (j - 2)) : 0ull;
            }
        }
        if (failed && lane == 0) raise_timeout(a.ws_header, a.dev_status, &s_abort, s_tag);
        return;
    }

    if (warp >= kFirstCopier) {
        // ------------------------------------------------------------ copier warps
        const uint32_t copier   = warp - kFirstCopier;
        using V                 = Stored<CAST, U>;
        V             *vals     = static_cast<V *>(a.values);
        uint64_t       capacity = a.capacity;
        if (a.arena_cursor) {
            const uint64_t c0 = s_arena_c0;
            vals              = reinterpret_cast<V *>(static_cast<unsigned char *>(a.values) + c0);
            capacity          = c0 <= a.arena_bytes ? (a.arena_bytes - c0) / sizeof(V) : 0;
        }
        const Extent vx = extent_of(vals, capacity * sizeof(V));
        constexpr bool kBulk = kBulkCopyOut16 && sizeof(U) == 2 && CAST == 0;   // 2-byte runs leave through the copy engine
        for (uint32_t it = 0;; ++it) {
            if (tile_of(it) >= num_tiles) break;
            const uint32_t s = it % kStages;
            if (!mbar_wait(&s_ready[s], (it / kStages) & 1u, &s_abort, wait_ns)) break;
            const uint64_t base = s_base[s];
#pragma unroll
            for (int q = 0; q < kSegsPerCopier; ++q) {
                const uint32_t seg  = copier * kSegsPerCopier + q;
                U *const       pseg = tiles + static_cast<size_t>(s) * kTile + seg * kSeg;
                const uint32_t cnt  = s_cnt[s][seg];
                const uint64_t dst  = base + s_off[s][seg];
                if (dst + cnt <= capacity) {
                    if constexpr (kBulk) copy_out_run16(pseg, lane, cnt, vals + dst, vx);
                    else copy_out_segment<U, CAST, false>(pseg, lane, cnt, vals + dst, 0, vx);
                } else {
                    copy_out_segment<U, CAST, true>(pseg, lane, cnt, vals + dst, dst < capacity ? capacity - dst : 0, vx);
                }
            }
            if constexpr (kBulk) {
                if (lane == 0) bulk_store_wait_read();            // the copy engine has read the segments
            }
            __syncwarp();
            asm volatile("" ::: "memory");        // the copy-out stays above the release of the slot
            if (lane == 0) mbar_arrive(&s_empty[s]);
        }
        return;
    }

    // ---------------------------------------------------------------- compactor warps
    const uint64_t words_total = (n + 31) >> 5;
    const Extent   bx          = extent_of(a.bitmap, 4 * words_total);
    const Extent   yx          = extent_of(a.y, n * sizeof(U));
    for (uint32_t g = warp;; g += kCompactors) {
        const uint32_t it  = g / kWarps;              // iteration (tile of this CTA) and segment of it
        const uint32_t seg = g % kWarps;
        const uint64_t t64 = tile_of(it);
        if (t64 >= num_tiles) break;
        const uint32_t s     = it % kStages;
        const uint32_t t     = static_cast<uint32_t>(t64);
        U *const       tile  = tiles + static_cast<size_t>(s) * kTile;
        const uint64_t first = t64 * kTile;
        if (!mbar_wait(&s_full[s], (it / kStages) & 1u, &s_abort, wait_ns)) {
            if (lane == 0) raise_timeout(a.ws_header, a.dev_status, &s_abort, s_tag);
            break;
        }
        if (n - first < static_cast<uint64_t>(kTile)) {
            // Ragged last tile: each warp completes its own segment -- what the 16-byte granular bulk copy left out,
            // zeros behind the end of the tensor -- and meets no other warp over it.  (A barrier among the compactor
            // warps here would never open if one of them had left the kernel because its wait ran out.)
            const uint32_t have    = static_cast<uint32_t>(n - first);
            const uint32_t by_bulk = ((have * static_cast<uint32_t>(sizeof(U))) & ~15u) / sizeof(U);
            const uint32_t seg0    = seg * kSeg;
            for (uint32_t e = (by_bulk > seg0 ? by_bulk : seg0) + lane; e < seg0 + kSeg; e += 32)
                tile[e] = (e < have) ? src[first + e] : U(0);
            __syncwarp();
        }

        // ---- in-place compaction of this warp's segment
        const uint64_t e0     = first + seg * kSeg;                 // first element of the segment
        uint32_t       yvalid = 0;
        U             *y      = nullptr;
        if constexpr (WRITE_Y) {
            y      = static_cast<U *>(a.y) + e0;
            yvalid = e0 + kSeg <= n ? static_cast<uint32_t>(kSeg) : (e0 < n ? static_cast<uint32_t>(n - e0) : 0u);
        }
        const uint32_t seg_addr = smem_addr(tile + seg * kSeg);
        uint32_t       run, word;
        if (!WRITE_Y || yvalid == static_cast<uint32_t>(kSeg))   // all but a ragged last tile: no bounds checks on y
            run = compact_segment<U, RELU_DT, WRITE_Y, false, kSteps>(seg_addr, word, lane, y, yvalid, a.tau, yx);
        else
            run = compact_segment<U, RELU_DT, WRITE_Y, true, kSteps>(seg_addr, word, lane, y, yvalid, a.tau, yx);
        if (lane < kSteps) {
            const uint64_t w = static_cast<uint64_t>(t) * (kTile / 32) + seg * kSteps + lane;
            if (w < words_total && bx.holds(a.bitmap + w, 4)) a.bitmap[w] = word;
        }
        __syncwarp();
        if (lane == 0) {
            s_cnt[s][seg] = run;
            mbar_arrive(&s_counted[s]);                   // hand the count to the scan warp
        }
    }
}

}  // namespace

// A value no other call of this process gets: a counter that starts at a salt drawn from the clock and the
// address space, so that words left in recycled memory by another run of the library do not line up either.
uint64_t next_call_tag()
{
    static std::atomic<uint64_t> counter{
        cmp::mix64(static_cast<uint64_t>(std::chrono::steady_clock::now().time_since_epoch().count()) ^
                   cmp::mix64(reinterpret_cast<uintptr_t>(&counter)))};
    return counter.fetch_add(1, std::memory_order_relaxed);
}

// The calling thread's limit on the CTAs of one compress launch (0: none).  A cooperative launch needs all its
// CTAs resident at once and a CTA of this kernel fills an SM, so two launches of more than half the SMs each run
// one after the other even on different streams; a caller that keeps several launches in flight gives each a
// share of the SMs.
thread_local uint32_t t_max_ctas = 0;
uint32_t compress_max_ctas() { return t_max_ctas; }
uint32_t set_compress_max_ctas(uint32_t max_ctas)
{
    const uint32_t before = t_max_ctas;
    t_max_ctas            = max_ctas;
    return before;
}

// The bound of the kernels' waits; only a test build can change it.
std::atomic<uint64_t> g_wait_ns{kDefaultWaitNs};
uint64_t compress_wait_ns() { return g_wait_ns.load(std::memory_order_relaxed); }
uint64_t set_compress_wait_ns(uint64_t wait_ns) { return g_wait_ns.exchange(wait_ns, std::memory_order_relaxed); }

namespace {

template <typename U, int RELU_DT, bool WRITE_Y, int CAST, int kWarps, int kSeg, int kStages, int kCopiers, int kCompactors = kWarps>
cudaError_t launch_shaped(const CompressArgs &a, cudaStream_t stream)
{
    constexpr int kTile    = kWarps * kSeg;
    constexpr int kThreads = (kCompactors + kCopiers + 3) * 32;
    constexpr size_t kSmem = static_cast<size_t>(kStages) * kTile * sizeof(U);
    static LaunchShape shape;   // one per instantiation
    auto kernel = compress_kernel<U, RELU_DT, WRITE_Y, CAST, kWarps, kSeg, kStages, kCopiers, kCompactors>;

    const uint32_t num_tiles = static_cast<uint32_t>((a.n + kTile - 1) / kTile);
    int            max_grid  = 0;
    cudaError_t    e         = shape.max_grid(kernel, kThreads, kSmem, max_grid);
    if (e != cudaSuccess) return e;
    if (max_grid > 32 * kMaxWindows) max_grid = 32 * kMaxWindows;
    if (t_max_ctas != 0 && static_cast<uint32_t>(max_grid) > t_max_ctas) max_grid = static_cast<int>(t_max_ctas);
    const uint32_t grid  = num_tiles < static_cast<uint32_t>(max_grid) ? num_tiles : static_cast<uint32_t>(max_grid);
    const uint32_t waves = (num_tiles + grid - 1) / grid;
    // cooperative launch: the runtime guarantees that all `grid` CTAs are resident together
    CompressArgs args = a;
    args.ws_waves     = (waves + 1) & ~1u;            // an even number of total words keeps the descriptors 16-byte aligned
    args.call_tag     = next_call_tag();
    args.wait_ns      = compress_wait_ns();
    uint32_t     nt   = num_tiles;
    void *params[] = {&args, &nt};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(kThreads), params, kSmem,
                                       stream);
}

template <typename U, int RELU_DT, bool WRITE_Y, int CAST = 0>
cudaError_t launch_typed(const CompressArgs &a, cudaStream_t stream)
{
    // One CTA per SM, the ring takes nearly all of its shared memory.
    //   8-byte elements: 8 compactor warps x 512 elements (32 KB tiles), 8 copiers, 7 stages;
    //   4-byte elements: 8 compactor warps x 1024 elements (32 KB tiles), 8 copiers, 7 stages;
    //   2-byte elements: 16 compactor warps x 1024 elements (32 KB tiles), 8 copiers, 7 stages --
    //   a 2-byte tile takes as many compaction steps per byte again, so it gets twice the warps.
    //   (More compactor warps than segments, taking segments in turn -- 18, 20, 21 or 24 with 8 or 4 copiers --
    //   measured slower on the 392 MiB bf16 tensor: 0.151-0.161 ms against 0.1485; with fewer than 8 copiers the
    //   copy-out falls behind: 0.19 ms with 4, 0.29 with 2.)
    if constexpr (sizeof(U) == 8) return launch_shaped<U, RELU_DT, WRITE_Y, CAST, 8, 512, 7, 8>(a, stream);
    else if constexpr (sizeof(U) == 4) return launch_shaped<U, RELU_DT, WRITE_Y, CAST, 8, 1024, 7, 8>(a, stream);
    else return launch_shaped<U, RELU_DT, WRITE_Y, CAST, 16, 1024, 7, 8>(a, stream);
}

}  // namespace

cudaError_t launch_compress(const CompressArgs &a, int dtype, int fused, cudaStream_t stream)
{
    // fused: 0 plain compressor, 1 threshold form (ReLU at tau = 0), 2 ReLU6
    const bool y = a.y != nullptr;
    if (a.cast != 0) {
        // down-cast on stash: binary32 tensors, plain and threshold forms
        if (dtype != BT_F32 || fused == 2) return cudaErrorInvalidValue;
        const bool h = a.cast == BT_F16;
        if (fused == 0) return h ? launch_typed<uint32_t, -1, false, 1>(a, stream) : launch_typed<uint32_t, -1, false, 2>(a, stream);
        if (y) return h ? launch_typed<uint32_t, BT_F32, true, 1>(a, stream) : launch_typed<uint32_t, BT_F32, true, 2>(a, stream);
        return h ? launch_typed<uint32_t, BT_F32, false, 1>(a, stream) : launch_typed<uint32_t, BT_F32, false, 2>(a, stream);
    }
    if (fused == 0) {
        return dtype == BT_F64   ? launch_typed<uint64_t, -1, false>(a, stream)
               : dtype == BT_F32 ? launch_typed<uint32_t, -1, false>(a, stream)
                                 : launch_typed<uint16_t, -1, false>(a, stream);
    }
    constexpr int k6 = kFusedRelu6;
    if (fused == 2) {
        switch (dtype) {
        case BT_F64:
            return y ? launch_typed<uint64_t, k6 + BT_F64, true>(a, stream) : launch_typed<uint64_t, k6 + BT_F64, false>(a, stream);
        case BT_F32:
            return y ? launch_typed<uint32_t, k6 + BT_F32, true>(a, stream) : launch_typed<uint32_t, k6 + BT_F32, false>(a, stream);
        // 2-byte types: the decisions by compares in the element's own type
        case BT_F16:
            return y ? launch_typed<uint16_t, kFusedRelu6Half + BT_F16, true>(a, stream) : launch_typed<uint16_t, kFusedRelu6Half + BT_F16, false>(a, stream);
        default:
            return y ? launch_typed<uint16_t, kFusedRelu6Half + BT_BF16, true>(a, stream)
                     : launch_typed<uint16_t, kFusedRelu6Half + BT_BF16, false>(a, stream);
        }
    }
    if (a.tau == 0.0f && (dtype == BT_F16 || dtype == BT_BF16)) {
        // The ReLU itself on a 2-byte type: decided by one compare in the element's own type (on the 392 MiB tensor
        // 0.165 -> 0.138 ms without the dense output, together with the multiply-add forms of the compaction step).
        constexpr int kh = kFusedReluHalf;
        if (dtype == BT_F16) return y ? launch_typed<uint16_t, kh + BT_F16, true>(a, stream) : launch_typed<uint16_t, kh + BT_F16, false>(a, stream);
        return y ? launch_typed<uint16_t, kh + BT_BF16, true>(a, stream) : launch_typed<uint16_t, kh + BT_BF16, false>(a, stream);
    }
    switch (dtype) {
    case BT_F64:
        return y ? launch_typed<uint64_t, BT_F64, true>(a, stream) : launch_typed<uint64_t, BT_F64, false>(a, stream);
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
