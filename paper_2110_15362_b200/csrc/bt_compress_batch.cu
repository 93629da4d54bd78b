// The batched forms of Algorithm 1 and of its fused ReLU form: the tensors of a batch in ONE launch of the
// persistent compaction kernel (bt_compress.cu describes the pipeline of a CTA, the compaction and the scan).
//
// What a batch adds.  The tiles of all tensors are dealt round robin to the same resident grid: tile t of
// tensor k goes to CTA (rot_k + t) mod G, where rot_k continues the deal of the tensor before it, so every CTA
// gets the same share of the batch whatever the tensors' sizes.  The prefix restarts at every tensor: inside
// tensor k, tiles [jG, (j+1)G) form "wave j", and the exclusive base of tile (k, j, v) -- v the CTA's place in
// the deal of tensor k -- is
//     sum of the totals of waves 0..j-1 of tensor k  +  sum of the counts of places 0..v-1 in wave j of tensor k.
// Every tensor has its own wave totals and descriptors in the workspace and gets exactly the bitmap, values,
// chunk prefix, count and status the single-tensor call would give it.  A step that stashes many activations of
// a few megabytes pays the fixed cost of a launch (load, compact, exchange counts, copy out: each a memory round
// trip) once per batch instead of once per tensor.
#include <cooperative_groups.h>

#include "bt_compress_common.cuh"

namespace bt {
namespace {

using namespace cmp;

template <int kJobs>
struct CompressParams {
    CompressCommon c;
    CompressJob    job[kJobs];
};

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
        const uint32_t rot = p.job[w.k].rot;
        w.tiles            = p.job[w.k].tiles;
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
// kJobs: room for tensors in the kernel's parameters (1, or kMaxBatch for the batched forms).
// kWarps compactor warps, kSeg elements per warp, kStages ring slots, kCopiers copier warps.
template <typename U, int FUSED, bool WRITE_Y, int kJobs, int kWarps, int kSeg, int kStages, int kCopiers>
__global__ void __launch_bounds__((kWarps + kCopiers + 3) * 32)
compress_kernel(const __grid_constant__ CompressParams<kJobs> p)
{
    constexpr int kTile           = kWarps * kSeg;
    constexpr int kChunksPerTile  = kTile / BT_CHUNK_ELEMS;
    constexpr int kWarpsPerChunk  = BT_CHUNK_ELEMS / kSeg;
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
    __shared__ uint64_t          s_dst[kStages];           // arena form: byte offset of the tile's tensor in the arena
    __shared__ uint64_t          s_arena_c0;               // arena form: the cursor as the launch found it
    __shared__ uint32_t          s_cnt[kStages][kWarps];   // packed count of each segment
    __shared__ uint32_t          s_off[kStages][kWarps];   // exclusive offset of each segment in the tile
    __shared__ uint32_t          s_agg[kStages];           // packed count of the tile
    __shared__ __align__(16) unsigned char s_bits[kWarps][kSeg / 8];   // bitmap bytes of the segment a warp is compacting
    __shared__ volatile uint32_t s_abort;
    __shared__ volatile uint64_t s_tag;                    // this launch's tag once the first scan warp has it, else 0

    const uint32_t tid  = threadIdx.x;
    const uint32_t lane = tid & 31u;
    // broadcast from lane 0 so that the compiler knows the role branches below are warp-uniform
    const uint32_t warp    = __shfl_sync(kFull, tid >> 5, 0);
    const uint32_t G       = gridDim.x;
    const uint32_t cta     = blockIdx.x;
    const uint64_t wait_ns = p.c.wait_ns;
    // One tensor of one wave has no totals, and its last tile's base needs a count from every CTA: no meeting.
    bool meet = false;
    for (uint32_t k = 0; k < p.c.jobs; ++k) meet = meet || p.job[k].tiles > G;

    const bool in_arena = p.c.arena != nullptr;
    if (tid == 0) {
        // read before the barrier below: the launch's first update of the cursor follows a tensor's last base,
        // which needs a publication from every CTA, and a CTA publishes only after this barrier
        s_arena_c0 = in_arena ? *reinterpret_cast<const volatile uint64_t *>(p.c.arena_cursor) : 0;
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

    // Tensors of more than one wave use wave totals: sums made by reductions, whose words must be zero before the
    // first count is added.  Every CTA zeroes a share and the grid meets once, here, before any warp takes up its
    // role; the first two bulk copies are on their way meanwhile.
    const Extent wsx = extent_of(p.c.ws_total, 8 * p.c.ws_words);
    if (meet) {
        for (uint32_t i = cta * blockDim.x + tid; i < p.c.ws_totals; i += G * blockDim.x)
            if (wsx.holds(p.c.ws_total + i, 8)) p.c.ws_total[i] = 0;
        cooperative_groups::this_grid().sync();
    }

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
                const U *const src   = static_cast<const U *>(p.job[w.k].src);
                const uint64_t first = static_cast<uint64_t>(w.tile(G)) * kTile;
                const uint64_t left  = p.job[w.k].n - first;
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

        // d0[k], d1[k], lane l <-> descriptor of virtual CTA l + 32k of the wave of this warp's previous tile;
        // w1, w2: total words of the one and the two waves before it (0: not read yet)
        uint64_t d0[kMaxWindows], d1[kMaxWindows], w1 = 0, w2 = 0;
#pragma unroll
        for (int k = 0; k < kMaxWindows; ++k) d0[k] = tag_w0, d1[k] = tag_w1;

        Walk cur;                                   // this warp's tile of the turn
        walk_begin(cur, p, cta, G);
        if (q == 1 && cur.valid) walk_next(cur, p, cta, G);
        uint32_t pk = 0, pj = 0, pv = 0;            // this warp's previous tile: tensor, wave, virtual CTA
        uint64_t waves_before = 0;                  // sum of the totals of the waves before the previous tile ...
        uint32_t waves_of     = 0xFFFFFFFFu;        // ... of this tensor
        uint64_t arena_at     = 0;                  // arena form: byte offset of the values of tensor arena_of ...
        uint32_t arena_of     = 0xFFFFFFFFu;        // ... (none yet)

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
                    uint64_t *const d = desc + 2 * (static_cast<uint64_t>(p.job[cur.k].desc0) + cur.tile(G));
                    if (wsx.holds(d, 16)) st_relaxed_2xu64(d, tag_w0 | agg, tag_w1 | agg);
                    s_agg[s] = agg;
                }
                if (lane < kWarps) s_off[s][lane] = inc - c;
                if (cur.tiles > G && lane == 0 && wsx.holds(wave_total + p.job[cur.k].total0 + cur.j, 8))
                    red_add_u64(wave_total + p.job[cur.k].total0 + cur.j, (1ull << kCountShift) + agg);
            }
            if (i >= 2) {
                // ---- (c): this warp's previous tile, (pk, pj, pv)
                const CompressJob &jb    = p.job[pk];
                uint32_t           polls = 0;
                uint64_t           t0    = 0;
                for (;;) {
                    bool missing = (pj > 0 && (w1 >> kCountShift) != G) || (pj > 1 && (w2 >> kCountShift) != G);
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k) missing |= !valid(d0[k], d1[k]);
                    if (!__any_sync(kFull, missing)) break;
                    __nanosleep(100);
                    if ((++polls & 255u) == 0 || (kTestHooks && wait_ns < kStrictLimitNs)) {
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
                    if (pj > 0 && (w1 >> kCountShift) != G) w1 = ld_relaxed_u64(wave_total + jb.total0 + (pj - 1));
                    if (pj > 1 && (w2 >> kCountShift) != G) w2 = ld_relaxed_u64(wave_total + jb.total0 + (pj - 2));
                }
                if (failed) break;
                uint64_t part = 0;
#pragma unroll
                for (int k = 0; k < kMaxWindows; ++k) part += static_cast<uint32_t>(d0[k]);
                // the waves in front of the tile: those in front of this warp's tile before it, if that was wave
                // pj - 2 of the same tensor, and the one or two waves read for this turn
                waves_before = (waves_of == pk ? waves_before : 0ull) + (w1 & ((1ull << kCountShift) - 1)) + (w2 & ((1ull << kCountShift) - 1));
                waves_of     = pk;
                const uint64_t base = waves_before + warp_sum_u64(part);
                const uint32_t ps   = (i - 2) % kStages;
                const uint64_t pt   = pv + static_cast<uint64_t>(pj) * G;
                // exclusive count in front of each chunk of that tile
                if (lane < kWarps && (lane % kWarpsPerChunk) == 0) {
                    const uint64_t ch = pt * kChunksPerTile + lane / kWarpsPerChunk;
                    const uint64_t chunks_total = (jb.n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS;
                    if (ch < chunks_total && extent_of(jb.prefix, 8 * chunks_total).holds(jb.prefix + ch, 8)) jb.prefix[ch] = base + s_off[ps][lane];
                }
                // Arena form: the tensor's values start where the tensor before it ended.  That cursor is published,
                // under the launch's tag, by whoever finishes that tensor's last tile; tensor 0 starts at the cursor
                // the launch found.  Read once per tensor and warp (bounded, like every wait here).
                if (in_arena && arena_of != pk) {
                    uint64_t at = s_arena_c0;
                    if (pk > 0) {
                        const uint64_t *const w = p.c.ws_arena + 2 * (pk - 1);
                        uint64_t       a0 = 0, a1 = 0;
                        const uint64_t ta = now_ns();
                        for (;;) {
                            ld_relaxed_2xu64(w, a0, a1);
                            if (((a0 ^ tag_w0) >> 32) == 0 && ((a1 ^ tag_w1) >> 32) == 0) break;
                            if (now_ns() - ta > wait_ns || ld_relaxed_u64(p.c.ws_header + kHdrAbort) == tag) {
                                failed = true;
                                break;
                            }
                            __nanosleep(100);
                        }
                        if (failed) break;
                        at = (a0 & 0xFFFFFFFFull) | (a1 << 32);
                    }
                    arena_at = at, arena_of = pk;
                }
                bool bump = false;              // lane 0: this is the launch's last tile
                if (pt == jb.tiles - 1 && lane == 0) {
                    const uint64_t nnz = base + s_agg[ps];
                    *jb.nnz_out        = nnz;
                    __threadfence();
                    const bool aborted  = ld_relaxed_u64(p.c.ws_header + kHdrAbort) == tag;
                    uint64_t   capacity = jb.capacity;
                    if (in_arena) {
                        // the room behind the tensor's start; the cursor moves past it only when everything fitted
                        capacity            = arena_at <= p.c.arena_bytes ? (p.c.arena_bytes - arena_at) / sizeof(U) : 0;
                        const bool     fits = !aborted && nnz <= capacity;
                        const uint64_t end  = fits ? arena_at + ((nnz * sizeof(U) + 15) & ~15ull) : arena_at;
                        if (fits) *jb.offset_out = arena_at;
                        if (pk + 1 == p.c.jobs) *p.c.arena_cursor = end;
                        if (wsx.holds(p.c.ws_arena + 2 * pk, 16))
                            st_relaxed_2xu64(p.c.ws_arena + 2 * pk, tag_w0 | (end & 0xFFFFFFFFull), tag_w1 | (end >> 32));
                    }
                    // without a meeting: every CTA has published its count by now, so every CTA has read the sequence
                    // number, and the next launch on this workspace gets another tag
                    bump = pk + 1 == p.c.jobs;
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
                if (__shfl_sync(kFull, bump ? 1 : 0, 0)) {
                    // The launch's last tile.  The next launch on this workspace must get another tag, and the sequence
                    // number may move only once every CTA has read it, i.e. has published a count.  The first G tiles
                    // of the launch are one per CTA: wait for their counts (they have been out for a long time).
                    bool seen[kMaxWindows];
#pragma unroll
                    for (int k = 0; k < kMaxWindows; ++k) seen[k] = lane + 32u * k >= G;
                    bool           all = true;
                    const uint64_t ts  = now_ns();
                    for (;;) {
                        bool miss = false;
#pragma unroll
                        for (int k = 0; k < kMaxWindows; ++k) {
                            if (!seen[k]) {
                                uint64_t x0, x1;
                                ld_relaxed_2xu64(desc + 2 * static_cast<uint64_t>(lane + 32u * k), x0, x1);
                                seen[k] = valid(x0, x1);
                                miss |= !seen[k];
                            }
                        }
                        if (!__any_sync(kFull, miss)) break;
                        if (__any_sync(kFull, now_ns() - ts > wait_ns)) {
                            all = false;
                            break;
                        }
                        __nanosleep(200);
                    }
                    if (lane == 0) red_add_u64(p.c.ws_header + kHdrSeq, all ? 1ull : 1ull << 32);
                }
                if (lane == 0) {
                    s_base[ps] = base;
                    s_dst[ps]  = arena_at;
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
                const uint64_t d_first = static_cast<uint64_t>(p.job[cur.k].desc0) + static_cast<uint64_t>(cur.j) * G;
#pragma unroll
                for (int k = 0; k < kMaxWindows; ++k) {
                    const uint32_t b = lane + 32u * k;
                    if (b < cur.v) ld_relaxed_2xu64(desc + 2 * (d_first + b), d0[k], d1[k]);
                    else d0[k] = tag_w0, d1[k] = tag_w1;             // not in front of this CTA: a valid count of 0
                }
                w1 = cur.j > 0 ? ld_relaxed_u64(wave_total + p.job[cur.k].total0 + (cur.j - 1)) : 0ull;
                w2 = cur.j > 1 ? ld_relaxed_u64(wave_total + p.job[cur.k].total0 + (cur.j - 2)) : 0ull;
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
        using V               = U;
        Walk w;
        walk_begin(w, p, cta, G);
        for (uint32_t it = 0; w.valid; ++it, walk_next(w, p, cta, G)) {
            const uint32_t s = it % kStages;
            if (!mbar_wait(&s_ready[s], (it / kStages) & 1u, &s_abort, wait_ns)) break;
            V             *vals     = static_cast<V *>(p.job[w.k].values);
            uint64_t       capacity = p.job[w.k].capacity;
            if (in_arena) {
                const uint64_t at = s_dst[s];
                vals              = reinterpret_cast<V *>(static_cast<unsigned char *>(p.c.arena) + at);
                capacity          = at <= p.c.arena_bytes ? (p.c.arena_bytes - at) / sizeof(V) : 0;
            }
            const Extent   vx       = extent_of(vals, capacity * sizeof(V));
            constexpr bool kBulk    = kBulkCopyOut16 && sizeof(U) == 2;             // 2-byte runs leave through the copy engine
            const uint64_t base     = s_base[s];
#pragma unroll
            for (int qq = 0; qq < kSegsPerCopier; ++qq) {
                const uint32_t seg  = copier * kSegsPerCopier + qq;
                U *const       pseg = tiles + static_cast<size_t>(s) * kTile + seg * kSeg;
                const uint32_t cnt  = s_cnt[s][seg];
                const uint64_t dst  = base + s_off[s][seg];
                if (dst + cnt <= capacity) {
                    if constexpr (kBulk) copy_out_run16(pseg, lane, cnt, vals + dst, vx);
                    else copy_out_segment<U, 0, false>(pseg, lane, cnt, vals + dst, 0, vx);
                } else {
                    copy_out_segment<U, 0, true>(pseg, lane, cnt, vals + dst, dst < capacity ? capacity - dst : 0, vx);
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
    const uint32_t bm_addr = smem_addr(&s_bits[warp][0]);
    Walk           w;
    walk_begin(w, p, cta, G);
    for (uint32_t it = 0; w.valid; ++it, walk_next(w, p, cta, G)) {
        const CompressJob &jb    = p.job[w.k];
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
            // Ragged last tile: each warp completes its own segment -- what the 16-byte granular bulk copy left out,
            // zeros behind the end of the tensor -- and meets no other warp over it.  (A barrier among the compactor
            // warps here would never open if one of them had left the kernel because its wait ran out.)
            const U *const src     = static_cast<const U *>(jb.src);
            const uint32_t have    = static_cast<uint32_t>(n - first);
            const uint32_t by_bulk = ((have * static_cast<uint32_t>(sizeof(U))) & ~15u) / sizeof(U);
            const uint32_t seg0    = warp * kSeg;
            for (uint32_t e = (by_bulk > seg0 ? by_bulk : seg0) + lane; e < seg0 + kSeg; e += 32)
                tile[e] = (e < have) ? src[first + e] : U(0);
            __syncwarp();
        }

        // ---- in-place compaction of this warp's segment
        const uint64_t e0     = first + warp * kSeg;                 // first element of the segment
        uint32_t       yvalid = 0;
        U             *y      = nullptr;
        if constexpr (WRITE_Y) {
            y      = static_cast<U *>(jb.y) + e0;
            yvalid = e0 + kSeg <= n ? static_cast<uint32_t>(kSeg) : (e0 < n ? static_cast<uint32_t>(n - e0) : 0u);
        }
        const Extent   yx       = extent_of(jb.y, n * sizeof(U));
        const uint32_t seg_addr = smem_addr(tile + warp * kSeg);
        uint32_t       run, word;
        if (!WRITE_Y || yvalid == static_cast<uint32_t>(kSeg))   // all but a ragged last tile: no bounds checks on y
            run = compact_segment<U, FUSED, WRITE_Y, false, kSeg / 32>(seg_addr, word, lane, y, yvalid, p.c.tau, yx);
        else
            run = compact_segment<U, FUSED, WRITE_Y, true, kSeg / 32>(seg_addr, word, lane, y, yvalid, p.c.tau, yx);
        if (lane < static_cast<uint32_t>(kSeg / 32)) {
            const uint64_t wd = t64 * (kTile / 32) + warp * (kSeg / 32) + lane;
            if (wd < ((n + 31) >> 5) && extent_of(jb.bitmap, 4 * ((n + 31) >> 5)).holds(jb.bitmap + wd, 4)) jb.bitmap[wd] = word;
        }
        __syncwarp();
        if (lane == 0) {
            s_cnt[s][warp] = run;
            mbar_arrive(&s_counted[s]);                   // hand the count to the scan warp
        }
    }
}

template <typename U, int FUSED, bool WRITE_Y, int kJobs, int kWarps, int kSeg, int kStages, int kCopiers>
cudaError_t launch_shaped(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, cudaStream_t stream)
{
    constexpr int    kTile    = kWarps * kSeg;
    constexpr int    kThreads = (kWarps + kCopiers + 3) * 32;
    constexpr size_t kSmem    = static_cast<size_t>(kStages) * kTile * sizeof(U);
    static LaunchShape shape;   // one per instantiation
    auto kernel = compress_kernel<U, FUSED, WRITE_Y, kJobs, kWarps, kSeg, kStages, kCopiers>;
    if (count == 0 || count > static_cast<uint32_t>(kJobs)) return cudaErrorInvalidValue;

    CompressParams<kJobs> p;
    p.c             = c;
    uint64_t tiles  = 0, chunks = 0;
    for (uint32_t k = 0; k < count; ++k) {
        p.job[k]            = jobs[k];
        const uint64_t t    = (jobs[k].n + kTile - 1) / kTile;
        if (t == 0 || t > 0xFFFFFFFFull) return cudaErrorInvalidValue;
        p.job[k].tiles      = static_cast<uint32_t>(t);
        tiles += t;
        chunks += (jobs[k].n + BT_CHUNK_ELEMS - 1) / BT_CHUNK_ELEMS;
    }
    if (tiles > 0xFFFFFFFFull) return cudaErrorInvalidValue;
    for (uint32_t k = count; k < static_cast<uint32_t>(kJobs); ++k) p.job[k] = CompressJob{};

    int         max_grid = 0;
    cudaError_t e        = shape.max_grid(kernel, kThreads, kSmem, max_grid);
    if (e != cudaSuccess) return e;
    if (max_grid > 32 * kMaxWindows) max_grid = 32 * kMaxWindows;
    if (compress_max_ctas() != 0 && static_cast<uint32_t>(max_grid) > compress_max_ctas()) max_grid = static_cast<int>(compress_max_ctas());
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
    p.c.ws_words  = (batch_workspace_bytes(chunks, count) - kWsHeaderBytes) / 8;
    p.c.ws_arena  = p.c.ws_desc + 2 * dealt;                          // behind the descriptors: 16-byte aligned like them
    p.c.call_tag  = next_call_tag();
    p.c.wait_ns   = compress_wait_ns();
    // cooperative launch: the runtime guarantees that all `grid` CTAs are resident together
    void *params[] = {&p};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(kThreads), params, kSmem, stream);
}

template <typename U, int FUSED, bool WRITE_Y>
cudaError_t launch_typed(const CompressCommon &c, const CompressJob *jobs, uint32_t count, void *workspace, cudaStream_t stream)
{
    // the shapes of the single-tensor kernel
    if constexpr (sizeof(U) == 8) return launch_shaped<U, FUSED, WRITE_Y, kMaxBatch, 8, 512, 7, 8>(c, jobs, count, workspace, stream);
    else if constexpr (sizeof(U) == 4) return launch_shaped<U, FUSED, WRITE_Y, kMaxBatch, 8, 1024, 7, 8>(c, jobs, count, workspace, stream);
    else return launch_shaped<U, FUSED, WRITE_Y, kMaxBatch, 16, 1024, 7, 8>(c, jobs, count, workspace, stream);
}

}  // namespace

cudaError_t launch_compress_batch(const CompressJob *jobs, uint32_t count, float tau, void *workspace, int dtype, int fused,
                                  const BatchArena *arena, cudaStream_t stream)
{
    // fused: 0 plain compressor, 1 threshold form (ReLU at tau = 0)
    // the dense output is written for all tensors of a launch or for none
    if (count == 0 || count > kMaxBatch || fused > 1) return cudaErrorInvalidValue;
    const bool y = jobs[0].y != nullptr;
    for (uint32_t k = 1; k < count; ++k)
        if ((jobs[k].y != nullptr) != y) return cudaErrorInvalidValue;
    CompressCommon c{};
    c.tau = tau;
    if (arena) {
        c.arena        = arena->arena;
        c.arena_bytes  = arena->arena_bytes;
        c.arena_cursor = arena->arena_cursor;
    }
    if (fused == 0) {
        return dtype == BT_F64   ? launch_typed<uint64_t, -1, false>(c, jobs, count, workspace, stream)
               : dtype == BT_F32 ? launch_typed<uint32_t, -1, false>(c, jobs, count, workspace, stream)
                                 : launch_typed<uint16_t, -1, false>(c, jobs, count, workspace, stream);
    }
    if (tau == 0.0f && (dtype == BT_F16 || dtype == BT_BF16)) {
        // the ReLU itself on a 2-byte type: decided by one compare in the element's own type (as in the single-tensor kernel)
        constexpr int kh = kFusedReluHalf;
        if (dtype == BT_F16)
            return y ? launch_typed<uint16_t, kh + BT_F16, true>(c, jobs, count, workspace, stream)
                     : launch_typed<uint16_t, kh + BT_F16, false>(c, jobs, count, workspace, stream);
        return y ? launch_typed<uint16_t, kh + BT_BF16, true>(c, jobs, count, workspace, stream)
                 : launch_typed<uint16_t, kh + BT_BF16, false>(c, jobs, count, workspace, stream);
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
