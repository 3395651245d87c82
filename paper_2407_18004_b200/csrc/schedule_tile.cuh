// Device code shared by the table kernel and the verification sweep: per-rank rows, the
// shared-memory queues of undecided entries, the closed-form pass over a tile of kThreads
// consecutive ranks in its two launch shapes, and the table kernel itself.
//
//   schedule_table_kernel   one thread per rank, one block per run of consecutive tiles of 256
//                           ranks.  The ranks of a tile agree on their digits at the high levels
//                           over long runs, so one warp describes those runs once (a lane per
//                           level) and every thread copies its rank's high-level entries from the
//                           description and walks only the low levels with the closed forms
//                           (schedule_fast.cuh).  Entries land as bytes in a shared-memory tile
//                           laid out exactly like the output; what the closed forms leave
//                           undecided is collected in shared-memory queues and resolved by the
//                           search of Algorithms 4 and 5 (schedule_core.cuh) or copied from a
//                           neighbouring row.  The tile is then widened to int32 and streamed out
//                           as one contiguous run of 16-byte stores, so every store instruction
//                           fills whole 32-byte sectors.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "schedule_core.cuh"
#include "schedule_fast.cuh"

namespace bcast {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kTableBlocksPerSm = 8;                   // resident blocks the table kernel is sized for
constexpr int kSweepBlocksPerSm = 6;                   // resident blocks of the verification sweep
constexpr int kBlocksPerSmWanted = 64;                 // grid size below which blocks take fewer tiles
constexpr int kMaxRowBytes = 32;                       // staged row: q <= 31 bytes (+ pad in batch form)

// ------------------------------------------------------------------ per-rank rows
// Where a thread puts entry k of a row: a byte row in shared memory ...
struct ByteRow {
    int8_t *row;
    __device__ __forceinline__ void operator()(int k, int val) const { row[k] = (int8_t)val; }
    __device__ __forceinline__ int get(int k) const { return row[k]; }
};
// ... or one column element of a round-major table (entry k of rank r at base[k*stride]).
struct StridedColumn {
    int8_t *base;
    size_t stride;
    __device__ __forceinline__ void operator()(int k, int val) const { base[(size_t)k * stride] = (int8_t)val; }
    __device__ __forceinline__ int get(int k) const { return base[(size_t)k * stride]; }
};

// Both rows of virtual rank r.  Returns the number of Algorithm 6 violations.
template <class Writer, class Stats>
__device__ __forceinline__ int rank_rows(const Geometry &g, uint32_t r, Writer recv_row, Writer send_row,
                                         bool want_recv, bool want_send, Stats &stats)
{
    const int q = g.q;
    const int b = want_recv ? recv_search_fast(g, r, q - 1, recv_row, stats) : baseblock(g, r);
    int nviol = 0;
    if (want_send) {
        if (r == 0u) {
            for (int k = 0; k < q; ++k) send_row(k, k);
        } else {
            uint32_t viol = send_walk(g, r, b, send_row);
            while (viol != 0u) {
                const int k = 31 - __clz(viol);
                viol ^= 1u << k;
                uint32_t t = r + skip_of(g, k);
                if (t >= g.p) t -= g.p;
                NoStats ns;
                send_row(k, recv_entry(g, t, k, ns));
                ++nviol;
            }
        }
    }
    return nviol;
}

__device__ __forceinline__ int sext_byte(uint32_t w, uint32_t selector)
{
    int out;
    // prmt: selector nibbles with bit 3 set replicate the sign of the chosen byte
    asm("prmt.b32 %0, %1, 0, %2;" : "=r"(out) : "r"(w), "r"(selector));
    return out;
}

__device__ __forceinline__ int4 widen4(uint32_t w)
{
    int4 v;
    v.x = sext_byte(w, 0x8880u);                       // byte 0 widened to int32
    v.y = sext_byte(w, 0x9991u);
    v.z = sext_byte(w, 0xAAA2u);
    v.w = sext_byte(w, 0xBBB3u);
    return v;
}

// Stream n_entries staged bytes out as int32, starting at out[0]; a group of kGroup
// threads (a warp or the whole block), `lane` being the index within the group.
template <int kGroup>
__device__ __forceinline__ void flush_tile(const uint32_t *stage_words, int32_t *out, int n_entries,
                                           bool vec_ok, int lane)
{
    const int8_t *stage_bytes = reinterpret_cast<const int8_t *>(stage_words);
    int done = 0;
    if (vec_ok) {
        const int nvec = n_entries >> 2;
        int4 *out4 = reinterpret_cast<int4 *>(out);
        for (int i = lane; i < nvec; i += kGroup) __stcs(out4 + i, widen4(stage_words[i]));
        done = nvec << 2;
    }
    for (int i = done + lane; i < n_entries; i += kGroup) __stcs(out + i, (int)stage_bytes[i]);
}

// Algorithm 1's preamble for n blocks, applied while a tile is streamed out: entry k of every
// row gets -x, and +q on top when k < x (the rounds before x are virtual, their entries
// belong to the next phase).  The tile starts at a row boundary, so staged byte e is column
// e mod Q.  shift_words[c] holds the four byte-wise addends for a word whose first byte is
// column c; the sums stay within [-2q+1, 2q-2] and fit a byte.
template <int Q>
__device__ __forceinline__ void fill_shift_words(uint32_t *shift_words, int x)
{
    if (threadIdx.x < Q) {
        uint32_t add = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = ((int)threadIdx.x + j) % Q;
            add |= (uint32_t)((c < x ? Q - x : -x) & 0xff) << (8 * j);
        }
        shift_words[threadIdx.x] = add;
    }
}

// Four byte sums without carries between the bytes.
__device__ __forceinline__ uint32_t add_bytes(uint32_t a, uint32_t b)
{
    return ((a & 0x7f7f7f7fu) + (b & 0x7f7f7f7fu)) ^ ((a ^ b) & 0x80808080u);
}

// flush_tile by the whole block with the preamble's addends applied on the way out.
template <int Q>
__device__ __forceinline__ void flush_tile_shifted(const uint32_t *stage_words, const uint32_t *shift_words,
                                                   int32_t *out, int n_entries, bool vec_ok, int x)
{
    const int8_t *stage_bytes = reinterpret_cast<const int8_t *>(stage_words);
    int done = 0;
    if (vec_ok) {
        const int nvec = n_entries >> 2;
        int4 *out4 = reinterpret_cast<int4 *>(out);
        int c0 = (4 * (int)threadIdx.x) % Q;               // column of the word's first byte
        constexpr int kStep = (4 * kThreads) % Q;
        for (int i = threadIdx.x; i < nvec; i += kThreads) {
            __stcs(out4 + i, widen4(add_bytes(stage_words[i], shift_words[c0])));
            c0 += kStep;
            if (c0 >= Q) c0 -= Q;
        }
        done = nvec << 2;
    }
    for (int i = done + (int)threadIdx.x; i < n_entries; i += kThreads)
        __stcs(out + i, (int)stage_bytes[i] + (i % Q < x ? Q - x : -x));
}

// ------------------------------------------------------------------ all ranks of one p
// Work the closed-form pass leaves behind, collected per tile of kThreads consecutive ranks.
//
// SearchItem: recvblock[k] of virtual rank `rank` is wanted for every k in `mask` and goes
// to row `row` of the tile's receive (table = 0) or send (table = 1) rows.
// A copy (packed into 32 bits) says: sendblock[k] of row dst is recvblock[k] of row src of
// the same tile (Section 2.3's definition, the to-processor being src), to be taken once
// the searches of the tile are done.
struct SearchItem {
    uint32_t rank;
    uint32_t mask;
    uint16_t row;
    uint16_t table;
};

constexpr int kLongFromRound = 2;               // searches wanted up to this round or beyond count as long

// A queue serves a GROUP of consecutive rows of the tile whose threads drain it together:
// the whole tile (kGroup = kThreads, the threads meet at block barriers) or one warp's 32
// rows (kGroup = 32, the warp goes through pass, drain and flush on its own and meets no
// other warp).  Items never leave their group: a copy's source row lies in it.
template <int kGroup>
struct GroupQueue {
    static constexpr int kGroupSize = kGroup;
    static constexpr int kSearchCapacity = 2 * kGroup;
    static constexpr int kCopyCapacity = 2 * kGroup;
    SearchItem search[kSearchCapacity];         // short searches from slot 0, long ones from the middle
    uint32_t copy[kCopyCapacity];               // src | dst << 9 | k << 18
    int n_search;                               // short: highest wanted round below kLongFromRound
    int n_long;
    int n_copy;
    __device__ __forceinline__ static void sync()
    {
        if constexpr (kGroup == 32) __syncwarp(); else __syncthreads();
    }
};
typedef GroupQueue<kThreads> TileQueue;

// Run the search for one item and drop the wanted entries into `row`.
template <class Row, class Stats>
__device__ __forceinline__ void resolve_item(const Geometry &g, const SearchItem &it, Row row, Stats &stats)
{
    const uint32_t mask = it.mask;
    recv_search_fast(g, it.rank, 31 - __clz(mask),
                     [&](int k, int val) { if ((mask >> k) & 1u) row(k, val); }, stats);
}

// Queue a search; when the queue is full the calling thread does it on the spot.
template <class Queue, class Tile, class Stats>
__device__ __forceinline__ void push_search(const Geometry &g, Queue &queue, const SearchItem &it,
                                            const Tile &tile, Stats &stats)
{
    // a search runs until its highest wanted round; like lengths side by side keep a warp's lanes together
    constexpr int kHalf = Queue::kSearchCapacity / 2;
    const bool is_long = it.mask >= (1u << kLongFromRound);
    const int slot = atomicAdd(is_long ? &queue.n_long : &queue.n_search, 1);
    if (slot < kHalf) {
        queue.search[(is_long ? kHalf : 0) + slot] = it;
    } else {
        resolve_item(g, it, it.table == 0 ? tile.recv_row(it.row) : tile.send_row(it.row), stats);
    }
}

// A send entry Algorithm 6 could not decide: round k of the rank in row `index`, virtual
// rank r.  Its to-processor is a row of the same group whose receive entry will be final
// after the group's searches (then a copy is queued), or a rank that needs a search of its own.
template <class Queue, class Tile, class Stats>
__device__ __forceinline__ void push_send_violation(const Geometry &g, uint32_t skip_k, int k, uint32_t r,
                                                    uint32_t index, uint32_t rows, bool want_recv,
                                                    Queue &queue, const Tile &tile, Stats &stats)
{
    if (want_recv && index + skip_k < rows &&
        (index + skip_k) / Queue::kGroupSize == index / Queue::kGroupSize) {
        const int slot = atomicAdd(&queue.n_copy, 1);
        if (slot < Queue::kCopyCapacity) {
            queue.copy[slot] = (index + skip_k) | (index << 9) | ((uint32_t)k << 18);
            return;
        }
    }
    uint32_t t = r + skip_k;
    if (t >= g.p) t -= g.p;
    push_search(g, queue, SearchItem{t, 1u << k, (uint16_t)index, 1}, tile, stats);
}

// Whether the ranks of a tile can share their high levels: a full tile of consecutive
// virtual ranks without the root and without a wrap past p-1.
template <int Q>
__device__ __forceinline__ bool tile_can_share(const Geometry &g, uint32_t r_first, uint32_t rows)
{
    return Q >= kSharedFrom + 2 && rows == (uint32_t)kThreads && r_first >= 1u &&
           r_first <= g.p - (uint32_t)kThreads;
}

// The closed-form pass for one tile: row i of the tile holds virtual rank (r_first + i) mod p,
// `rows` rows are real.  Called by every thread of the block; thread i owns row i.  With a
// run description of the tile (runs.n_runs > 0, see build_tile_runs) every rank copies its
// high-level entries from it and walks only the low levels; without one each rank walks
// all levels, with rank 1 as a stand-in for the root and for rows that are not real.  What
// the pass cannot decide is queued.  Returns Algorithm 6's violations of this thread's rank.
template <int Q, class Tile, class Queue, class Stats>
__device__ __forceinline__ uint32_t tile_pass(const LevelTables &tab, const Geometry &g,
                                              const TileRuns<typename WalkInt<Q>::type> &runs,
                                              uint32_t r_first, uint32_t rows, const Tile &tile,
                                              bool want_recv, bool want_send, Queue &queue, Stats &stats)
{
    const uint32_t index = threadIdx.x;
    const bool active = index < rows;
    uint32_t r = 1u;
    if (active) {
        r = r_first + index;                               // < 2p: index < rows <= p
        if (r >= g.p) r -= g.p;
    }
    auto recv_row = tile.recv_row(index);
    auto send_row = tile.send_row(index);
    uint32_t recv_flags = 0, send_flags = 0;

    bool shared = false;
    if constexpr (Q >= kSharedFrom + 2) {
        shared = runs.n_runs > 0;                          // the same for the whole block
        if (shared) {
            auto st = apply_tile_runs<Q>(runs, (int)index, recv_row, send_row);
            closed_form_levels<Q, kSharedFrom>(tab, st, recv_row, send_row, recv_flags, send_flags);
            closed_form_finish<Q>(tab, r, st.j, recv_row, send_row, recv_flags);
            // entries of the high levels that the description left undecided (at most kMaxPending = 32,
            // so the threads of one group see them all); each goes to the queue of its row's group
            const uint32_t member = index % Queue::kGroupSize;
            const uint32_t item = (int)member < runs.n_pending ? runs.pending[member] : 0xffffffffu;
            if (item != 0xffffffffu && (item & 511u) / Queue::kGroupSize == index / Queue::kGroupSize) {
                const uint32_t row = item & 511u;
                const int k = (int)((item >> 9) & 31u);
                const uint32_t rr = r_first + row;
                if ((item >> 14) & 1u) {
                    stats.violation(row, k);
                    if (want_send)
                        push_send_violation(g, tab.skip[k], k, rr, row, rows, want_recv, queue, tile, stats);
                } else if (want_recv) {
                    push_search(g, queue, SearchItem{rr, 1u << k, (uint16_t)row, 0}, tile, stats);
                }
            }
        }
    }
    if (!shared) {
        const bool is_root = r == 0u;
        int b = 0;
        recv_flags = closed_form_rows<Q>(tab, g.p, is_root ? 1u : r, recv_row, send_row, &send_flags, &b);
        if (!active) return 0u;
        if (is_root) {                                     // the root sends block k in round k
            for (int k = 0; k < Q; ++k) send_row(k, k);
            recv_flags = (2u << (Q - 1)) - 1u;             // and its receive row comes from the search
            send_flags = 0u;
        }
    }
    if (want_recv && recv_flags != 0u)
        push_search(g, queue, SearchItem{r, recv_flags, (uint16_t)index, 0}, tile, stats);
    uint32_t todo = want_send ? send_flags : 0u;
    while (todo != 0u) {
        const int k = 31 - __clz(todo);
        todo ^= 1u << k;
        push_send_violation(g, tab.skip[k], k, r, index, rows, want_recv, queue, tile, stats);
    }
    return send_flags;
}

// After the closed-form pass of a group's rows and its barrier: searches, then (after another
// barrier, only if needed) the copies.  Every thread of the group calls this.
template <class Queue, class Tile, class Stats>
__device__ __forceinline__ void drain_queue(const Geometry &g, Queue &queue, const Tile &tile, Stats &stats)
{
    constexpr int kGroup = Queue::kGroupSize;
    const int member = threadIdx.x % kGroup;
    constexpr int kHalf = Queue::kSearchCapacity / 2;
    const int n_short = min(queue.n_search, kHalf);
    const int n_search = n_short + min(queue.n_long, kHalf);
    const int n_copy = min(queue.n_copy, Queue::kCopyCapacity);
    for (int i = member; i < n_search; i += kGroup) {
        const SearchItem it = queue.search[i < n_short ? i : kHalf + (i - n_short)];
        // one call site: items for either table run the same instructions side by side
        resolve_item(g, it, it.table == 0 ? tile.recv_row(it.row) : tile.send_row(it.row), stats);
    }
    if (n_copy > 0) {
        Queue::sync();                                     // n_copy is the same for every thread of the group
        for (int i = member; i < n_copy; i += kGroup) {
            const uint32_t c = queue.copy[i];
            const int k = (int)(c >> 18);
            tile.send_row((c >> 9) & 511u)(k, tile.recv_row(c & 511u).get(k));
        }
    }
}

// The table kernel's tile: byte rows in shared memory, laid out like the output.  Row i of
// the pass (ranks ascending) is output row i, or output row rows-1-i when the output lists
// the ranks in descending order (the all-broadcast tables); rows beyond the real ones keep
// their own slot.
template <int Q>
struct SharedTile {
    int8_t *recv;
    int8_t *send;
    uint32_t rows;
    bool descending;
    __device__ __forceinline__ uint32_t slot(uint32_t i) const { return descending && i < rows ? rows - 1u - i : i; }
    __device__ __forceinline__ ByteRow recv_row(uint32_t i) const { return ByteRow{recv + slot(i) * Q}; }
    __device__ __forceinline__ ByteRow send_row(uint32_t i) const { return ByteRow{send + slot(i) * Q}; }
};

// ------------------------------------------------------------------ warps on their own, searches deferred
// The launch shapes of bcast_schedule proper.  After the run descriptions are built no warp
// waits for another: each takes its own 32 rows of every tile through the closed-form pass
// and streams them out at once, undecided entries included (with whatever the pass left
// there).  What is undecided is queued, and between two groups of kWarpsPerBlock tiles the whole
// block works the queues off, storing every entry straight into the output table, over the
// placeholder -- after every group where the block's first group fills a quarter of a queue (a
// dirty p), else once a queue is half full and after the last group (a p with few undecided
// entries gathers several groups' worth, which keeps more lanes busy per search):
//   1. searches (DeferredItem): the receive schedule of a virtual rank is searched up to a round k;
//      kind 0 writes the receive entries of the rank's own row for every round up to k (the search
//      yields them all, and those the pass had decided are the same), kind 1 the send entry of
//      round k of a row whose to-processor the rank is;
//   2. after a barrier, fix-ups: a send entry whose to-processor is a row of the same
//      group is that row's receive entry (Section 2.3), final in the output table by
//      then, and is copied from there.
// (Per tile, the undecided entries of 256 rows keep only a third of a block's lanes busy;
// per warp even fewer.)
struct DeferredItem {
    uint32_t rank;                                         // virtual rank whose receive schedule is searched
    uint32_t what;                                         // output row relative to the block | k << 14 | kind << 19
};                                                         // kind 0: every round up to k; kind 1: round k alone

constexpr int kDeferredCapacity = 384;
constexpr int kFixupCapacity = 768;
constexpr int kGroupRows = kWarpsPerBlock * kThreads;  // rows of a group of tiles
constexpr int kLowFrameTiles = 16;                     // most tiles of a block that works with the table of low states
constexpr int kLowFrameStates = 512;                   // skip[kSharedFrom] <= 2^kSharedFrom states of the low frame

// The table of low states as the host hands it to the kernel (low_frame_fill).
struct LowFrameTable {
    uint32_t word[kLowFrameStates];
};

// Launch shapes of the table kernel.
constexpr int kShapeBlockPerTile = 0;                  // the block meets after every tile and drains its queues
constexpr int kShapeWarps = 1;                         // warps on their own, searches deferred to the group's end
constexpr int kShapeWarpsLowFrame = 2;                 // the same, undecided low rounds from the table of low states
constexpr int kShapeWarpsTight = 3;                    // kShapeWarps with room for kTightCapacity queue entries (tests)
constexpr int kTightCapacity = 8;
constexpr int kDescWarpsFromQ = 16;                    // smallest q with a descending-rows kernel of that shape

struct DeferredQueue {
    DeferredItem items[kDeferredCapacity];
    uint32_t fixups[kFixupCapacity];                       // row relative to the block | k << 14
    uint32_t low_frame[kLowFrameStates];                   // low_frame_entry(u) for u < skip[kSharedFrom], if given
    uint32_t need_recv[kWarpsPerBlock][32];                // per warp and row of its slice: rounds to search
    int n_items;
    int n_fixups;
    uint32_t overflow;                                     // groups of the block (a bit each) that found a queue full
};

union QueueStorage {
    TileQueue tile;                                        // one queue for the block, or
    DeferredQueue deferred;                                // the group's deferred work
};

// Both rows of `rows` consecutive output rows by the search alone (Algorithms 4-6 per rank,
// as for independent queries), written straight into the tables.  Slow: the way out for a
// group of tiles whose queues overflowed, run at the block's end, apart from the code of the pass.
// index0: output index of the first row (row x holds virtual rank (index - anchor) mod p, or
// (anchor - index) mod p for descending rows); recv/send point at that row (either may be null).
struct IntRow {
    int32_t *row;
    __device__ __forceinline__ void operator()(int k, int val) const { row[k] = val; }
};

static __device__ __forceinline__ void rows_by_search(uint32_t p, uint32_t anchor, uint32_t index0, int descending,
                                                   uint32_t rows, int32_t *recv, int32_t *send)
{
    const Geometry g = make_geometry(p);
    NoStats ns;
    for (uint32_t i = threadIdx.x; i < rows; i += blockDim.x) {
        const uint32_t index = index0 + i;
        const uint32_t r = descending ? (anchor >= index ? anchor - index : anchor + (p - index))
                                      : (index >= anchor ? index - anchor : index + (p - anchor));
        rank_rows(g, r, IntRow{recv + (size_t)i * g.q}, IntRow{send + (size_t)i * g.q}, recv != nullptr,
                  send != nullptr, ns);
    }
}

// Whether the search completed all kLowFrameRounds rounds of the word inside the low levels; round
// kLowFrameRounds is then the lowest shared digit, like a kLowFramePop nibble.
__device__ __forceinline__ bool low_frame_full(uint32_t word) { return (word >> 28) < kLowFramePop; }

// Search for one deferred item; emit(table, row, k, value) receives every wanted entry
// (table 0 = receive, 1 = send; row relative to the group's first row).
template <class Emit>
__device__ __forceinline__ void resolve_deferred(const Geometry &g, const DeferredItem &it, Emit emit)
{
    const uint32_t row = it.what & 16383u;
    const int k_last = (int)((it.what >> 14) & 31u);
    const bool one_send = (it.what >> 19) != 0u;
    NoStats ns;
    recv_search_fast(g, it.rank, k_last, [&](int k, int val) {
        if (!one_send) emit(0, row, k, val);
        else if (k == k_last) emit(1, row, k, val);
    }, ns);
}

// A table word of low_frame_entry as schedule values: byte k of the pair holds the value of
// round k (index - q; the lowest shared digit j_high - q where the search returned past the
// low levels), and bit k of the result says whether the table has that round at all.
template <int Q>
__device__ __forceinline__ uint32_t low_frame_values(uint32_t word, int j_high, uint32_t &rounds_0_3,
                                                     uint32_t &rounds_4_7)
{
    const uint32_t even = word & 0x0f0f0f0fu, odd = (word >> 4) & 0x0f0f0f0fu;     // nibbles 0,2,4,6 / 1,3,5,7
    uint32_t lo = __byte_perm(even, odd, 0x5140), hi = __byte_perm(even, odd, 0x7362);
    const uint32_t none_lo = __vcmpeq4(lo, 0x0f0f0f0fu), none_hi = __vcmpeq4(hi, 0x0f0f0f0fu);
    const uint32_t pop_lo = __vcmpeq4(lo, 0x0e0e0e0eu), pop_hi = __vcmpeq4(hi, 0x0e0e0e0eu);
    const uint32_t j4 = (uint32_t)j_high * 0x01010101u;
    lo = (lo & ~pop_lo) | (j4 & pop_lo);
    hi = (hi & ~pop_hi) | (j4 & pop_hi);
    constexpr uint32_t kMinusQ = (uint32_t)((-Q) & 0xff) * 0x01010101u;
    rounds_0_3 = add_bytes(lo, kMinusQ);
    rounds_4_7 = add_bytes(hi, kMinusQ);
    // one bit per byte: 0x80 of each byte gathered into bits 0..3
    const uint32_t have_lo = ~none_lo & 0x80808080u, have_hi = ~none_hi & 0x80808080u;
    uint32_t have = ((have_lo * 0x00204081u) >> 28) | (((have_hi * 0x00204081u) >> 28) << 4);
    // eight rounds inside the low levels use up every index there, so the ninth is the return past them
    if (low_frame_full(word)) have |= 1u << kLowFrameRounds;
    return have;
}

// Undecided low rounds from the table of the search's low states (low_frame_entry): the
// rank's own receive entries from its own state u_low, and its send entries from the state
// of its to-processor where that is a rank of the same run (same digits at the levels
// >= kSharedFrom, u_low + skip[k] left below them), whether or not it is a row of the same
// tile: `room` = the ranks from this one on that lie in its run and below p.
template <int Q, class Row>
__device__ __forceinline__ void low_frame_lookups(const LevelTables &tab, const uint32_t *low_frame,
                                                  uint32_t u_low, int j_high, uint32_t room,
                                                  Row recv_row, Row send_row, uint32_t &recv_flags,
                                                  uint32_t &send_flags, bool any_recv)
{
    constexpr uint32_t kLowMask = (2u << kLowFrameRounds) - 1u;   // the table's rounds and the one after them
    if (any_recv) {                                        // the same for the whole warp
        // receive entries: straight-line, a predicated byte store per round
        uint32_t v03, v47;
        const uint32_t have = low_frame_values<Q>(low_frame[u_low], j_high, v03, v47);
        const uint32_t take = recv_flags & have & kLowMask;
#pragma unroll
        for (int k = 0; k < kLowFrameRounds && k < Q; ++k)
            if ((take >> k) & 1u) recv_row(k, (int)(int8_t)((k < 4 ? v03 : v47) >> (8 * (k & 3))));
        if (kLowFrameRounds < Q && ((take >> kLowFrameRounds) & 1u)) recv_row(kLowFrameRounds, j_high - Q);
        recv_flags ^= take;
    }
    // send entries: at most four per rank (Theorem 3), one table word each
    uint32_t todo = send_flags & kLowMask;
    while (todo != 0u) {
        const int k = __ffs(todo) - 1;
        todo &= todo - 1u;
        const uint32_t skip_k = skip_of(make_geometry(tab.skip[Q]), k);
        if (skip_k < room) {
            const uint32_t word_t = low_frame[u_low + skip_k];
            const uint32_t nib = k < kLowFrameRounds ? (word_t >> (4 * k)) & 15u
                                                     : (low_frame_full(word_t) ? kLowFramePop : kLowFrameNone);
            if (nib <= kLowFramePop) {
                send_row(k, (nib == kLowFramePop ? j_high : (int)nib) - Q);
                send_flags ^= 1u << k;
            }
        }
    }
}

// The closed-form pass of one warp's 32 rows of a tile (lane l owns row 32*warp + l).  Rounds
// the pass cannot decide are looked up (low_frame, if given) or queued; a full queue drops the
// item and marks the group, whose rows the caller then computes again by the search alone.
// capacity_cut takes room away from the queues (0 normally; the tests' tight shape).  group_row0: the tile's first output row relative to the group; group_rows:
// output rows of the group.
template <int Q, bool desc, class Tile>
__device__ __forceinline__ void warp_pass(const LevelTables &tab, const Geometry &g,
                                          const TileRuns<typename WalkInt<Q>::type> &runs,
                                          uint32_t r_first, uint32_t rows, uint32_t block_row0,
                                          uint32_t group_rows, const Tile &tile,
                                          bool want_recv, bool want_send, DeferredQueue &dq,
                                          uint32_t group_bit, int capacity_cut, const uint32_t *low_frame)
{
    // block_row0: the tile's first output row relative to the block's; groups are kGroupRows rows each,
    // so its place within its group is the remainder
    const uint32_t group_row0 = block_row0 & (uint32_t)(kGroupRows - 1);
    // index: the thread's row of the staged tile = its output row within the tile.  The ranks of a tile
    // ascend with the row, or descend (Algorithm 7's tables); `ahead` is the thread's place counted from
    // the tile's lowest rank r_first, which is how the run descriptions number the rows.
    const uint32_t index = threadIdx.x;
    const uint32_t lane = index & 31u;
    const uint32_t warp = index >> 5;
    uint32_t *need_recv = dq.need_recv[warp];
    const bool active = index < rows;
    const uint32_t ahead = desc && active ? rows - 1u - index : index;
    uint32_t r = 1u;
    if (active) {
        r = r_first + ahead;
        if (r >= g.p) r -= g.p;
    }
    auto recv_row = tile.recv_row(index);
    auto send_row = tile.send_row(index);
    need_recv[lane] = 0u;
    __syncwarp();

    auto defer = [&](const DeferredItem &it) {
        const int slot = atomicAdd(&dq.n_items, 1);
        if (slot < kDeferredCapacity - capacity_cut) {
            dq.items[slot] = it;
        } else {
            atomicOr(&dq.overflow, group_bit);             // the group's rows are redone by rows_by_search
        }
    };
    // Algorithm 6 could not decide round k of the send row of tile row `row` (virtual rank rr): the entry
    // is the receive entry of the to-processor, skip[k] ranks ahead.  If that is a row of this group and
    // the receive table is written, the entry is copied from there once the group's searches are done;
    // otherwise the to-processor's receive schedule is searched for it.
    auto violation = [&](uint32_t row, int k, uint32_t rr) {
        const uint32_t skip_k = tab.skip[k];
        const uint32_t out_row = group_row0 + row;
        const bool in_group = desc ? out_row >= skip_k : out_row + skip_k < group_rows;
        if (want_recv && in_group) {
            const int slot = atomicAdd(&dq.n_fixups, 1);
            if (slot < kFixupCapacity - capacity_cut * (kFixupCapacity / kDeferredCapacity)) {
                dq.fixups[slot] = (block_row0 + row) | ((uint32_t)k << 14);
                return;
            }
        }
        uint32_t t = rr + skip_k;
        if (t >= g.p) t -= g.p;
        defer(DeferredItem{t, (block_row0 + row) | ((uint32_t)k << 14) | (1u << 19)});
    };

    uint32_t recv_flags = 0, send_flags = 0;
    bool shared = false;
    if constexpr (Q >= kSharedFrom + 2) {
        shared = runs.n_runs > 0;                          // the same for the whole block
        if (shared) {
            auto st = apply_tile_runs<Q>(runs, (int)ahead, recv_row, send_row);
            closed_form_levels<Q, kSharedFrom>(tab, st, recv_row, send_row, recv_flags, send_flags);
            closed_form_finish<Q>(tab, r, st.j, recv_row, send_row, recv_flags);
            constexpr uint32_t kLowMask = (2u << kLowFrameRounds) - 1u;
            if (low_frame != nullptr && __any_sync(0xffffffffu, ((recv_flags | send_flags) & kLowMask) != 0u)) {
                // the rank's state below the shared levels, read again from its run's description
                // rather than kept in registers across the pass
                int run = 0;
#pragma unroll
                for (int i = 1; i < kMaxRuns; ++i) run += (int)ahead >= runs.start[i] ? 1 : 0;
                const uint32_t t = ahead - (uint32_t)runs.start[run];
                const uint32_t u_low = (uint32_t)runs.state[run].rp + t;
                const int j_high = runs.state[run].j;      // lowest digit at the shared levels (Q: none)
                const bool any_recv = __any_sync(0xffffffffu, (recv_flags & kLowMask) != 0u);
                if (j_high < Q)
                    low_frame_lookups<Q>(tab, low_frame, u_low, j_high, runs.full_len[run] - t,
                                         recv_row, send_row, recv_flags, send_flags, any_recv);
            }
            // entries of the high levels that the description left undecided (at most 32, one per
            // lane); each warp takes those of its own rows, once their placeholders are written
            __syncwarp();
            const uint32_t item = (int)lane < runs.n_pending ? runs.pending[lane] : 0xffffffffu;
            // (a described tile is full, so place `a` from the lowest rank is row a, or row 255 - a)
            const uint32_t item_row = desc ? (uint32_t)kThreads - 1u - (item & 511u) : (item & 511u);
            if (item != 0xffffffffu && item_row >> 5 == warp) {
                const uint32_t row = item_row;
                const int k = (int)((item >> 9) & 31u);
                if ((item >> 14) & 1u) {
                    if (want_send) violation(row, k, r_first + (item & 511u));
                } else if (want_recv) {
                    atomicOr(&need_recv[row & 31u], 1u << k);
                }
            }
        }
    }
    if (!shared) {
        const bool is_root = r == 0u;
        int b = 0;
        recv_flags = closed_form_rows<Q>(tab, g.p, is_root ? 1u : r, recv_row, send_row, &send_flags, &b);
        if (is_root) {                                     // the root sends block k in round k
            for (int k = 0; k < Q; ++k) send_row(k, k);
            recv_flags = (2u << (Q - 1)) - 1u;             // and its receive row comes from the search
            send_flags = 0u;
        }
        if (!active) { recv_flags = 0u; send_flags = 0u; }
    }
    uint32_t todo = want_send ? send_flags : 0u;
    while (todo != 0u) {
        const int k = 31 - __clz(todo);
        todo ^= 1u << k;
        violation(index, k, r);
    }
    __syncwarp();
    const uint32_t mine = (want_recv ? recv_flags : 0u) | need_recv[lane];
    if (mine != 0u) defer(DeferredItem{r, (block_row0 + index) | ((uint32_t)(31 - __clz(mine)) << 14)});
}

}  // namespace bcast
