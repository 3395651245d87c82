// C ABI and kernels of the broadcast-schedule library (see include/bcast_sched.h).
//
// Kernels
//   schedule_table_kernel   one thread per rank, one block per run of up to 8 tiles of 256
//                           consecutive ranks.  The ranks of a tile agree on their digits at
//                           the high levels over long runs, so one warp describes those runs
//                           once (a lane per level) and every thread copies its rank's
//                           high-level entries from the description and walks only the low
//                           levels with the closed forms (schedule_fast.cuh).  Entries land as
//                           bytes in a shared-memory tile laid out exactly like the output;
//                           what the closed forms leave undecided is collected in shared-
//                           memory queues and resolved by the search of Algorithms 4 and 5
//                           (schedule_core.cuh) or copied from a neighbouring row.  The block
//                           then widens the tile to int32 and streams it out as one
//                           contiguous run of 16-byte stores, so every store instruction
//                           fills whole 32-byte sectors.
//   schedule_batch_kernel   independent (p, rank, root) queries, one per thread, sorted by q within
//                           a block so that a warp's lanes run loops of like length: receive row
//                           by the search, send row by Algorithm 6; rows padded to row_stride.
//   verify_sweep_kernel     persistent blocks pull values of p from a queue, build the tables
//                           of one p in scratch memory with the table kernel's device
//                           functions, then check the paper's correctness conditions against
//                           them and reduce a checksum.
#include <cuda_runtime.h>
#include <stdint.h>

#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "../../include/bcast_sched.h"
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
// The launch shape of bcast_schedule proper.  After the run descriptions are built no warp
// waits for another: each takes its own 32 rows of every tile through the closed-form pass
// and streams them out at once, undecided entries included (with whatever the pass left
// there).  What is undecided goes to ONE queue per block, and when all tiles are out the
// whole block runs the searches side by side, every lane busy, and stores each found entry
// straight into the output table, over the placeholder.  (Per tile, the undecided entries of
// 256 rows keep only a third of a block's lanes busy; per warp even fewer.)
//
// A deferred item names a virtual rank whose receive schedule is searched, the output row
// (relative to the block's first row) and two sets of rounds:
//   own rows  (kind 0): recv_mask  - rounds of the row's receive entries;
//                       other_mask - rounds k whose value ALSO is the send entry of the row
//                                    skip[k] above (its to-processor is this row, Section 2.3),
//                                    noted by that row's lane when Algorithm 6 could not
//                                    decide it and both rows belong to the same warp;
//   send only (kind 1): other_mask - rounds k of the row's SEND entries, `rank` being the
//                                    row's to-processor for that round.
struct DeferredItem {
    uint32_t rank;
    uint32_t row_kind;                                     // row | kind << 31
    uint32_t recv_mask;
    uint32_t other_mask;
};

constexpr int kDeferredCapacity = 384;
constexpr int kDescWarpsFromQ = 16;                    // smallest q with a descending-rows kernel of that shape

struct DeferredQueue {
    DeferredItem items[kDeferredCapacity];
    uint32_t need_recv[kWarpsPerBlock][32];                // per warp and row of its slice: rounds to search
    uint32_t need_partner[kWarpsPerBlock][32];             // rounds whose value the row skip[k] above sends
    int n;
};

union QueueStorage {
    TileQueue tile;                                        // one queue for the block, or
    DeferredQueue deferred;                                // the block's deferred searches
};

// Search for one deferred item; emit(table, row, k, value) receives every wanted entry
// (table 0 = receive, 1 = send; row relative to the block's first row).
template <bool desc, class Emit>
__device__ __forceinline__ void resolve_deferred(const Geometry &g, const LevelTables &tab, const DeferredItem &it,
                                                 Emit emit)
{
    const uint32_t row = it.row_kind & 0x7fffffffu;
    const bool send_only = (it.row_kind >> 31) != 0u;
    const uint32_t recv_mask = it.recv_mask, other_mask = it.other_mask;
    NoStats ns;
    recv_search_fast(g, it.rank, 31 - __clz(recv_mask | other_mask), [&](int k, int val) {
        if ((recv_mask >> k) & 1u) emit(0, row, k, val);
        // the row whose to-processor this row is: skip[k] ranks below, i.e. skip[k] rows above it when the
        // rows are listed by descending rank
        if ((other_mask >> k) & 1u)
            emit(1, send_only ? row : (desc ? row + tab.skip[k] : row - tab.skip[k]), k, val);
    }, ns);
}

// The closed-form pass of one warp's 32 rows of a tile (lane l owns row 32*warp + l).  Rounds
// the pass cannot decide become deferred items; when the block's queue is full the lane runs
// the search itself and puts the entries into the staged rows, which are not flushed yet.
template <int Q, bool desc, class Tile>
__device__ __forceinline__ void warp_pass(const LevelTables &tab, const Geometry &g,
                                          const TileRuns<typename WalkInt<Q>::type> &runs,
                                          uint32_t r_first, uint32_t rows, uint32_t block_row0, const Tile &tile,
                                          bool want_recv, bool want_send, DeferredQueue &dq)
{
    // index: the thread's row of the staged tile = its output row within the tile.  The ranks of a tile
    // ascend with the row, or descend (Algorithm 7's tables); `ahead` is the thread's place counted from
    // the tile's lowest rank r_first, which is how the run descriptions number the rows.
    const uint32_t index = threadIdx.x;
    const uint32_t lane = index & 31u;
    const uint32_t warp = index >> 5;
    uint32_t *need_recv = dq.need_recv[warp];
    uint32_t *need_partner = dq.need_partner[warp];
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
    need_partner[lane] = 0u;
    __syncwarp();

    auto defer = [&](const DeferredItem &it) {
        const int slot = atomicAdd(&dq.n, 1);
        if (slot < kDeferredCapacity) {
            dq.items[slot] = it;
        } else {
            resolve_deferred<desc>(g, tab, it, [&](int table, uint32_t row, int k, int val) {
                const uint32_t in_tile = row - block_row0;
                if (table == 0) tile.recv_row(in_tile)(k, val); else tile.send_row(in_tile)(k, val);
            });
        }
    };
    // Algorithm 6 could not decide round k of the send row of tile row `row` (virtual rank rr)
    auto violation = [&](uint32_t row, int k, uint32_t rr) {
        const uint32_t skip_k = tab.skip[k];
        // the to-processor's row: skip[k] ranks ahead; its lane will search the entry if it is in this warp
        const bool near = desc ? (row & 31u) >= skip_k : (row & 31u) + skip_k < 32u && row + skip_k < rows;
        if (want_recv && near) {
            atomicOr(&need_partner[desc ? (row & 31u) - skip_k : (row & 31u) + skip_k], 1u << k);
        } else {
            uint32_t t = rr + skip_k;
            if (t >= g.p) t -= g.p;
            defer(DeferredItem{t, (block_row0 + row) | 0x80000000u, 0u, 1u << k});
        }
    };

    uint32_t recv_flags = 0, send_flags = 0;
    bool shared = false;
    if constexpr (Q >= kSharedFrom + 2) {
        shared = runs.n_runs > 0;                          // the same for the whole block
        if (shared) {
            auto st = apply_tile_runs<Q>(runs, (int)ahead, recv_row, send_row);
            closed_form_levels<Q, kSharedFrom>(tab, st, recv_row, send_row, recv_flags, send_flags);
            closed_form_finish<Q>(tab, r, st.j, recv_row, send_row, recv_flags);
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
    if (want_recv && recv_flags != 0u) atomicOr(&need_recv[lane], recv_flags);
    uint32_t todo = want_send ? send_flags : 0u;
    while (todo != 0u) {
        const int k = 31 - __clz(todo);
        todo ^= 1u << k;
        violation(index, k, r);
    }
    __syncwarp();
    const uint32_t mine = need_recv[lane], partner = need_partner[lane];
    if ((mine | partner) != 0u) defer(DeferredItem{r, block_row0 + index, mine, partner});
}


// kDescWarps = false: the kernel of bcast_schedule and its variants, either launch shape, rows by
// ascending rank in the warps-on-their-own shape.  kDescWarps = true: only that shape, rows by
// descending rank (Algorithm 7's tables); a kernel of its own so that the other one is compiled
// exactly as it would be without it.
template <int Q, bool kDescWarps>
__global__ void __launch_bounds__(kThreads, kTableBlocksPerSm)
schedule_table_kernel(const __grid_constant__ LevelTables tab, uint32_t p, uint32_t anchor,
                      uint32_t row_begin, uint32_t n_ranks, int descending, int tiles_per_block,
                      int32_t *__restrict__ recv_out, int32_t *__restrict__ send_out,
                      int recv_vec_ok, int send_vec_ok, int shift_x, int warps_alone)
{
    typedef typename WalkInt<Q>::type Int;
    __shared__ uint32_t stage[2][(kThreads * Q + 15) / 16 * 4];   // byte tiles, kThreads rows of Q entries
    __shared__ QueueStorage queues;
    __shared__ LevelTables lookup;                         // the tables again, for per-lane indices
    __shared__ TileRuns<Int> runs[kWarpsPerBlock];         // descriptions of the next kWarpsPerBlock tiles
    __shared__ uint32_t shift_words[32];                   // used only when shift_x != 0
    const Geometry g = make_geometry(p);
    const uint32_t n_tiles = (n_ranks + kThreads - 1u) / kThreads;
    const bool want_recv = recv_out != nullptr;
    const bool want_send = send_out != nullptr;
    int8_t *const recv_bytes = reinterpret_cast<int8_t *>(stage[0]);
    int8_t *const send_bytes = reinterpret_cast<int8_t *>(stage[1]);
    // Output row x (global index row_begin + x) holds virtual rank (index - anchor) mod p, anchor
    // being the root (bcast_schedule), or (anchor - index) mod p, anchor being the processor and
    // the index the root (bcast_allbroadcast_schedule).  A tile's first virtual rank, ascending:
    auto first_rank_of = [&](uint32_t first, uint32_t rows) {
        const uint32_t lo = row_begin + first;
        if (!descending) return lo >= anchor ? lo - anchor : lo + (p - anchor);
        const uint32_t hi = lo + rows - 1u;
        return anchor >= hi ? anchor - hi : anchor + (p - hi);
    };
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    NoStats ns;
    if (threadIdx.x <= Q) lookup.skip[threadIdx.x] = tab.skip[threadIdx.x];
    if (threadIdx.x <= Q + 1) lookup.below[threadIdx.x] = tab.below[threadIdx.x];
    if (shift_x != 0) fill_shift_words<Q>(shift_words, shift_x);
    __syncthreads();

    // This block's tiles: tiles_per_block (at most kWarpsPerBlock) consecutive ones.  Each warp first
    // describes the runs of one of them, then the block goes through them.  Many short-lived blocks
    // instead of a persistent grid: the hardware's block scheduler evens out the load, which measured
    // 12 % faster than striding a resident grid over the tiles.
    const uint32_t group = blockIdx.x * (uint32_t)tiles_per_block;
    {
        const uint32_t t = group + (uint32_t)warp;
        bool share = false;
        if (warp < tiles_per_block && t < n_tiles) {
            const uint32_t first = t * kThreads;
            const uint32_t rows = min((uint32_t)kThreads, n_ranks - first);
            const uint32_t r_first = first_rank_of(first, rows);
            share = tile_can_share<Q>(g, r_first, rows);
            if constexpr (Q >= kSharedFrom + 2)
                if (share) build_tile_runs<Q>(tab, lookup, p, r_first, (int)rows, lane, runs[warp]);
        }
        if (!share && lane == 0) { runs[warp].n_runs = 0; runs[warp].n_pending = 0; }
    }
    if (kDescWarps || warps_alone) {                       // host: never with the shifted rows
        constexpr bool desc = kDescWarps;
        DeferredQueue &dq = queues.deferred;
        if (threadIdx.x == 0) dq.n = 0;
        __syncthreads();                                   // descriptions built, queue empty
        for (int slot = 0; slot < tiles_per_block; ++slot) {
            const uint32_t t = group + (uint32_t)slot;
            if (t >= n_tiles) break;
            const uint32_t first = t * kThreads;
            const uint32_t rows = min((uint32_t)kThreads, n_ranks - first);
            const SharedTile<Q> tile{recv_bytes, send_bytes, rows, false};
            warp_pass<Q, desc>(tab, g, runs[slot], first_rank_of(first, rows), rows, (uint32_t)slot * kThreads,
                               tile, want_recv, want_send, dq);
            __syncwarp();                                  // the slice is staged
            const uint32_t my_first = (uint32_t)warp * 32u;
            if (my_first < rows) {
                const int my_entries = (int)min(32u, rows - my_first) * Q;
                const size_t base = (size_t)(first + my_first) * (size_t)Q;
                const uint32_t word = my_first * Q / 4u;   // 32 rows of Q bytes are whole words
                if (want_recv) flush_tile<32>(stage[0] + word, recv_out + base, my_entries, recv_vec_ok, lane);
                if (want_send) flush_tile<32>(stage[1] + word, send_out + base, my_entries, send_vec_ok, lane);
            }
            __syncwarp();                                  // flushed before the next tile's pass overwrites it
        }
        __syncthreads();                                   // every slice is out; now the searches
        const int n_deferred = min(dq.n, kDeferredCapacity);
        const size_t block_base = (size_t)group * kThreads * (size_t)Q;
        for (int i = threadIdx.x; i < n_deferred; i += kThreads) {
            resolve_deferred<desc>(g, tab, dq.items[i], [&](int table, uint32_t row, int k, int val) {
                int32_t *out = table == 0 ? recv_out : send_out;
                out[block_base + (size_t)row * Q + k] = val;
            });
        }
        return;
    }
    TileQueue &queue = queues.tile;
    for (int slot = 0; slot < tiles_per_block; ++slot) {
        const uint32_t t = group + (uint32_t)slot;
        if (t >= n_tiles) break;
        if (threadIdx.x == 0) { queue.n_search = 0; queue.n_long = 0; queue.n_copy = 0; }
        __syncthreads();                                   // descriptions built; previous tile flushed
        const uint32_t first = t * kThreads;
        const uint32_t rows = min((uint32_t)kThreads, n_ranks - first);
        const SharedTile<Q> tile{recv_bytes, send_bytes, rows, descending != 0};
        tile_pass<Q>(tab, g, runs[slot], first_rank_of(first, rows), rows, tile, want_recv, want_send,
                     queue, ns);
        __syncthreads();
        if (queue.n_search + queue.n_long + queue.n_copy > 0) {           // the same for every thread
            drain_queue(g, queue, tile, ns);
            __syncthreads();
        }
        const size_t base = (size_t)first * (size_t)Q;
        if (shift_x != 0) {                                // rows as Algorithm 1 starts with them for n blocks
            if (want_recv)
                flush_tile_shifted<Q>(stage[0], shift_words, recv_out + base, (int)rows * Q, recv_vec_ok, shift_x);
            if (want_send)
                flush_tile_shifted<Q>(stage[1], shift_words, send_out + base, (int)rows * Q, send_vec_ok, shift_x);
            continue;
        }
        if (want_recv) flush_tile<kThreads>(stage[0], recv_out + base, (int)rows * Q, recv_vec_ok, threadIdx.x);
        if (want_send) flush_tile<kThreads>(stage[1], send_out + base, (int)rows * Q, send_vec_ok, threadIdx.x);
    }
}

// ------------------------------------------------------------------ independent queries
// A block takes kThreads consecutive queries.  Their q = ceil(log2 p) differ (1..31 for p drawn
// log-uniformly), and every loop of the per-rank computation runs q or a few q times, so a
// warp whose lanes hold unlike q idles most lanes most of the time.  The block therefore sorts
// its queries by q (a counting sort in shared memory, longest first) and thread t computes the
// query in position t of that order; rows are staged in shared memory at the query's own
// position, so the output stays in the caller's order.
constexpr int kBatchItems = 4 * kThreads;              // Theorem 3: at most four undecided rounds per query
constexpr int kBatchRowBytes = 36;                     // staged row: 31 entries + pad; 9 words keep 32 rows on 32 banks

__global__ void __launch_bounds__(kThreads)
schedule_batch_kernel(const int32_t *__restrict__ p_in, const int32_t *__restrict__ rank_in,
                      const int32_t *__restrict__ root_in, int64_t nq, int row_stride,
                      int32_t *__restrict__ recv_out, int32_t *__restrict__ send_out,
                      int32_t *bad_count, int recv_vec_ok, int send_vec_ok)
{
    __shared__ uint32_t stage[2][kThreads * kBatchRowBytes / 4];
    __shared__ uint32_t query_p[kThreads];             // p of the query in each row (0: nothing to compute)
    __shared__ uint32_t query_r[kThreads];             // its virtual rank
    __shared__ uint16_t order[kThreads];               // rows sorted by q, longest first
    __shared__ int bin_count[32];
    __shared__ int bin_start[32];
    __shared__ uint16_t items[kBatchItems];            // undecided send entries: row | k << 8
    __shared__ int n_items;
    const bool want_recv = recv_out != nullptr;
    const bool want_send = send_out != nullptr;
    constexpr int8_t kPadMark = -128;                  // no schedule entry is below -31
    const int64_t n_tiles = (nq + kThreads - 1) / kThreads;

    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t first = tile * kThreads;
        const int rows = (int)min((int64_t)kThreads, nq - first);
        if (threadIdx.x < 32) bin_count[threadIdx.x] = 0;
        if (threadIdx.x == 32) n_items = 0;
        __syncthreads();                               // previous tile flushed, bins cleared
        int q = 0, slot = 0;
        {
            uint32_t p = 0, r = 0;
            if ((int)threadIdx.x < rows) {
                const int64_t idx = first + threadIdx.x;
                const int32_t pi = p_in[idx], ai = rank_in[idx], ri = root_in[idx];
                const bool ok = pi >= 1 && ai >= 0 && ai < pi && ri >= 0 && ri < pi;
                if (!ok) {
                    if (bad_count) atomicAdd(bad_count, 1);
                } else if (pi >= 2) {
                    p = (uint32_t)pi;
                    q = 32 - __clz(p - 1u);
                    r = ai >= ri ? (uint32_t)(ai - ri) : (uint32_t)ai + (p - (uint32_t)ri);
                }
            }
            query_p[threadIdx.x] = p;
            query_r[threadIdx.x] = r;
            slot = atomicAdd(&bin_count[q], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {                        // bins in descending q: start = rows with a larger q
            int above = 0;
            for (int b = threadIdx.x + 1; b < 32; ++b) above += bin_count[b];
            bin_start[threadIdx.x] = above;
        }
        __syncthreads();
        order[bin_start[q] + slot] = (uint16_t)threadIdx.x;
        __syncthreads();

        {
            const int row = order[threadIdx.x];
            const uint32_t p = query_p[row];
            const ByteRow recv_row{reinterpret_cast<int8_t *>(stage[0]) + row * kBatchRowBytes};
            const ByteRow send_row{reinterpret_cast<int8_t *>(stage[1]) + row * kBatchRowBytes};
            int qq = 0;
            uint32_t viol = 0;
            if (p >= 2u) {
                const Geometry g = make_geometry(p);
                qq = g.q;
                const uint32_t r = query_r[row];
                NoStats ns;
                const int b = want_recv ? recv_search_fast(g, r, qq - 1, recv_row, ns) : baseblock(g, r);
                if (want_send) {
                    if (r == 0u) {
                        for (int k = 0; k < qq; ++k) send_row(k, k);
                    } else {
                        viol = send_walk(g, r, b, send_row);
                    }
                }
            }
            for (int k = qq; k < kMaxRowBytes; ++k) { recv_row(k, kPadMark); send_row(k, kPadMark); }
            // Rounds Algorithm 6 could not decide (at most four per query, Theorem 3) are queued
            // for the whole block, so that the lanes that have one do not hold up the others;
            // a warp's items stay together, which keeps like q side by side.
            const int lane = threadIdx.x & 31;
            while (__any_sync(0xffffffffu, viol != 0u)) {
                const bool has = viol != 0u;
                const unsigned int mask = __ballot_sync(0xffffffffu, has);
                int base = 0;
                if (lane == 0) base = atomicAdd(&n_items, __popc(mask));
                base = __shfl_sync(0xffffffffu, base, 0);
                if (has) {
                    const int k = 31 - __clz(viol);
                    viol ^= 1u << k;
                    const int at = base + __popc(mask & ((1u << lane) - 1u));
                    if (at < kBatchItems) {
                        items[at] = (uint16_t)(row | (k << 8));
                    } else {                               // cannot happen by Theorem 3; done on the spot
                        const Geometry g = make_geometry(p);
                        uint32_t t = query_r[row] + skip_of(g, k);
                        if (t >= g.p) t -= g.p;
                        NoStats ns;
                        send_row(k, recv_entry(g, t, k, ns));
                    }
                }
            }
        }
        __syncthreads();
        {
            const int n = min(n_items, kBatchItems);
            for (int i = threadIdx.x; i < n; i += kThreads) {
                const int row = items[i] & 255;
                const int k = items[i] >> 8;
                const Geometry g = make_geometry(query_p[row]);
                uint32_t t = query_r[row] + skip_of(g, k);
                if (t >= g.p) t -= g.p;
                NoStats ns;
                const ByteRow send_row{reinterpret_cast<int8_t *>(stage[1]) + row * kBatchRowBytes};
                send_row(k, recv_entry(g, t, k, ns));      // Section 2.3: recvblock[k] of the to-processor
            }
        }
        __syncthreads();

        const int n_entries = rows * row_stride;
        for (int t = 0; t < 2; ++t) {
            int32_t *out = t == 0 ? recv_out : send_out;
            if (out == nullptr) continue;
            out += (size_t)first * (size_t)row_stride;
            const int8_t *bytes = reinterpret_cast<const int8_t *>(stage[t]);
            const bool vec_ok = (t == 0 ? recv_vec_ok : send_vec_ok) && (row_stride & 3) == 0;
            if (vec_ok) {
                int4 *out4 = reinterpret_cast<int4 *>(out);
                const int nvec = n_entries >> 2;
                const int vec_per_row = row_stride >> 2;
                for (int i = threadIdx.x; i < nvec; i += kThreads) {
                    const int row = i / vec_per_row;
                    const int col = (i - row * vec_per_row) << 2;
                    int e[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int cc = col + j;
                        const int val = cc < kMaxRowBytes ? (int)bytes[row * kBatchRowBytes + cc] : (int)kPadMark;
                        e[j] = val == (int)kPadMark ? BCAST_PAD : val;
                    }
                    __stcs(out4 + i, make_int4(e[0], e[1], e[2], e[3]));
                }
            } else {
                for (int i = threadIdx.x; i < n_entries; i += kThreads) {
                    const int row = i / row_stride;
                    const int cc = i - row * row_stride;
                    const int val = cc < kMaxRowBytes ? (int)bytes[row * kBatchRowBytes + cc] : (int)kPadMark;
                    __stcs(out + i, val == (int)kPadMark ? BCAST_PAD : val);
                }
            }
        }
    }
}

// ------------------------------------------------------------------ verification sweep
__device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z ^= z >> 30; z *= 0xbf58476d1ce4e5b9ULL;
    z ^= z >> 27; z *= 0x94d049bb133111ebULL;
    z ^= z >> 31;
    return z;
}

// Level tables of p, built by the block itself (skip[] by Algorithm 2's closed form).
__device__ __forceinline__ void fill_tables(LevelTables &tab, const Geometry &g)
{
    if (threadIdx.x == 0) {
        uint32_t sum = 0;
        for (int l = 0; l <= g.q; ++l) {
            const uint32_t s = skip_of(g, l);
            tab.skip[l] = s;
            tab.below[l] = sum;
            sum += s;
        }
        tab.below[g.q + 1] = sum;
    }
}

// The sweep's tile: kThreads consecutive ranks of the round-major tables of one p, which
// have p + 1 slots per round; slot p takes the stand-in rows of lanes beyond the last rank.
struct ScratchTile {
    int8_t *recv_tab;
    int8_t *send_tab;
    uint32_t first;
    uint32_t p;
    __device__ __forceinline__ uint32_t slot(uint32_t i) const { return first + i < p ? first + i : p; }
    __device__ __forceinline__ StridedColumn recv_row(uint32_t i) const
    { return StridedColumn{recv_tab + slot(i), (size_t)p + 1u}; }
    __device__ __forceinline__ StridedColumn send_row(uint32_t i) const
    { return StridedColumn{send_tab + slot(i), (size_t)p + 1u}; }
};

// Both tables of one p into the block's scratch, with the table kernel's own pass, queues
// and run descriptions, kThreads ranks at a time.  Called by every thread of the block;
// adds to the thread's failure counters [4] (violations), [5] (search bounds), [7] (cap).
template <int Q>
__device__ __forceinline__ void sweep_tables_of_p(const LevelTables &tab, const Geometry &g, int8_t *recv_tab,
                                                  int8_t *send_tab, TileQueue &queue, void *runs_storage,
                                                  uint32_t *row_viol, uint32_t *fail)
{
    typedef typename WalkInt<Q>::type Int;
    TileRuns<Int> *runs = reinterpret_cast<TileRuns<Int> *>(runs_storage);
    const uint32_t p = g.p;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    for (uint32_t group = 0; group < p; group += kThreads * kWarpsPerBlock) {
        {
            const uint32_t first = group + (uint32_t)warp * kThreads;
            bool share = false;
            if (first < p) {
                const uint32_t rows = min((uint32_t)kThreads, p - first);
                share = tile_can_share<Q>(g, first, rows);
                if constexpr (Q >= kSharedFrom + 2)
                    if (share) build_tile_runs<Q>(tab, tab, p, first, (int)rows, lane, runs[warp]);
            }
            if (!share && lane == 0) { runs[warp].n_runs = 0; runs[warp].n_pending = 0; }
        }
        for (int slot = 0; slot < kWarpsPerBlock; ++slot) {
            const uint32_t first = group + (uint32_t)slot * kThreads;
            if (first >= p) break;
            if (threadIdx.x == 0) { queue.n_search = 0; queue.n_long = 0; queue.n_copy = 0; }
            row_viol[threadIdx.x] = 0u;
            __syncthreads();
            const ScratchTile tile{recv_tab, send_tab, first, p};
            const uint32_t rows = min((uint32_t)kThreads, p - first);
            CountStats st;
            st.row_violations = row_viol;
            uint32_t viol = tile_pass<Q>(tab, g, runs[slot], first, rows, tile, true, true, queue, st);
            __syncthreads();
            viol |= row_viol[threadIdx.x];                 // violations noted by the run descriptions
            if (__popc(viol) > 4) fail[4]++;
            drain_queue(g, queue, tile, st);
            // Lemmas 5 and 6, over the searches this thread ran for the tile
            if (st.s.capped) fail[7]++;
            if (st.s.over_bound) fail[5]++;
        }
        __syncthreads();
    }
}

// Work queue: *queue_next counts values of p handed out, largest p first.
__global__ void __launch_bounds__(kThreads, kSweepBlocksPerSm)
verify_sweep_kernel(uint32_t p_lo, uint32_t p_hi, uint64_t *__restrict__ checksum_out,
                    uint32_t *__restrict__ fail_counts, int8_t *scratch,
                    size_t scratch_per_block, unsigned int *queue_next)
{
    __shared__ uint32_t s_p;
    __shared__ uint64_t s_sum[kWarpsPerBlock];
    __shared__ uint32_t s_fail[8];
    __shared__ LevelTables s_tab;
    __shared__ uint32_t s_row_viol[kThreads];
    __shared__ __align__(16) unsigned char s_runs[sizeof(TileRuns<int64_t>) * kWarpsPerBlock];
    __shared__ TileQueue queue;
    int8_t *tab = scratch + (size_t)blockIdx.x * scratch_per_block;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;

    while (true) {
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned int ticket = atomicAdd(queue_next, 1u);
            s_p = ticket <= p_hi - p_lo ? p_hi - ticket : 0u;
        }
        if (threadIdx.x < 8) s_fail[threadIdx.x] = 0u;
        __syncthreads();
        const uint32_t p = s_p;
        if (p == 0u) break;
        if (p == 1u) {
            if (threadIdx.x == 0) checksum_out[p - p_lo] = 0ull;
            continue;
        }
        const Geometry g = make_geometry(p);
        const int q = g.q;
        fill_tables(s_tab, g);
        __syncthreads();
        // tables of this p, round-major so that the checks read coalesced: tab[k*(p+1) + r]
        const size_t stride = (size_t)p + 1u;
        int8_t *recv_tab = tab;
        int8_t *send_tab = tab + (size_t)q * stride;
        uint32_t fail[8] = {0, 0, 0, 0, 0, 0, 0, 0};

        switch (q) {
#define BCAST_CASE(N) case N: sweep_tables_of_p<N>(s_tab, g, recv_tab, send_tab, queue, s_runs, s_row_viol, fail); break;
            BCAST_CASE(1) BCAST_CASE(2) BCAST_CASE(3) BCAST_CASE(4) BCAST_CASE(5) BCAST_CASE(6)
            BCAST_CASE(7) BCAST_CASE(8) BCAST_CASE(9) BCAST_CASE(10) BCAST_CASE(11) BCAST_CASE(12)
            BCAST_CASE(13) BCAST_CASE(14) BCAST_CASE(15) BCAST_CASE(16) BCAST_CASE(17) BCAST_CASE(18)
            BCAST_CASE(19) BCAST_CASE(20) BCAST_CASE(21) BCAST_CASE(22) BCAST_CASE(23) BCAST_CASE(24)
            BCAST_CASE(25) BCAST_CASE(26) BCAST_CASE(27) BCAST_CASE(28) BCAST_CASE(29) BCAST_CASE(30)
            BCAST_CASE(31)
#undef BCAST_CASE
        }
        __syncthreads();

        uint64_t sum = 0;
        for (uint32_t r = threadIdx.x; r < p; r += kThreads) {
            uint64_t seen = 0;                      // blocks received so far, bit (value + q)
            int base = -1;                          // the non-negative received block
            int first_send = 0;
            for (int k = 0; k < q; ++k) {
                const int rv = recv_tab[(size_t)k * stride + r];
                const int sv = send_tab[(size_t)k * stride + r];
                const uint32_t sk = skip_of(g, k);
                const uint32_t f = r >= sk ? r - sk : r + (p - sk);
                uint32_t t = r + sk; if (t >= p) t -= p;
                if (rv != (int)send_tab[(size_t)k * stride + f]) fail[0]++;
                if (sv != (int)recv_tab[(size_t)k * stride + t]) fail[1]++;
                if (k == 0) first_send = sv;
                if (r != 0u && k > 0) {
                    // condition 4: sent block was received earlier, or is b - q (= sendblock[0])
                    const bool held = ((seen >> ((sv + q) & 63)) & 1ull) != 0ull || sv == first_send;
                    if (!held) fail[3]++;
                }
                if (r == 0u && sv != k) fail[6]++;
                if (rv >= 0) base = rv;
                seen |= 1ull << ((rv + q) & 63);
                const uint64_t key = ((uint64_t)r << 32) | ((uint64_t)k << 16)
                                   | ((uint64_t)(rv & 0xff) << 8) | (uint64_t)(sv & 0xff);
                sum += mix64(key);
            }
            // condition 3 (and the root's row)
            uint64_t want = (1ull << q) - 1ull;
            if (r != 0u) {
                if (base < 0) { fail[2]++; }
                else {
                    want = (want & ~(1ull << base)) | (1ull << (base + q));
                    if (first_send != base - q) fail[6]++;
                    if (base != baseblock(g, r)) fail[2]++;
                }
            }
            if (seen != want) fail[2]++;
        }
        // block reduction of the checksum and the failure counters
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, off);
        if (lane == 0) s_sum[warp] = sum;
        for (int i = 0; i < 8; ++i)
            if (fail[i] != 0u) atomicAdd(&s_fail[i], fail[i]);
        __syncthreads();
        if (threadIdx.x == 0) {
            uint64_t total = 0;
            for (int w = 0; w < kWarpsPerBlock; ++w) total += s_sum[w];
            checksum_out[p - p_lo] = total;
        }
        if (threadIdx.x < 8 && s_fail[threadIdx.x] != 0u) atomicAdd(&fail_counts[threadIdx.x], s_fail[threadIdx.x]);
    }
}

__global__ void zero_counter_kernel(unsigned int *c) { *c = 0u; }

// ------------------------------------------------------------------ host helpers
static int host_q(int64_t p)
{
    int q = 0;
    while (((int64_t)1 << q) < p) ++q;
    return q;
}

static int sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    return sms;
}

static LevelTables host_tables(int64_t p, int q)
{
    LevelTables tab = {};
    int64_t s = p;
    tab.skip[q] = (uint32_t)p;
    for (int k = q; k > 0; --k) {
        s = s - s / 2;
        tab.skip[k - 1] = (uint32_t)s;
    }
    uint32_t sum = 0;
    for (int l = 0; l <= q; ++l) {
        tab.below[l] = sum;
        sum += tab.skip[l];
    }
    tab.below[q + 1] = sum;
    return tab;
}

static int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

static int64_t sweep_bytes_per_block(int32_t p_hi)
{
    return round_up((int64_t)2 * host_q(p_hi) * ((int64_t)p_hi + 1), 256);
}

constexpr int64_t kSweepHeaderBytes = 256;             // the work-queue counter lives here

// Arguments of one launch of the table kernel, and the launch for a given q.
struct TableLaunch {
    LevelTables tab;
    uint32_t p, anchor, row_begin, n_rows;
    int descending, tiles_per_block;
    int32_t *recv_dev, *send_dev;
    int recv_vec, send_vec, shift_x, asc_warps;
    bool desc_warps;
    int grid;
    cudaStream_t stream;
};

template <int N>
static void launch_table_kernel(const TableLaunch &l)
{
    if constexpr (N >= kDescWarpsFromQ) {
        if (l.desc_warps) {
            schedule_table_kernel<N, true><<<l.grid, kThreads, 0, l.stream>>>(
                l.tab, l.p, l.anchor, l.row_begin, l.n_rows, l.descending, l.tiles_per_block, l.recv_dev,
                l.send_dev, l.recv_vec, l.send_vec, l.shift_x, 0);
            return;
        }
    }
    schedule_table_kernel<N, false><<<l.grid, kThreads, 0, l.stream>>>(
        l.tab, l.p, l.anchor, l.row_begin, l.n_rows, l.descending, l.tiles_per_block, l.recv_dev, l.send_dev,
        l.recv_vec, l.send_vec, l.shift_x, l.asc_warps);
}

}  // namespace bcast

using namespace bcast;

extern "C" {

const char *bcast_strerror(int code)
{
    switch (code) {
    case BCAST_OK:            return "success";
    case BCAST_EINVAL_P:      return "p must satisfy 1 <= p <= 2^31-1";
    case BCAST_EINVAL_ROOT:   return "root must satisfy 0 <= root < p";
    case BCAST_EINVAL_RANGE:  return "range must satisfy 0 <= begin <= end <= p (or p_lo <= p_hi)";
    case BCAST_ENULL:         return "a required pointer is NULL";
    case BCAST_EALIGN:        return "a device pointer is not aligned as documented";
    case BCAST_EINVAL_N:      return "n, q and nq must be positive (nq may be 0)";
    case BCAST_EINVAL_ROUND:  return "round j must satisfy 0 <= j < n-1+q";
    case BCAST_ECUDA:         return "a CUDA runtime call failed";
    case BCAST_ESTRIDE:       return "row_stride must be at least 31";
    case BCAST_ESCRATCH:      return "scratch buffer too small";
    case BCAST_ETOOBIG:       return "p_hi exceeds what the built-in scratch of bcast_verify_sweep_static holds";
    default:                  return code > 0 ? "success" : "unknown error code";
    }
}

int bcast_q(int32_t p)
{
    if (p < 1) return BCAST_EINVAL_P;
    return host_q(p);
}

int bcast_skips(int32_t p, int32_t *skip_host)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (skip_host == nullptr) return BCAST_ENULL;
    const int q = host_q(p);
    int64_t s = p;
    skip_host[q] = p;
    for (int k = q; k > 0; --k) {
        s = s - s / 2;
        skip_host[k - 1] = (int32_t)s;
    }
    return q;
}

// Algorithm 6's violations of virtual rank r (1 <= r < p), counted on the host.
static int host_violations(const LevelTables &tab, int64_t p, int q, int64_t r)
{
    int64_t rp = r, e = p;
    int b = q;                                             // baseblock: only "b > 0" matters below
    {
        int64_t rem = r;
        for (int k = q - 1; k >= 0; --k) {
            if ((int64_t)tab.skip[k] == rem) { b = k; break; }
            if ((int64_t)tab.skip[k] < rem) rem -= tab.skip[k];
        }
    }
    int count = 0;
    for (int k = q - 1; k >= 1; --k) {
        const int64_t sk = tab.skip[k], sk_below = tab.skip[k - 1];
        if (rp < sk) {
            if (!(rp + sk < e || e < sk_below || (k == 1 && b > 0))) ++count;
            if (e > sk) e = sk;
        } else {
            if (!(k == 1 || rp > sk || e - sk < sk_below) && rp + sk > e) ++count;
            rp -= sk;
            e -= sk;
        }
    }
    return count;
}

// Which launch shape suits p: with few undecided entries per tile the warps go through the
// tiles on their own and the block runs the few searches at the end (the deferred queue of a
// block holds kDeferredCapacity items for up to kWarpsPerBlock tiles); with many, the block
// meets after every tile and drains them there.  The density is estimated from Algorithm 6's
// violations on a fixed sample of ranks; a wrong guess costs time, never correctness.
static bool few_undecided_entries(const LevelTables &tab, int64_t p, int q)
{
    if (q < 2) return true;
    const int kSamples = 80;
    const int kMost = kSamples / 20;                       // at most 0.05 per rank
    int total = 0;
    uint64_t state = 0x9e3779b97f4a7c15ull ^ (uint64_t)p;
    for (int i = 0; i < kSamples && total <= kMost; ++i) {
        state = state * 6364136223846793005ull + 1442695040888963407ull;
        const int64_t r = 1 + (int64_t)((state >> 33) % (uint64_t)(p - 1));
        total += host_violations(tab, p, q, r);
    }
    return total <= kMost;
}

// Launch of the table kernel for n_rows output rows starting at global row index row_begin.
static int launch_table(int32_t p, int q, int32_t anchor, int64_t row_begin, int64_t n_rows, int descending,
                        int32_t *recv_dev, int32_t *send_dev, void *cuda_stream, int shift_x = 0)
{
    const int sms = sm_count();
    if (sms <= 0) return BCAST_ECUDA;
    const int64_t n_tiles = (n_rows + kThreads - 1) / kThreads;
    // up to kWarpsPerBlock consecutive tiles per block, fewer while the grid would have less than
    // kBlocksPerSmWanted blocks per SM (short launches want many small blocks)
    int64_t tiles_per_block = n_tiles / ((int64_t)sms * kBlocksPerSmWanted);
    if (tiles_per_block < 1) tiles_per_block = 1;
    if (tiles_per_block > kWarpsPerBlock) tiles_per_block = kWarpsPerBlock;
    const int grid = (int)((n_tiles + tiles_per_block - 1) / tiles_per_block);
    const LevelTables tab = host_tables(p, q);
    const int recv_vec = ((uintptr_t)recv_dev & 15u) == 0, send_vec = ((uintptr_t)send_dev & 15u) == 0;
    // BCAST_LAUNCH_SHAPE=block|warps overrides the estimate (for tuning and for the tests, which
    // run both shapes on the same p); results never depend on it
    bool few = false;
    if (shift_x == 0) {
        const char *forced = getenv("BCAST_LAUNCH_SHAPE");
        if (forced != nullptr && strcmp(forced, "block") == 0) few = false;
        else if (forced != nullptr && strcmp(forced, "warps") == 0) few = true;
        else few = few_undecided_entries(tab, p, q);
    }
    const int warps_alone = few ? 1 : 0;
    // rows by descending rank take the warps-on-their-own shape only for q >= kDescWarpsFromQ (the
    // sizes where it matters; each q is a kernel to compile), else the block-per-tile shape
    TableLaunch launch;
    launch.tab = tab;
    launch.p = (uint32_t)p;
    launch.anchor = (uint32_t)anchor;
    launch.row_begin = (uint32_t)row_begin;
    launch.n_rows = (uint32_t)n_rows;
    launch.descending = descending;
    launch.tiles_per_block = (int)tiles_per_block;
    launch.recv_dev = recv_dev;
    launch.send_dev = send_dev;
    launch.recv_vec = recv_vec;
    launch.send_vec = send_vec;
    launch.shift_x = shift_x;
    launch.asc_warps = !descending && warps_alone;
    launch.desc_warps = descending && warps_alone && q >= kDescWarpsFromQ;
    launch.grid = grid;
    launch.stream = (cudaStream_t)cuda_stream;
    switch (q) {
#define BCAST_CASE(N) case N: launch_table_kernel<N>(launch); break;
        BCAST_CASE(1) BCAST_CASE(2) BCAST_CASE(3) BCAST_CASE(4) BCAST_CASE(5) BCAST_CASE(6) BCAST_CASE(7)
        BCAST_CASE(8) BCAST_CASE(9) BCAST_CASE(10) BCAST_CASE(11) BCAST_CASE(12) BCAST_CASE(13)
        BCAST_CASE(14) BCAST_CASE(15) BCAST_CASE(16) BCAST_CASE(17) BCAST_CASE(18) BCAST_CASE(19)
        BCAST_CASE(20) BCAST_CASE(21) BCAST_CASE(22) BCAST_CASE(23) BCAST_CASE(24) BCAST_CASE(25)
        BCAST_CASE(26) BCAST_CASE(27) BCAST_CASE(28) BCAST_CASE(29) BCAST_CASE(30) BCAST_CASE(31)
#undef BCAST_CASE
    default: return BCAST_EINVAL_P;
    }
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return q;
}

int bcast_schedule(int32_t p, int32_t root, int64_t rank_begin, int64_t rank_end,
                   int32_t *recvblock_dev, int32_t *sendblock_dev, void *cuda_stream)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (root < 0 || root >= p) return BCAST_EINVAL_ROOT;
    if (rank_begin < 0 || rank_begin > rank_end || rank_end > p) return BCAST_EINVAL_RANGE;
    const int q = host_q(p);
    const int64_t n_ranks = rank_end - rank_begin;
    if (q == 0 || n_ranks == 0) return q;              // zero-size tables: nothing to write
    if (recvblock_dev == nullptr && sendblock_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)recvblock_dev & 3u) || ((uintptr_t)sendblock_dev & 3u)) return BCAST_EALIGN;
    return launch_table(p, q, root, rank_begin, n_ranks, 0, recvblock_dev, sendblock_dev, cuda_stream);
}

int bcast_schedule_shifted(int32_t p, int32_t root, int64_t n, int64_t rank_begin, int64_t rank_end,
                           int32_t *recvblock_dev, int32_t *sendblock_dev, void *cuda_stream)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (root < 0 || root >= p) return BCAST_EINVAL_ROOT;
    if (n < 1) return BCAST_EINVAL_N;
    if (rank_begin < 0 || rank_begin > rank_end || rank_end > p) return BCAST_EINVAL_RANGE;
    const int q = host_q(p);
    const int64_t n_ranks = rank_end - rank_begin;
    if (q == 0 || n_ranks == 0) return q;
    if (recvblock_dev == nullptr && sendblock_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)recvblock_dev & 3u) || ((uintptr_t)sendblock_dev & 3u)) return BCAST_EALIGN;
    const int x = (int)((q - (n - 1) % q) % q);
    return launch_table(p, q, root, rank_begin, n_ranks, 0, recvblock_dev, sendblock_dev, cuda_stream, x);
}

int bcast_allbroadcast_schedule(int32_t p, int32_t rank, int64_t root_begin, int64_t root_end,
                                int32_t *recvblocks_dev, int32_t *sendblocks_dev, void *cuda_stream)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (rank < 0 || rank >= p) return BCAST_EINVAL_ROOT;
    if (root_begin < 0 || root_begin > root_end || root_end > p) return BCAST_EINVAL_RANGE;
    const int q = host_q(p);
    const int64_t n_roots = root_end - root_begin;
    if (q == 0 || n_roots == 0) return q;
    if (recvblocks_dev == nullptr && sendblocks_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)recvblocks_dev & 3u) || ((uintptr_t)sendblocks_dev & 3u)) return BCAST_EALIGN;
    return launch_table(p, q, rank, root_begin, n_roots, 1, recvblocks_dev, sendblocks_dev, cuda_stream);
}

int bcast_schedule_host(int32_t p, int32_t root, int64_t rank_begin, int64_t rank_end,
                        int32_t *recvblock_host, int32_t *sendblock_host,
                        void *staging_dev, int64_t staging_bytes, void *cuda_stream)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (root < 0 || root >= p) return BCAST_EINVAL_ROOT;
    if (rank_begin < 0 || rank_begin > rank_end || rank_end > p) return BCAST_EINVAL_RANGE;
    const int q = host_q(p);
    if (q == 0 || rank_end == rank_begin) return q;
    if (recvblock_host == nullptr && sendblock_host == nullptr) return BCAST_ENULL;
    if (staging_dev == nullptr) return BCAST_ENULL;
    if ((uintptr_t)staging_dev & 15u) return BCAST_EALIGN;
    const int n_tables = (recvblock_host != nullptr) + (sendblock_host != nullptr);
    // ranks per chunk: a multiple of 32 so that every table slice stays 16-byte aligned
    const int64_t row_bytes = (int64_t)q * 4;
    int64_t chunk = staging_bytes / (row_bytes * n_tables) / 32 * 32;
    if (chunk < 32) return BCAST_ESCRATCH;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    for (int64_t lo = rank_begin; lo < rank_end; lo += chunk) {
        const int64_t hi = lo + chunk < rank_end ? lo + chunk : rank_end;
        const int64_t rows = hi - lo;
        int32_t *recv_dev = recvblock_host ? reinterpret_cast<int32_t *>(staging_dev) : nullptr;
        int32_t *send_dev = sendblock_host
            ? reinterpret_cast<int32_t *>(staging_dev) + (recvblock_host ? chunk * q : 0) : nullptr;
        const int rc = bcast_schedule(p, root, lo, hi, recv_dev, send_dev, cuda_stream);
        if (rc < 0) return rc;
        const size_t off = (size_t)(lo - rank_begin) * q;
        if (recvblock_host &&
            cudaMemcpyAsync(recvblock_host + off, recv_dev, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
            return BCAST_ECUDA;
        if (sendblock_host &&
            cudaMemcpyAsync(sendblock_host + off, send_dev, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
            return BCAST_ECUDA;
    }
    return q;
}

int bcast_schedule_batch(const int32_t *p_dev, const int32_t *rank_dev, const int32_t *root_dev,
                         int64_t nq, int32_t row_stride,
                         int32_t *recvblock_dev, int32_t *sendblock_dev,
                         int32_t *bad_count_dev, void *cuda_stream)
{
    if (nq < 0) return BCAST_EINVAL_N;
    if (row_stride < BCAST_MAX_Q) return BCAST_ESTRIDE;
    if (p_dev == nullptr || rank_dev == nullptr || root_dev == nullptr) return BCAST_ENULL;
    if (recvblock_dev == nullptr && sendblock_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)p_dev | (uintptr_t)rank_dev | (uintptr_t)root_dev | (uintptr_t)recvblock_dev |
         (uintptr_t)sendblock_dev | (uintptr_t)bad_count_dev) & 3u) return BCAST_EALIGN;
    if (nq == 0) return BCAST_OK;
    const int sms = sm_count();
    if (sms <= 0) return BCAST_ECUDA;
    const int64_t blocks_needed = (nq + kThreads - 1) / kThreads;
    // one tile of kThreads queries per block while that keeps the grid below 2^20 blocks:
    // short-lived blocks balance better than a resident grid striding over the tiles
    const int64_t grid_cap = (int64_t)1 << 20;
    const int grid = (int)(blocks_needed < grid_cap ? blocks_needed : grid_cap);
    schedule_batch_kernel<<<grid, kThreads, 0, (cudaStream_t)cuda_stream>>>(
        p_dev, rank_dev, root_dev, nq, row_stride, recvblock_dev, sendblock_dev, bad_count_dev,
        ((uintptr_t)recvblock_dev & 15u) == 0, ((uintptr_t)sendblock_dev & 15u) == 0);
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return BCAST_OK;
}

int64_t bcast_verify_sweep_scratch_bytes(int32_t p_lo, int32_t p_hi)
{
    if (p_lo < 1 || p_hi < 1) return BCAST_EINVAL_P;
    if (p_lo > p_hi) return BCAST_EINVAL_RANGE;
    const int sms = sm_count();
    if (sms <= 0) return BCAST_ECUDA;
    int64_t blocks = (int64_t)sms * kSweepBlocksPerSm;
    const int64_t count = (int64_t)p_hi - p_lo + 1;
    if (blocks > count) blocks = count;
    return kSweepHeaderBytes + blocks * sweep_bytes_per_block(p_hi);
}

int bcast_verify_sweep(int32_t p_lo, int32_t p_hi, uint64_t *checksum_dev,
                       uint32_t *fail_counts_dev, void *scratch_dev, int64_t scratch_bytes,
                       void *cuda_stream)
{
    if (p_lo < 1 || p_hi < 1) return BCAST_EINVAL_P;
    if (p_lo > p_hi) return BCAST_EINVAL_RANGE;
    if (checksum_dev == nullptr || fail_counts_dev == nullptr || scratch_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)checksum_dev & 7u) || ((uintptr_t)fail_counts_dev & 3u) || ((uintptr_t)scratch_dev & 15u))
        return BCAST_EALIGN;
    const int64_t per_block = sweep_bytes_per_block(p_hi);
    const int64_t usable = scratch_bytes - kSweepHeaderBytes;
    if (usable < per_block) return BCAST_ESCRATCH;
    const int sms = sm_count();
    if (sms <= 0) return BCAST_ECUDA;
    int64_t blocks = (int64_t)sms * kSweepBlocksPerSm;
    const int64_t count = (int64_t)p_hi - p_lo + 1;
    if (blocks > count) blocks = count;
    if (blocks > usable / per_block) blocks = usable / per_block;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned int *queue = reinterpret_cast<unsigned int *>(scratch_dev);
    zero_counter_kernel<<<1, 1, 0, stream>>>(queue);
    verify_sweep_kernel<<<(int)blocks, kThreads, 0, stream>>>(
        (uint32_t)p_lo, (uint32_t)p_hi, checksum_dev, fail_counts_dev,
        reinterpret_cast<int8_t *>(scratch_dev) + kSweepHeaderBytes, (size_t)per_block, queue);
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return BCAST_OK;
}

int bcast_round(int32_t q, int64_t n, int64_t j, int32_t *k_out, int64_t *shift_out)
{
    if (q < 1 || n < 1) return BCAST_EINVAL_N;
    if (j < 0 || j >= n - 1 + q) return BCAST_EINVAL_ROUND;
    const int64_t x = (q - (n - 1) % q) % q;
    const int64_t i = x + j;
    if (k_out) *k_out = (int32_t)(i % q);
    if (shift_out) *shift_out = (i / q) * q - x;
    return BCAST_OK;
}

int64_t bcast_round_block(int32_t q, int64_t n, int64_t j, const int32_t *sched_row_host)
{
    if (sched_row_host == nullptr) return BCAST_ENULL;
    int32_t k = 0;
    int64_t shift = 0;
    const int rc = bcast_round(q, n, j, &k, &shift);
    if (rc != BCAST_OK) return rc;
    const int64_t raw = (int64_t)sched_row_host[k] + shift;
    if (raw < 0) return BCAST_NONE;
    return raw > n - 1 ? n - 1 : raw;
}

// ------------------------------------------------------------------ sweep without caller scratch
// The tables of the sweep live in this array instead of in memory the caller allocated.
// It is part of the loaded module: every device that loads the library carries these
// bytes until the process exits, which is why the size is kept modest.
static __device__ __align__(256) unsigned char g_sweep_static_scratch[BCAST_STATIC_SWEEP_BYTES];

// Device address of the array, looked up once per device.  In host code the array's
// name is only a handle for the runtime, never an address a kernel may be given.
static void *g_sweep_static_ptr[64];
static std::mutex g_sweep_static_mutex;

int bcast_verify_sweep_static(int32_t p_lo, int32_t p_hi, uint64_t *checksum_dev,
                              uint32_t *fail_counts_dev, void *cuda_stream)
{
    if (p_lo < 1 || p_hi < 1) return BCAST_EINVAL_P;
    if (p_lo > p_hi) return BCAST_EINVAL_RANGE;
    if (p_hi > BCAST_STATIC_SWEEP_MAX_P) return BCAST_ETOOBIG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BCAST_ECUDA;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_sweep_static_mutex);
        if (g_sweep_static_ptr[dev] == nullptr) {
            void *addr = nullptr;
            if (cudaGetSymbolAddress(&addr, g_sweep_static_scratch) != cudaSuccess || addr == nullptr)
                return BCAST_ECUDA;
            g_sweep_static_ptr[dev] = addr;
        }
        scratch = g_sweep_static_ptr[dev];
    }
    return bcast_verify_sweep(p_lo, p_hi, checksum_dev, fail_counts_dev, scratch,
                              (int64_t)BCAST_STATIC_SWEEP_BYTES, cuda_stream);
}

}  // extern "C"
