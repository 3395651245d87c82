// The table kernel (bcast_schedule, bcast_schedule_shifted, bcast_allbroadcast_schedule), a
// template on q, and its launch.  Each q is instantiated in one of the table_q_*.cu files.
#pragma once
#include "schedule_tile.cuh"

namespace bcast {

// kDescWarps = false: the kernel of bcast_schedule and its variants, either launch shape, rows by
// ascending rank in the warps-on-their-own shape.  kDescWarps = true: only that shape, rows by
// descending rank (Algorithm 7's tables); a kernel of its own so that the other one is compiled
// exactly as it would be without it.
template <int Q, bool kDescWarps>
__global__ void __launch_bounds__(kThreads, kTableBlocksPerSm)
schedule_table_kernel(const __grid_constant__ LevelTables tab, uint32_t p, uint32_t anchor,
                      uint32_t row_begin, uint32_t n_ranks, int descending, int tiles_per_block,
                      int32_t *__restrict__ recv_out, int32_t *__restrict__ send_out,
                      int recv_vec_ok, int send_vec_ok, int shift_x, int shape,
                      const __grid_constant__ LowFrameTable low_states)
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

    // This block's tiles: tiles_per_block consecutive ones, taken in groups of kWarpsPerBlock.  Each
    // warp first describes the runs of one tile of the group, then the block goes through them.  Many
    // short-lived blocks instead of a persistent grid: the hardware's block scheduler evens out the
    // load, which measured 12 % faster than striding a resident grid over the tiles.
    const uint32_t block_first_tile = blockIdx.x * (uint32_t)tiles_per_block;
    auto describe_group = [&](uint32_t group, int n_slots) {
        const uint32_t t = group + (uint32_t)warp;
        bool share = false;
        if (warp < n_slots && t < n_tiles) {
            const uint32_t first = t * kThreads;
            const uint32_t rows = min((uint32_t)kThreads, n_ranks - first);
            const uint32_t r_first = first_rank_of(first, rows);
            share = tile_can_share<Q>(g, r_first, rows);
            if constexpr (Q >= kSharedFrom + 2)
                if (share) build_tile_runs<Q>(tab, lookup, p, r_first, (int)rows, lane, runs[warp]);
        }
        if (!share && lane == 0) { runs[warp].n_runs = 0; runs[warp].n_pending = 0; }
    };
    if (kDescWarps || shape != kShapeBlockPerTile) {       // host: never with the shifted rows
        constexpr bool desc = kDescWarps;
        DeferredQueue &dq = queues.deferred;
        if (threadIdx.x == 0) { dq.n_items = 0; dq.n_fixups = 0; }
        if (threadIdx.x == 2) dq.overflow = 0u;
        // the low rounds of the search for every low state of this p, filled in by the host when it
        // expects enough undecided entries to pay for the lookups
        const int capacity_cut = shape == kShapeWarpsTight ? kDeferredCapacity - kTightCapacity : 0;
        const uint32_t *low_frame = nullptr;
        if constexpr (Q >= kSharedFrom + 2) {
            if (shape == kShapeWarpsLowFrame) {            // the same for the whole block
                for (int i = threadIdx.x; i < kLowFrameStates; i += kThreads) dq.low_frame[i] = low_states.word[i];
                low_frame = dq.low_frame;
            }
        }
        const size_t block_base = (size_t)block_first_tile * kThreads * (size_t)Q;
        const int item_room = kDeferredCapacity - capacity_cut;
        const int fixup_room = kFixupCapacity - capacity_cut * (kFixupCapacity / kDeferredCapacity);
        bool gather = false;                               // whether later groups may share a drain
        for (int done = 0; done < tiles_per_block; done += kWarpsPerBlock) {
            const uint32_t group = block_first_tile + (uint32_t)done;
            if (group >= n_tiles) break;
            const int n_slots = min(kWarpsPerBlock, tiles_per_block - done);
            const uint32_t group_rows = min((uint32_t)n_slots * kThreads, n_ranks - group * kThreads);
            describe_group(group, n_slots);
            __syncthreads();                               // descriptions (and table) built, queues reset if drained
            for (int slot = 0; slot < n_slots; ++slot) {
                const uint32_t t = group + (uint32_t)slot;
                if (t >= n_tiles) break;
                const uint32_t first = t * kThreads;
                const uint32_t rows = min((uint32_t)kThreads, n_ranks - first);
                const SharedTile<Q> tile{recv_bytes, send_bytes, rows, false};
                warp_pass<Q, desc>(tab, g, runs[slot], first_rank_of(first, rows), rows,
                                   (uint32_t)(done + slot) * kThreads, group_rows, tile, want_recv, want_send, dq,
                                   1u << (done / kWarpsPerBlock), capacity_cut, low_frame);
                __syncwarp();                              // the slice is staged
                const uint32_t my_first = (uint32_t)warp * 32u;
                if (my_first < rows) {
                    const int my_entries = (int)min(32u, rows - my_first) * Q;
                    const size_t base = (size_t)(first + my_first) * (size_t)Q;
                    const uint32_t word = my_first * Q / 4u;   // 32 rows of Q bytes are whole words
                    if (want_recv) flush_tile<32>(stage[0] + word, recv_out + base, my_entries, recv_vec_ok, lane);
                    if (want_send) flush_tile<32>(stage[1] + word, send_out + base, my_entries, send_vec_ok, lane);
                }
                __syncwarp();                              // flushed before the next tile's pass overwrites it
            }
            __syncthreads();                               // every slice of the group is out
            // Work the queues off now?  The same answer in every thread: the counters rest until the next pass.
            // The block's first group tells how dense the undecided entries of this p are.
            const bool last = done + kWarpsPerBlock >= tiles_per_block || group + kWarpsPerBlock >= n_tiles;
            const int queued_items = dq.n_items, queued_fixups = dq.n_fixups;
            if (done == 0) gather = queued_items <= item_room / 4 && queued_fixups <= fixup_room / 4;
            if (!last && gather && queued_items <= item_room / 2 && queued_fixups <= fixup_room / 2) continue;
            const int n_items = min(queued_items, item_room);
            const int n_fixups = min(queued_fixups, fixup_room);
            for (int i = threadIdx.x; i < n_items; i += kThreads) {
                resolve_deferred(g, dq.items[i], [&](int table, uint32_t row, int k, int val) {
                    int32_t *out = table == 0 ? recv_out : send_out;
                    out[block_base + (size_t)row * Q + k] = val;
                });
            }
            if (n_fixups > 0) __syncthreads();             // the receive entries of every group so far are final
            for (int i = threadIdx.x; i < n_fixups; i += kThreads) {
                const uint32_t f = dq.fixups[i];
                const uint32_t row = f & 16383u, k = f >> 14;
                const uint32_t from = desc ? row - tab.skip[k] : row + tab.skip[k];
                send_out[block_base + (size_t)row * Q + k] = __ldcg(recv_out + block_base + (size_t)from * Q + k);
            }
            // (every thread read the counters before its first search; the next pushes come after the barrier
            // that follows the next group's descriptions)
            if (queued_items + queued_fixups > 0) {
                __syncthreads();
                if (threadIdx.x == 0) { dq.n_items = 0; dq.n_fixups = 0; }
            }
        }
        // groups that found a queue full (bit = number of the group within the block): their rows
        // again, by the search alone
        __syncthreads();
        uint32_t redo = dq.overflow;
        while (redo != 0u) {                               // the same for the whole block
            const uint32_t first_tile = block_first_tile + (uint32_t)(__ffs(redo) - 1) * kWarpsPerBlock;
            redo &= redo - 1u;
            const uint32_t first = first_tile * kThreads;
            const uint32_t left = (uint32_t)tiles_per_block * kThreads - (first - block_first_tile * kThreads);
            const uint32_t rows = min(min((uint32_t)kGroupRows, left), n_ranks - first);
            const size_t at = (size_t)first * (size_t)Q;
            rows_by_search(p, anchor, row_begin + first, descending, rows,
                           want_recv ? recv_out + at : nullptr, want_send ? send_out + at : nullptr);
        }
        return;
    }
    describe_group(block_first_tile, tiles_per_block);
    const uint32_t group = block_first_tile;
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


// Arguments of one launch of the table kernel, and the launch for a given q.
struct TableLaunch {
    LevelTables tab;
    uint32_t p, anchor, row_begin, n_rows;
    int descending, tiles_per_block;
    int32_t *recv_dev, *send_dev;
    int recv_vec, send_vec, shift_x;
    int shape;                          // kShape*; descending rows take a warps shape only for q >= kDescWarpsFromQ
    LowFrameTable low_states;           // filled for kShapeWarpsLowFrame only

    int grid;
    cudaStream_t stream;
};

template <int N>
static void launch_table_kernel(const TableLaunch &l)
{
    if constexpr (N >= kDescWarpsFromQ) {
        if (l.descending && l.shape != kShapeBlockPerTile) {
            schedule_table_kernel<N, true><<<l.grid, kThreads, 0, l.stream>>>(
                l.tab, l.p, l.anchor, l.row_begin, l.n_rows, l.descending, l.tiles_per_block, l.recv_dev,
                l.send_dev, l.recv_vec, l.send_vec, l.shift_x, l.shape, l.low_states);
            return;
        }
    }
    schedule_table_kernel<N, false><<<l.grid, kThreads, 0, l.stream>>>(
        l.tab, l.p, l.anchor, l.row_begin, l.n_rows, l.descending, l.tiles_per_block, l.recv_dev, l.send_dev,
        l.recv_vec, l.send_vec, l.shift_x, l.descending ? kShapeBlockPerTile : l.shape, l.low_states);
}

// One translation unit per range of q (they compile side by side); each returns false for
// a q outside its range.
bool launch_table_q_low(const TableLaunch &l, int q);      //  1 .. 14
bool launch_table_q_mid(const TableLaunch &l, int q);      // 15 .. 20
bool launch_table_q_high(const TableLaunch &l, int q);     // 21 .. 25
bool launch_table_q_top(const TableLaunch &l, int q);      // 26 .. 31

}  // namespace bcast
