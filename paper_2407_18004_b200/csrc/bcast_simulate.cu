// Device-side use of schedule tables: Algorithm 1 of arXiv 2407.18004 run by all p
// processors at once, round by round, on tables in device memory (bcast_simulate_broadcast),
// the same rounds reversed as a reduction (Observation 1, item 3: bcast_simulate_reduce), and both
// for all p roots at once (Algorithm 7 and Observation 1, items 2 and 4:
// bcast_simulate_allbroadcast, bcast_simulate_allreduce).
// See include/bcast_sched.h for the contracts.
//
// Layout and launch shape
//   * The int32 tables [p][q] are first turned into round-major byte tables [q][P]
//     (P = p rounded up to 128) in the caller's scratch: a round then reads one byte per
//     processor from each table, consecutive processors from consecutive addresses, and the
//     2q*P bytes stay in L2 over the n-1+q rounds.  Entries outside [-q, q-1] are counted
//     and stored as kInvalid, which moves nothing in any round.
//   * One thread per processor on a grid that strides over the processors, all on the
//     caller's stream.  The single-root simulators run their rounds inside cooperative
//     launches whose blocks meet between two rounds (a bounded wait; see grid_barrier), or
//     as one launch per round; the all-roots ones as one launch per round, in which nothing
//     waits on another block.
//   * Broadcast state is arrival[b][a], the round in which processor a got block b, and a bit
//     per (processor, block), held[w][a], which is what a round reads.  A sender "held the
//     block before the round" iff its bit was set before; where the bit may be changing in
//     this very round the arrival cell decides: a value written during the round is >= round,
//     so concurrent readers decide the same way whether or not they see it.
//   * Reduction state is value[b][a] plus two bit sets (sent once, sent twice); a receiver reads
//     its to-processor's partial result in place (see reduce_round for why the outcome
//     does not depend on the order of the threads).
//   * Counters are summed per warp with redux, per block in shared memory, and added to the
//     64-bit statistics with one atomic per block and counter that is not zero.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "../../include/bcast_sched.h"

namespace bcast_sim {

constexpr int kThreads = 256;
constexpr int8_t kInvalid = -128;
constexpr int64_t kHeaderBytes = 256;

__host__ __device__ inline int64_t padded(int64_t p) { return (p + 127) / 128 * 128; }
inline int64_t set_words(int64_t n) { return (n + 63) / 64; }      // 64-bit words of a bit set over n blocks

static int host_q(int64_t p)
{
    int q = 0;
    while (((int64_t)1 << q) < p) ++q;
    return q;
}

// SMs of the current device (148 if the query fails: only a grid size depends on it).
static int device_sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return 148;
    return sms;
}

// Counters of one block: summed per warp with redux, per block in shared memory, and added
// to the 64-bit statistics with one atomic per block and counter that is not zero (a round
// of 2^20 processors would otherwise queue tens of thousands of atomics on one address).
struct BlockStats {
    unsigned int count[8];
    unsigned int last_round;
};

__device__ __forceinline__ void stats_begin(BlockStats &bs)
{
    if (threadIdx.x < 8) bs.count[threadIdx.x] = 0u;
    if (threadIdx.x == 8) bs.last_round = 0u;
    __syncthreads();
}

__device__ __forceinline__ void add_stat(BlockStats &bs, int index, unsigned int mine)
{
    const unsigned int total = __reduce_add_sync(0xffffffffu, mine);
    if (total != 0u && (threadIdx.x & 31) == 0) atomicAdd(&bs.count[index], total);
}

__device__ __forceinline__ void stats_end(BlockStats &bs, unsigned long long *stats)
{
    __syncthreads();
    if (threadIdx.x < 8 && bs.count[threadIdx.x] != 0u)
        atomicAdd(stats + threadIdx.x, (unsigned long long)bs.count[threadIdx.x]);
    if (threadIdx.x == 8 && bs.last_round != 0u) atomicMax(stats + 7, (unsigned long long)bs.last_round);
}

// int32 [p][q] -> int8 [q][P], both tables (blockIdx.y), a tile of kThreads processors per block.
__global__ void __launch_bounds__(kThreads)
transpose_tables_kernel(const int32_t *__restrict__ recv_tab, const int32_t *__restrict__ send_tab,
                        int8_t *__restrict__ recv_t, int8_t *__restrict__ send_t,
                        uint32_t p, int q, size_t P, unsigned long long *stats)
{
    __shared__ int8_t tile[kThreads * 33];                 // rows of q <= 31 bytes, 33 apart
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    const int32_t *in = blockIdx.y == 0 ? recv_tab : send_tab;
    int8_t *out = blockIdx.y == 0 ? recv_t : send_t;
    const uint32_t first = blockIdx.x * kThreads;
    const uint32_t rows = min((uint32_t)kThreads, p - first);
    const int n_entries = (int)rows * q;
    const int32_t *src = in + (size_t)first * q;
    unsigned int bad = 0;
    // entry i of the tile is column i mod q of row i / q: kept up to date from one step to the next
    // (a division per entry would cost more than the load)
    int row = threadIdx.x / q, col = threadIdx.x - row * q;
    const int row_step = kThreads / q, col_step = kThreads - row_step * q;
    for (int i = threadIdx.x; i < n_entries; i += kThreads) {
        const int v = __ldcs(src + i);
        const bool ok = v >= -q && v <= q - 1;
        bad += ok ? 0u : 1u;
        tile[row * 33 + col] = ok ? (int8_t)v : kInvalid;
        row += row_step;
        col += col_step;
        if (col >= q) { col -= q; ++row; }
    }
    __syncthreads();
    if (threadIdx.x < rows)
        for (int k = 0; k < q; ++k) out[(size_t)k * P + first + threadIdx.x] = tile[threadIdx.x * 33 + k];
    add_stat(bstats, 5, bad);
    stats_end(bstats, stats);
}

// The root's column of the arrival table (the rest is set to -1 by a memset): it holds every block from the start.
__global__ void __launch_bounds__(kThreads)
root_arrival_kernel(int32_t *__restrict__ arrival, uint32_t p, uint32_t root, int64_t n)
{
    const int64_t b = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (b < n) arrival[(size_t)b * p + root] = 0;
}

// Bit sets over the blocks, a word of 64 blocks per processor: set[w * P + a].  Cleared for everybody
// and, where `root_full`, filled with the n blocks for the root.
__global__ void __launch_bounds__(kThreads)
init_block_sets_kernel(unsigned long long *__restrict__ set, size_t P, uint32_t p, uint32_t root, int64_t n,
                       int root_full)
{
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    const int64_t w = blockIdx.y;
    if (a >= P) return;
    unsigned long long word = 0ull;
    if (root_full && a == root && a < p) {
        const int64_t left = n - 64 * w;
        word = left >= 64 ? ~0ull : ((1ull << left) - 1ull);
    }
    set[(size_t)w * P + a] = word;
}

// Block of a table entry in a round: entry + shift, nothing (-1) when negative or invalid,
// n-1 when above it.
__device__ __forceinline__ int64_t block_of(int8_t entry, int64_t shift, int64_t n)
{
    if (entry == kInvalid) return -1;
    const int64_t raw = (int64_t)entry + shift;
    if (raw < 0) return -1;
    return raw > n - 1 ? n - 1 : raw;
}

// The same in 32 bits for the kernels that run once per round over all processors (n < 2^31 - 64 and
// shift <= n - 1, so entry + shift does not overflow); last = n - 1.
__device__ __forceinline__ int block32(int8_t entry, int shift, int last)
{
    const int raw = min((int)entry + shift, last);
    return entry == kInvalid || raw < 0 ? -1 : raw;
}

// One communication round of Algorithm 1 for every processor: skip index k (the rows of the
// byte tables passed in), blocks = entry + shift, `round` counted from 1.
//
// Who holds what is kept twice: arrival[b][a], the result, written once per delivery, and
// held[w][a], a bit per block, which is what the round reads (8 bytes per processor, consecutive
// processors side by side, where the arrival cells of a round lie in up to 2q different rows).
// Thread a alone writes a's word.  A reader of f's word asks whether f held the block BEFORE the
// round; the bit can only be about to change in this round if f is itself receiving that very
// block now, and then the answer is taken from f's arrival cell, which is -1 or >= round for
// anything not held before, whether or not f's write is seen.
struct RoundCounts {
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0, c6 = 0;
};

__device__ __forceinline__ void add_round_counts(BlockStats &bs, const RoundCounts &c)
{
    add_stat(bs, 0, c.c0);
    add_stat(bs, 1, c.c1);
    add_stat(bs, 2, c.c2);
    add_stat(bs, 3, c.c3);
    add_stat(bs, 6, c.c6);
}

// What the rounds of the broadcast need besides the round's own rows of the byte tables.
struct BroadcastFrame {
    int32_t *arrival;                      // arrival[b * p + a]: the round in which processor a got block b
    unsigned long long *held;              // held[w * P + a]: a bit per block of word w that processor a holds
    size_t P;
    uint32_t p, root;
    int last;                              // n - 1
};

// One communication round of Algorithm 1 for every processor: skip index k (the rows of the
// byte tables passed in), blocks = entry + shift, `round` counted from 1.
//
// Who holds what is kept twice: arrival[b][a], the result, written once per delivery, and
// held[w][a], a bit per block, which is what the round reads (8 bytes per processor, consecutive
// processors side by side, where the arrival cells of a round lie in up to 2q different rows).
// Thread a alone writes a's word.  A reader of f's word asks whether f held the block BEFORE the
// round; the bit can only be about to change in this round if f is itself expecting that very
// block now, and then the answer is taken from f's arrival cell, which is -1 or >= round for
// anything not held before, whether or not f's write is seen.  What another processor wrote is
// read past L1 (ld.global.cg): in the kernel that runs several rounds in one launch a line that
// L1 kept from an earlier round would be stale.
__device__ __forceinline__ void broadcast_round(const BroadcastFrame &fr, const int8_t *__restrict__ recv_k,
                                                const int8_t *__restrict__ send_k, uint32_t skip_k, int shift,
                                                int32_t round, RoundCounts &c)
{
    // a resident grid strides over the processors: a few thousand blocks would each add their
    // counters to the same statistics words, and those atomics would set the pace of the round
    const uint32_t p = fr.p, root = fr.root;
    for (uint32_t a = blockIdx.x * blockDim.x + threadIdx.x; a < p; a += gridDim.x * blockDim.x) {
        if (a == root) continue;
        const uint32_t f = a >= skip_k ? a - skip_k : a + (p - skip_k);     // from-processor
        const int want = block32(recv_k[a], shift, fr.last);
        // f's to-processor is a, which is not the root, so f's send is not suppressed
        const int sent = block32(send_k[f], shift, fr.last);
        // what f itself expects in this round: read here, beside the other two table bytes, not
        // where it is needed at the end of the chain of loads below
        const int f_wants = f == root ? -1 : block32(recv_k[f], shift, fr.last);
        if (want < 0) {
            c.c3 += sent >= 0 ? 1u : 0u;
        } else if (sent != want) {
            c.c0 += 1;
        } else {
            unsigned long long *words = fr.held + (size_t)(want >> 6) * fr.P;
            const unsigned long long bit = 1ull << (want & 63);
            const unsigned long long theirs = __ldcg(words + f), mine = __ldcg(words + a);
            bool f_held = (theirs & bit) != 0ull;
            if (f_held && f_wants == want) {
                const int32_t at_f = __ldcg(fr.arrival + (size_t)want * p + f);    // f may be getting it only now
                f_held = at_f >= 0 && at_f < round;
            }
            if (!f_held) c.c1 += 1;                                          // not held before the round
            else if ((mine & bit) != 0ull) c.c2 += 1;
            else {
                words[a] = mine | bit;
                fr.arrival[(size_t)want * p + a] = round;
                c.c6 += 1;
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 8)
broadcast_round_kernel(const __grid_constant__ BroadcastFrame fr, const int8_t *__restrict__ recv_k,
                       const int8_t *__restrict__ send_k, uint32_t skip_k, int shift, int32_t round,
                       unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    RoundCounts c;
    broadcast_round(fr, recv_k, send_k, skip_k, shift, round, c);
    add_round_counts(bstats, c);
    if (__any_sync(0xffffffffu, c.c6 != 0u) && (threadIdx.x & 31) == 0) bstats.last_round = (unsigned int)round;
    stats_end(bstats, stats);
}

// ------------------------------------------------------------------ several rounds in one launch
// The blocks of a cooperative launch (all resident at once, or the launch is refused) meet between
// two rounds at a counter in the caller's scratch: every block adds one after its threads' writes
// are fenced, and waits until all blocks of the round have.  The wait is bounded: a block that
// sees nothing for a second or two raises `failed`, every block leaves its loop, and the
// statistics are overwritten with all-ones by seal_stats_kernel.
struct GridBarrier {
    unsigned long long arrived;            // blocks that have reached a barrier, over all barriers of the call
    unsigned int failed;
};
static_assert(sizeof(GridBarrier) <= kHeaderBytes, "the barrier lives in the scratch header");

constexpr unsigned int kBarrierSpins = 1u << 21;      // a poll and its pause take about a microsecond
#ifndef BCAST_FUSED_THREADS
#define BCAST_FUSED_THREADS 1024
#endif
#ifndef BCAST_FUSED_BLOCKS
#define BCAST_FUSED_BLOCKS 2
#endif
constexpr int kFusedThreads = BCAST_FUSED_THREADS;     // large blocks: few arrivals per barrier
constexpr int kFusedBlocks = BCAST_FUSED_BLOCKS;       // resident per SM

// `index` = this barrier's number in the call, from 1.  The arrival is a release (the block's
// writes, ordered before it by the block barrier, are visible to whoever sees the count) and, for
// the last block in, an acquire; the others' wait is an acquire.
__device__ __forceinline__ bool grid_barrier(GridBarrier *gb, unsigned long long index, unsigned int blocks)
{
    __shared__ int through;
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long target = index * blocks;
        unsigned long long seen;
        asm volatile("atom.add.acq_rel.gpu.global.u64 %0, [%1], 1;" : "=l"(seen) : "l"(&gb->arrived) : "memory");
        bool good = seen + 1ull >= target;
        for (unsigned int spin = 0; !good && spin < kBarrierSpins; ++spin) {
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(&gb->arrived) : "memory");
            if (seen >= target) good = true;
            else if (*(volatile unsigned int *)&gb->failed != 0u) break;
            else if (spin >= 64u) __nanosleep(200u);
        }
        if (!good) *(volatile unsigned int *)&gb->failed = 1u;
        through = good ? 1 : 0;
    }
    __syncthreads();
    return through != 0;
}

__global__ void seal_stats_kernel(const GridBarrier *gb, unsigned long long *stats)
{
    if (gb->failed != 0u && threadIdx.x < 8) stats[threadIdx.x] = ~0ull;
}

struct RoundPlan {
    uint32_t skip[32];
    int q;
    int x;
    unsigned int blocks;                   // blocks a barrier waits for: the grid's (one more in the test of the wait's limit)
};

// Counters of a block over many rounds (64 bits: 2^31 rounds of a few thousand processors).
struct BlockStats64 {
    unsigned long long count[8];
    unsigned int last_round;
};

__device__ __forceinline__ void add_stat64(BlockStats64 &bs, int index, unsigned int mine)
{
    const unsigned int total = __reduce_add_sync(0xffffffffu, mine);
    if (total != 0u && (threadIdx.x & 31) == 0) atomicAdd(&bs.count[index], (unsigned long long)total);
}

__device__ __forceinline__ void stats64_begin(BlockStats64 &bs)
{
    if (threadIdx.x < 8) bs.count[threadIdx.x] = 0ull;
    if (threadIdx.x == 8) bs.last_round = 0u;
    __syncthreads();
}

__device__ __forceinline__ void stats64_end(BlockStats64 &bs, unsigned long long *stats)
{
    __syncthreads();
    if (threadIdx.x < 8 && bs.count[threadIdx.x] != 0ull) atomicAdd(stats + threadIdx.x, bs.count[threadIdx.x]);
    if (threadIdx.x == 8 && bs.last_round != 0u) atomicMax(stats + 7, (unsigned long long)bs.last_round);
}

// Rounds j0 .. j1-1 of the broadcast (j counted from 0), one block barrier between two rounds;
// `barriers_before` = the barriers of the launches before this one in the same call.
__global__ void __launch_bounds__(kFusedThreads, kFusedBlocks)
broadcast_rounds_kernel(const __grid_constant__ BroadcastFrame fr, const int8_t *__restrict__ recv_t,
                        const int8_t *__restrict__ send_t, const __grid_constant__ RoundPlan plan, long long j0, long long j1,
                        GridBarrier *gb, unsigned long long barriers_before, unsigned long long *stats)
{
    __shared__ BlockStats64 bstats;
    stats64_begin(bstats);
    const long long i0 = plan.x + j0;
    int k = (int)(i0 % plan.q);
    int shift = (int)((i0 / plan.q) * plan.q - plan.x);               // Theorem 1
    unsigned int last_delivery = 0;
    unsigned long long barriers = barriers_before;
    bool failed = false;
    // a thread's counts of one launch fit 32 bits: at most 65536 rounds of 2^31 / (threads of the grid) processors
    RoundCounts c;
    for (long long j = j0; j < j1; ++j) {
        const unsigned int delivered_before = c.c6;
        broadcast_round(fr, recv_t + (size_t)k * fr.P, send_t + (size_t)k * fr.P, plan.skip[k], shift, (int32_t)(j + 1), c);
        if (c.c6 != delivered_before) last_delivery = (unsigned int)(j + 1);
        if (++k == plan.q) { k = 0; shift += plan.q; }
        if (j + 1 < j1 && !grid_barrier(gb, ++barriers, plan.blocks)) { failed = true; break; }
    }
    if (failed) return;
    add_stat64(bstats, 0, c.c0);
    add_stat64(bstats, 1, c.c1);
    add_stat64(bstats, 2, c.c2);
    add_stat64(bstats, 3, c.c3);
    add_stat64(bstats, 6, c.c6);
    last_delivery = __reduce_max_sync(0xffffffffu, last_delivery);
    if ((threadIdx.x & 31) == 0 && last_delivery != 0u) atomicMax(&bstats.last_round, last_delivery);
    stats64_end(bstats, stats);
}

__global__ void __launch_bounds__(kThreads)
count_missing_kernel(const int32_t *__restrict__ arrival, size_t cells, unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    unsigned int missing = 0;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < cells; i += (size_t)gridDim.x * kThreads)
        missing += arrival[i] < 0 ? 1u : 0u;
    add_stat(bstats, 4, missing);
    stats_end(bstats, stats);
}

// (processor, block) pairs still missing, from the bit sets (a bit is set exactly when the arrival
// cell is): word w of a processor covers min(64, n - 64 w) blocks.
__global__ void __launch_bounds__(kThreads)
count_missing_sets_kernel(const unsigned long long *__restrict__ held, size_t P, uint32_t p, int64_t n,
                          unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    const int64_t w = blockIdx.y;
    const int in_word = (int)(n - 64 * w >= 64 ? 64 : n - 64 * w);
    unsigned int missing = 0;
    for (uint32_t a = blockIdx.x * kThreads + threadIdx.x; a < p; a += gridDim.x * kThreads)
        missing += (unsigned int)(in_word - __popcll(held[(size_t)w * P + a]));
    add_stat(bstats, 4, missing);
    stats_end(bstats, stats);
}

// ------------------------------------------------------------------ reduction (reversed rounds)
// One reduction round for every processor.  Processor a sends its partial result of the block
// it RECEIVED in the corresponding broadcast round to its from-processor (the root sends
// nothing), and takes, from its to-processor t, a partial result of the block it SENT to t in
// that broadcast round, which it adds to its own; then it notes its own send as done.
//
// The receiver reads the sender's value in place, in the same launch, and the outcome does
// not depend on the order of the threads: value[b][t] is read by t's from-processor only when
// t sends b in this round, and t adds to value[b][t] only when it receives b and is NOT
// sending b (a processor that receives the block it is sending would never pass the sum on,
// which is counted instead); sent[.][a] is read and written by thread a alone.
__device__ __forceinline__ void reduce_round(const int8_t *__restrict__ recv_k, const int8_t *__restrict__ send_k,
                                             uint64_t *value, unsigned long long *once, unsigned long long *twice,
                                             size_t P, uint32_t p, uint32_t root, int last, uint32_t skip_k,
                                             int shift, RoundCounts &c)
{
    for (uint32_t a = blockIdx.x * blockDim.x + threadIdx.x; a < p; a += gridDim.x * blockDim.x) {
        uint32_t t = a + skip_k;                           // < 2^32: p, skip_k < 2^31
        if (t >= p) t -= p;
        const int mine = a == root ? -1 : block32(recv_k[a], shift, last);         // what a sends
        const int got = t == root ? -1 : block32(recv_k[t], shift, last);          // what t sends to a
        const int want = t == root ? -1 : block32(send_k[a], shift, last);
        // every load the round may need is issued here, before any of them is looked at: the two
        // partial results, and a's words of the sets for the block it sends and the block it expects
        const bool match = want >= 0 && got == want;
        uint64_t theirs = 0, own = 0;
        unsigned long long once_mine = 0ull, once_want = 0ull;
        if (match) {
            theirs = __ldcg(value + (size_t)want * p + t);                          // t's: read past L1
            own = value[(size_t)want * p + a];
            once_want = once[(size_t)(want >> 6) * P + a];
        }
        if (mine >= 0) once_mine = once[(size_t)(mine >> 6) * P + a];
        // how often a has sent a block: bit in once[] after the first time, in twice[] after the second;
        // thread a alone reads and writes a's words
        const bool sent_mine = mine >= 0 && ((once_mine >> (mine & 63)) & 1ull) != 0ull;
        if (sent_mine) c.c2 += 1;
        if (want < 0) {
            if (got >= 0) c.c3 += 1;
        } else if (got != want) {
            c.c0 += 1;
        } else if (a != root && (mine == want || ((once_want >> (want & 63)) & 1ull) != 0ull)) {
            c.c1 += 1;                                     // it would never be passed on
        } else {
            value[(size_t)want * p + a] = own + theirs;
            c.c6 += 1;
        }
        if (mine >= 0) {
            if (sent_mine) twice[(size_t)(mine >> 6) * P + a] |= 1ull << (mine & 63);
            else once[(size_t)(mine >> 6) * P + a] = once_mine | (1ull << (mine & 63));
        }
    }
}

__global__ void __launch_bounds__(kThreads)
reduce_round_kernel(const int8_t *__restrict__ recv_k, const int8_t *__restrict__ send_k,
                    uint64_t *value, unsigned long long *once, unsigned long long *twice, size_t P,
                    uint32_t p, uint32_t root, int last, uint32_t skip_k, int shift,
                    unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    RoundCounts c;
    reduce_round(recv_k, send_k, value, once, twice, P, p, root, last, skip_k, shift, c);
    add_round_counts(bstats, c);
    stats_end(bstats, stats);
}

// Rounds j1-1 down to j0 of the reduction in one cooperative launch (see broadcast_rounds_kernel).
__global__ void __launch_bounds__(kFusedThreads, kFusedBlocks)
reduce_rounds_kernel(const int8_t *__restrict__ recv_t, const int8_t *__restrict__ send_t,
                     uint64_t *value, unsigned long long *once, unsigned long long *twice, size_t P,
                     uint32_t p, uint32_t root, int last, const __grid_constant__ RoundPlan plan,
                     long long j0, long long j1, GridBarrier *gb, unsigned long long barriers_before,
                     unsigned long long *stats)
{
    __shared__ BlockStats64 bstats;
    stats64_begin(bstats);
    const long long i1 = plan.x + j1 - 1;
    int k = (int)(i1 % plan.q);
    int shift = (int)((i1 / plan.q) * plan.q - plan.x);
    unsigned long long barriers = barriers_before;
    bool failed = false;
    RoundCounts c;                                         // 32 bits are enough: see broadcast_rounds_kernel
    for (long long j = j1 - 1; j >= j0; --j) {
        reduce_round(recv_t + (size_t)k * P, send_t + (size_t)k * P, value, once, twice, P, p, root, last,
                     plan.skip[k], shift, c);
        if (--k < 0) { k = plan.q - 1; shift -= plan.q; }
        if (j > j0 && !grid_barrier(gb, ++barriers, plan.blocks)) { failed = true; break; }
    }
    if (failed) return;
    add_stat64(bstats, 0, c.c0);
    add_stat64(bstats, 1, c.c1);
    add_stat64(bstats, 2, c.c2);
    add_stat64(bstats, 3, c.c3);
    add_stat64(bstats, 6, c.c6);
    stats64_end(bstats, stats);
}

__global__ void __launch_bounds__(kThreads)
reduce_finish_kernel(const uint64_t *__restrict__ value, const unsigned long long *__restrict__ once,
                     const unsigned long long *__restrict__ twice, size_t P, uint64_t *__restrict__ result,
                     uint32_t p, uint32_t root, int64_t b0, unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    const int64_t b = b0 + blockIdx.y;
    unsigned int c4 = 0;
    if (a < p) {
        if (a == root) {
            result[b] = value[(size_t)b * p + a];
        } else {
            const bool sent_once = (once[(size_t)(b >> 6) * P + a] >> (b & 63)) & 1ull;
            const bool sent_twice = (twice[(size_t)(b >> 6) * P + a] >> (b & 63)) & 1ull;
            if (!sent_once || sent_twice) c4 = 1;           // not exactly once
        }
    }
    add_stat(bstats, 4, c4);
    stats_end(bstats, stats);
}

__global__ void copy_row_kernel(const uint64_t *__restrict__ value, uint64_t *__restrict__ result, int64_t n)
{
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b < n) result[b] = value[b];
}

// ------------------------------------------------------------------ all roots at once (Algorithm 7 and its reversal)
// The p broadcasts of Algorithm 7 share the rounds, and processor a's rows for root j are the
// rows of virtual rank v = (a - j) mod p of the broadcast tables of root 0.  Thread (a, j) does
// for root j what the kernels above do for their one root, with the byte tables read at v:
// "packed for every root but the to-processor" is "nothing is sent to the root", "unpacked for
// every root but oneself" is "the root receives nothing".  State: one slab of n*p cells per root.
__global__ void __launch_bounds__(kThreads)
init_arrival_all_kernel(int32_t *__restrict__ arrival, uint32_t p, uint32_t root0, int64_t n)
{
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    const uint32_t j = root0 + blockIdx.y;
    if (a >= p) return;
    int32_t *slab = arrival + (size_t)j * (size_t)n * p;
    for (int64_t b = 0; b < n; ++b) slab[(size_t)b * p + a] = a == j ? 0 : -1;
}

// Every (processor, root) pair reads one row of the given tables, and each row serves p pairs: the count
// of entries out of range, taken once over the tables, is that of all pairs after this.
__global__ void scale_bad_entries_kernel(unsigned long long *stats, unsigned long long p) { stats[5] *= p; }

__global__ void __launch_bounds__(kThreads)
allbroadcast_round_kernel(const int8_t *__restrict__ recv_k, const int8_t *__restrict__ send_k,
                          int32_t *arrival, uint32_t p, uint32_t root0, int64_t n, uint32_t skip_k,
                          int64_t shift, int32_t round, unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    const uint32_t j = root0 + blockIdx.y;
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0, c6 = 0;
    if (a < p && a != j) {
        const uint32_t v = a >= j ? a - j : a + (p - j);                       // a's virtual rank for root j, > 0
        const uint32_t vf = v >= skip_k ? v - skip_k : v + (p - skip_k);       // and its from-processor's
        const uint32_t f = a >= skip_k ? a - skip_k : a + (p - skip_k);
        int32_t *slab = arrival + (size_t)j * (size_t)n * p;
        const int64_t want = block_of(recv_k[v], shift, n);
        const int64_t sent = block_of(send_k[vf], shift, n);                   // f's to-processor is a, not the root
        if (want < 0) {
            if (sent >= 0) c3 = 1;
        } else if (sent != want) {
            c0 = 1;
        } else {
            const int32_t at_f = slab[(size_t)want * p + f];
            const int32_t at_a = slab[(size_t)want * p + a];
            if (!(at_f >= 0 && at_f < round)) c1 = 1;
            else if (at_a >= 0) c2 = 1;
            else { slab[(size_t)want * p + a] = round; c6 = 1; }
        }
    }
    add_stat(bstats, 0, c0);
    add_stat(bstats, 1, c1);
    add_stat(bstats, 2, c2);
    add_stat(bstats, 3, c3);
    add_stat(bstats, 6, c6);
    if (__any_sync(0xffffffffu, c6 != 0u) && (threadIdx.x & 31) == 0) bstats.last_round = (unsigned int)round;
    stats_end(bstats, stats);
}

// One all-reduction round: thread (a, j) as reduce_round_kernel's thread a with root j.
__global__ void __launch_bounds__(kThreads)
allreduce_round_kernel(const int8_t *__restrict__ recv_k, const int8_t *__restrict__ send_k,
                       uint64_t *value, uint8_t *sent, uint32_t p, uint32_t root0, int64_t n,
                       uint32_t skip_k, int64_t shift, unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    const uint32_t j = root0 + blockIdx.y;
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0, c6 = 0;
    if (a < p) {
        uint32_t t = a + skip_k;
        if (t >= p) t -= p;
        const uint32_t v = a >= j ? a - j : a + (p - j);
        uint32_t vt = v + skip_k;
        if (vt >= p) vt -= p;
        uint64_t *val = value + (size_t)j * (size_t)n * p;
        uint8_t *snt = sent + (size_t)j * (size_t)n * p;
        const int64_t mine = a == j ? -1 : block_of(recv_k[v], shift, n);          // what a sends
        const int64_t got = t == j ? -1 : block_of(recv_k[vt], shift, n);          // what t sends to a
        const int64_t want = t == j ? -1 : block_of(send_k[v], shift, n);
        uint8_t sent_mine = 0;
        if (mine >= 0) {
            sent_mine = snt[(size_t)mine * p + a];
            if (sent_mine > 0) c2 = 1;
        }
        if (want < 0) {
            if (got >= 0) c3 = 1;
        } else if (got != want) {
            c0 = 1;
        } else if (a != j && (mine == want || snt[(size_t)want * p + a] > 0)) {
            c1 = 1;
        } else {
            val[(size_t)want * p + a] += val[(size_t)want * p + t];
            c6 = 1;
        }
        if (mine >= 0 && sent_mine < 2) snt[(size_t)mine * p + a] = sent_mine + 1;
    }
    add_stat(bstats, 0, c0);
    add_stat(bstats, 1, c1);
    add_stat(bstats, 2, c2);
    add_stat(bstats, 3, c3);
    add_stat(bstats, 6, c6);
    stats_end(bstats, stats);
}

__global__ void __launch_bounds__(kThreads)
allreduce_finish_kernel(const uint64_t *__restrict__ value, const uint8_t *__restrict__ sent,
                        uint64_t *__restrict__ result, uint32_t p, uint32_t root0, int64_t n,
                        unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    const uint32_t j = root0 + blockIdx.y;
    unsigned int c4 = 0;
    if (a < p) {
        const size_t slab = (size_t)j * (size_t)n * p;
        for (int64_t b = 0; b < n; ++b) {
            if (a == j) result[(size_t)j * n + b] = value[slab + (size_t)b * p + a];
            else if (sent[slab + (size_t)b * p + a] != 1) c4 += 1;
        }
    }
    add_stat(bstats, 4, c4);
    stats_end(bstats, stats);
}

struct Plan {
    int q;
    int64_t P;
    int64_t x;
    uint32_t skip[33];
};

static Plan make_plan(int32_t p, int64_t n)
{
    Plan plan = {};
    plan.q = host_q(p);
    plan.P = padded(p);
    plan.x = plan.q > 0 ? (plan.q - (n - 1) % plan.q) % plan.q : 0;
    int64_t s = p;
    plan.skip[plan.q] = (uint32_t)p;
    for (int k = plan.q; k > 0; --k) {
        s = s - s / 2;
        plan.skip[k - 1] = (uint32_t)s;
    }
    return plan;
}

static int check_common(int32_t p, int32_t root, int64_t n, const void *recv, const void *send,
                        const void *state, const void *stats)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (root < 0 || root >= p) return BCAST_EINVAL_ROOT;
    if (n < 1 || n > (int64_t)0x7fffffff - 64) return BCAST_EINVAL_N;
    if (state == nullptr || stats == nullptr) return BCAST_ENULL;
    if (p > 1 && (recv == nullptr || send == nullptr)) return BCAST_ENULL;
    if (((uintptr_t)recv & 3u) || ((uintptr_t)send & 3u) || ((uintptr_t)stats & 7u)) return BCAST_EALIGN;
    return BCAST_OK;
}

// How the rounds of the single-root simulators are launched: one launch per round, or all rounds in
// cooperative launches whose blocks meet between two rounds.  BCAST_SIMULATE_ROUNDS=launches|fused in
// the environment, read once, or bcast_set_simulate_rounds; otherwise fused where the device allows it.
static std::atomic<int> g_rounds_mode{-1};

static int rounds_mode()
{
    int mode = g_rounds_mode.load(std::memory_order_relaxed);
    if (mode >= 0) return mode;
    mode = BCAST_ROUNDS_AUTO;
    if (const char *env = getenv("BCAST_SIMULATE_ROUNDS")) {
        if (strcmp(env, "launches") == 0) mode = BCAST_ROUNDS_LAUNCHES;
        else if (strcmp(env, "fused") == 0) mode = BCAST_ROUNDS_FUSED;
    }
    int expected = -1;
    g_rounds_mode.compare_exchange_strong(expected, mode, std::memory_order_relaxed);
    return g_rounds_mode.load(std::memory_order_relaxed);
}

// Blocks of a cooperative launch of `kernel` that run all at once on the current device; 0 if the
// device has no cooperative launches.
static unsigned int cooperative_blocks(const void *kernel)
{
    int dev = 0, can = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&can, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !can)
        return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kFusedThreads, 0) != cudaSuccess || per_sm <= 0)
        return 0;
    return (unsigned int)per_sm * (unsigned int)device_sm_count();
}

static RoundPlan round_plan(const Plan &plan)
{
    RoundPlan rp = {};
    for (int k = 0; k < plan.q && k < 32; ++k) rp.skip[k] = plan.skip[k];
    rp.q = plan.q;
    rp.x = (int)plan.x;
    return rp;
}

// Rounds of one cooperative launch: bounds the time a single kernel runs for huge n.
constexpr int64_t kRoundsPerLaunch = 1 << 16;

}  // namespace bcast_sim

using namespace bcast_sim;

extern "C" {

int bcast_set_simulate_rounds(int mode)
{
    if (mode != BCAST_ROUNDS_AUTO && mode != BCAST_ROUNDS_LAUNCHES && mode != BCAST_ROUNDS_FUSED &&
        mode != BCAST_ROUNDS_FUSED_MISS)
        return BCAST_EINVAL_SHAPE;
    g_rounds_mode.store(mode, std::memory_order_relaxed);
    return BCAST_OK;
}

int64_t bcast_simulate_scratch_bytes(int32_t p, int64_t n, int reduction)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (n < 1) return BCAST_EINVAL_N;
    const int q = host_q(p);
    const int64_t P = padded(p);
    // byte tables, then bit sets over the blocks (8 bytes per processor and 64 blocks): who holds what
    // (broadcast), or what was sent once and what twice (reduction)
    return kHeaderBytes + 2 * (int64_t)q * P + (reduction ? 2 : 1) * set_words(n) * P * 8;
}

int bcast_simulate_broadcast(int32_t p, int32_t root, int64_t n,
                             const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                             int32_t *arrival_dev, uint64_t *stats_dev,
                             void *scratch_dev, int64_t scratch_bytes, void *cuda_stream)
{
    const int rc = check_common(p, root, n, recvblock_dev, sendblock_dev, arrival_dev, stats_dev);
    if (rc != BCAST_OK) return rc;
    if ((uintptr_t)arrival_dev & 3u) return BCAST_EALIGN;
    const Plan plan = make_plan(p, n);
    const int q = plan.q;
    if (q > 0) {
        if (scratch_dev == nullptr) return BCAST_ENULL;
        if ((uintptr_t)scratch_dev & 15u) return BCAST_EALIGN;
        if (scratch_bytes < bcast_simulate_scratch_bytes(p, n, 0)) return BCAST_ESCRATCH;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long *stats = reinterpret_cast<unsigned long long *>(stats_dev);
    if (cudaMemsetAsync(stats_dev, 0, 8 * sizeof(uint64_t), stream) != cudaSuccess) return BCAST_ECUDA;
    const unsigned int blocks = (unsigned int)(((int64_t)p + kThreads - 1) / kThreads);
    const GridBarrier *seal_stats_after = nullptr;
    // -1 everywhere (all bytes 0xff), then 0 down the root's column
    if (cudaMemsetAsync(arrival_dev, 0xff, (size_t)n * (size_t)p * sizeof(int32_t), stream) != cudaSuccess)
        return BCAST_ECUDA;
    root_arrival_kernel<<<(unsigned int)((n + kThreads - 1) / kThreads), kThreads, 0, stream>>>(
        arrival_dev, (uint32_t)p, (uint32_t)root, n);
    if (q == 0) return cudaGetLastError() == cudaSuccess ? 0 : BCAST_ECUDA;
    int8_t *recv_t = reinterpret_cast<int8_t *>(scratch_dev) + kHeaderBytes;
    int8_t *send_t = recv_t + (size_t)q * plan.P;
    unsigned long long *held = reinterpret_cast<unsigned long long *>(send_t + (size_t)q * plan.P);
    const int64_t rounds = n - 1 + q;
    BroadcastFrame fr = {};
    fr.arrival = arrival_dev;
    fr.held = held;
    fr.P = (size_t)plan.P;
    fr.p = (uint32_t)p;
    fr.root = (uint32_t)root;
    fr.last = (int)(n - 1);
    const unsigned int pblocks = (unsigned int)(plan.P / kThreads + (plan.P % kThreads != 0));
    for (int64_t w0 = 0; w0 < set_words(n); w0 += 65535) {
        const unsigned int nw = (unsigned int)(set_words(n) - w0 < 65535 ? set_words(n) - w0 : 65535);
        init_block_sets_kernel<<<dim3(pblocks, nw), kThreads, 0, stream>>>(
            held + (size_t)w0 * plan.P, (size_t)plan.P, (uint32_t)p, (uint32_t)root, n - 64 * w0, 1);
    }
    transpose_tables_kernel<<<dim3(blocks, 2), kThreads, 0, stream>>>(
        recvblock_dev, sendblock_dev, recv_t, send_t, (uint32_t)p, q, (size_t)plan.P, stats);
    const unsigned int resident = (unsigned int)device_sm_count() * 8u;
    const int mode = rounds_mode();
    const unsigned int together =
        mode == BCAST_ROUNDS_LAUNCHES ? 0u : cooperative_blocks((const void *)broadcast_rounds_kernel);
    if ((mode == BCAST_ROUNDS_FUSED || mode == BCAST_ROUNDS_FUSED_MISS) && together == 0u) return BCAST_ECUDA;
    bool fused = together != 0u;
    if (fused) {
        GridBarrier *gb = reinterpret_cast<GridBarrier *>(scratch_dev);
        if (cudaMemsetAsync(gb, 0, sizeof(GridBarrier), stream) != cudaSuccess) return BCAST_ECUDA;
        const unsigned int wanted = (unsigned int)(((int64_t)p + kFusedThreads - 1) / kFusedThreads);
        const unsigned int grid = wanted < together ? wanted : together;
        const int8_t *recv_c = recv_t, *send_c = send_t;
        RoundPlan rp = round_plan(plan);
        rp.blocks = grid + (mode == BCAST_ROUNDS_FUSED_MISS ? 1u : 0u);
        unsigned long long barriers = 0;
        for (int64_t j0 = 0; j0 < rounds; j0 += kRoundsPerLaunch) {
            long long first = j0, end = j0 + kRoundsPerLaunch < rounds ? j0 + kRoundsPerLaunch : rounds;
            void *args[] = {&fr, &recv_c, &send_c, &rp, &first, &end, &gb, &barriers, &stats};
            if (cudaLaunchCooperativeKernel((const void *)broadcast_rounds_kernel, dim3(grid), dim3(kFusedThreads),
                                            args, 0, stream) != cudaSuccess) {
                // refused before anything ran (the device is shared, say): one launch per round instead,
                // unless the fused form was asked for
                if (j0 != 0 || mode != BCAST_ROUNDS_AUTO) return BCAST_ECUDA;
                (void)cudaGetLastError();
                fused = false;
                break;
            }
            barriers += (unsigned long long)(end - first - 1);
        }
        if (fused) seal_stats_after = gb;
    }
    if (!fused) {
        const unsigned int round_blocks = blocks < resident ? blocks : resident;
        for (int64_t j = 0; j < rounds; ++j) {
            const int64_t i = plan.x + j;
            const int k = (int)(i % q);
            const int64_t shift = (i / q) * q - plan.x;                // Theorem 1
            broadcast_round_kernel<<<round_blocks, kThreads, 0, stream>>>(
                fr, recv_t + (size_t)k * plan.P, send_t + (size_t)k * plan.P, plan.skip[k], (int)shift, (int32_t)(j + 1),
                stats);
        }
    }
    for (int64_t w0 = 0; w0 < set_words(n); w0 += 65535) {
        const unsigned int nw = (unsigned int)(set_words(n) - w0 < 65535 ? set_words(n) - w0 : 65535);
        count_missing_sets_kernel<<<dim3(blocks < resident ? blocks : resident, nw), kThreads, 0, stream>>>(
            held + (size_t)w0 * plan.P, (size_t)plan.P, (uint32_t)p, n - 64 * w0, stats);
    }
    if (seal_stats_after != nullptr) seal_stats_kernel<<<1, 32, 0, stream>>>(seal_stats_after, stats);
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return q;
}

int bcast_simulate_reduce(int32_t p, int32_t root, int64_t n,
                          const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                          uint64_t *value_dev, uint64_t *result_dev, uint64_t *stats_dev,
                          void *scratch_dev, int64_t scratch_bytes, void *cuda_stream)
{
    const int rc = check_common(p, root, n, recvblock_dev, sendblock_dev, value_dev, stats_dev);
    if (rc != BCAST_OK) return rc;
    if (result_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)value_dev & 7u) || ((uintptr_t)result_dev & 7u)) return BCAST_EALIGN;
    const Plan plan = make_plan(p, n);
    const int q = plan.q;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long *stats = reinterpret_cast<unsigned long long *>(stats_dev);
    if (cudaMemsetAsync(stats_dev, 0, 8 * sizeof(uint64_t), stream) != cudaSuccess) return BCAST_ECUDA;
    if (q == 0) {                                                  // one processor: its values are the result
        copy_row_kernel<<<(unsigned int)((n + 255) / 256), 256, 0, stream>>>(value_dev, result_dev, n);
        return cudaGetLastError() == cudaSuccess ? 0 : BCAST_ECUDA;
    }
    if (scratch_dev == nullptr) return BCAST_ENULL;
    if ((uintptr_t)scratch_dev & 15u) return BCAST_EALIGN;
    if (scratch_bytes < bcast_simulate_scratch_bytes(p, n, 1)) return BCAST_ESCRATCH;
    int8_t *recv_t = reinterpret_cast<int8_t *>(scratch_dev) + kHeaderBytes;
    int8_t *send_t = recv_t + (size_t)q * plan.P;
    unsigned long long *once = reinterpret_cast<unsigned long long *>(send_t + (size_t)q * plan.P);
    unsigned long long *twice = once + (size_t)set_words(n) * plan.P;
    if (cudaMemsetAsync(once, 0, (size_t)2 * set_words(n) * plan.P * 8, stream) != cudaSuccess) return BCAST_ECUDA;
    const unsigned int blocks = (unsigned int)(((int64_t)p + kThreads - 1) / kThreads);
    transpose_tables_kernel<<<dim3(blocks, 2), kThreads, 0, stream>>>(
        recvblock_dev, sendblock_dev, recv_t, send_t, (uint32_t)p, q, (size_t)plan.P, stats);
    const int64_t rounds = n - 1 + q;
    const unsigned int resident = (unsigned int)device_sm_count() * 8u;
    const unsigned int round_blocks = blocks < resident ? blocks : resident;
    const int mode = rounds_mode();
    const unsigned int together =
        mode == BCAST_ROUNDS_LAUNCHES ? 0u : cooperative_blocks((const void *)reduce_rounds_kernel);
    if ((mode == BCAST_ROUNDS_FUSED || mode == BCAST_ROUNDS_FUSED_MISS) && together == 0u) return BCAST_ECUDA;
    GridBarrier *gb = nullptr;
    bool fused = together != 0u;
    if (fused) {
        gb = reinterpret_cast<GridBarrier *>(scratch_dev);
        if (cudaMemsetAsync(gb, 0, sizeof(GridBarrier), stream) != cudaSuccess) return BCAST_ECUDA;
        const unsigned int wanted = (unsigned int)(((int64_t)p + kFusedThreads - 1) / kFusedThreads);
        const unsigned int grid = wanted < together ? wanted : together;
        const int8_t *recv_c = recv_t, *send_c = send_t;
        size_t P = (size_t)plan.P;
        uint32_t up = (uint32_t)p, uroot = (uint32_t)root;
        int last = (int)(n - 1);
        RoundPlan rp = round_plan(plan);
        rp.blocks = grid + (mode == BCAST_ROUNDS_FUSED_MISS ? 1u : 0u);
        unsigned long long barriers = 0;
        for (int64_t j1 = rounds; j1 > 0; j1 -= kRoundsPerLaunch) {    // the broadcast's rounds, last one first
            long long end = j1, first = j1 > kRoundsPerLaunch ? j1 - kRoundsPerLaunch : 0;
            void *args[] = {&recv_c, &send_c, &value_dev, &once, &twice, &P, &up, &uroot, &last, &rp, &first, &end,
                            &gb, &barriers, &stats};
            if (cudaLaunchCooperativeKernel((const void *)reduce_rounds_kernel, dim3(grid), dim3(kFusedThreads), args, 0,
                                            stream) != cudaSuccess) {
                if (j1 != rounds || mode != BCAST_ROUNDS_AUTO) return BCAST_ECUDA;
                (void)cudaGetLastError();                          // refused before anything ran: see the broadcast
                fused = false;
                gb = nullptr;
                break;
            }
            barriers += (unsigned long long)(end - first - 1);
        }
    }
    if (!fused) {
        for (int64_t j = rounds - 1; j >= 0; --j) {                // the broadcast's rounds, last one first
            const int64_t i = plan.x + j;
            const int k = (int)(i % q);
            const int64_t shift = (i / q) * q - plan.x;
            reduce_round_kernel<<<round_blocks, kThreads, 0, stream>>>(
                recv_t + (size_t)k * plan.P, send_t + (size_t)k * plan.P, value_dev, once, twice, (size_t)plan.P,
                (uint32_t)p, (uint32_t)root, (int)(n - 1), plan.skip[k], (int)shift, stats);
        }
    }
    for (int64_t b0 = 0; b0 < n; b0 += 65535) {
        const unsigned int nb = (unsigned int)(n - b0 < 65535 ? n - b0 : 65535);
        reduce_finish_kernel<<<dim3(blocks, nb), kThreads, 0, stream>>>(
            value_dev, once, twice, (size_t)plan.P, result_dev, (uint32_t)p, (uint32_t)root, b0, stats);
    }
    if (gb != nullptr) seal_stats_kernel<<<1, 32, 0, stream>>>(gb, stats);
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return q;
}

int64_t bcast_simulate_all_scratch_bytes(int32_t p, int64_t n, int reduction)
{
    if (p < 1) return BCAST_EINVAL_P;
    if (n < 1) return BCAST_EINVAL_N;
    const int q = host_q(p);
    int64_t bytes = kHeaderBytes + 2 * (int64_t)q * padded(p);
    if (reduction) bytes += (int64_t)p * n * (int64_t)p;           // sent counts, a byte per (root, block, processor)
    return bytes;
}

int bcast_simulate_allbroadcast(int32_t p, int64_t n,
                                const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                                int32_t *arrival_dev, uint64_t *stats_dev,
                                void *scratch_dev, int64_t scratch_bytes, void *cuda_stream)
{
    const int rc = check_common(p, 0, n, recvblock_dev, sendblock_dev, arrival_dev, stats_dev);
    if (rc != BCAST_OK) return rc;
    if ((uintptr_t)arrival_dev & 3u) return BCAST_EALIGN;
    const Plan plan = make_plan(p, n);
    const int q = plan.q;
    if (q > 0) {
        if (scratch_dev == nullptr) return BCAST_ENULL;
        if ((uintptr_t)scratch_dev & 15u) return BCAST_EALIGN;
        if (scratch_bytes < bcast_simulate_all_scratch_bytes(p, n, 0)) return BCAST_ESCRATCH;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long *stats = reinterpret_cast<unsigned long long *>(stats_dev);
    if (cudaMemsetAsync(stats_dev, 0, 8 * sizeof(uint64_t), stream) != cudaSuccess) return BCAST_ECUDA;
    const unsigned int blocks = (unsigned int)(((int64_t)p + kThreads - 1) / kThreads);
    // the roots go in slices of at most 65535 (the grid's y limit)
    for (int64_t j0 = 0; j0 < p; j0 += 65535) {
        const unsigned int nj = (unsigned int)(p - j0 < 65535 ? p - j0 : 65535);
        init_arrival_all_kernel<<<dim3(blocks, nj), kThreads, 0, stream>>>(arrival_dev, (uint32_t)p, (uint32_t)j0, n);
    }
    if (q > 0) {
        int8_t *recv_t = reinterpret_cast<int8_t *>(scratch_dev) + kHeaderBytes;
        int8_t *send_t = recv_t + (size_t)q * plan.P;
        transpose_tables_kernel<<<dim3(blocks, 2), kThreads, 0, stream>>>(
            recvblock_dev, sendblock_dev, recv_t, send_t, (uint32_t)p, q, (size_t)plan.P, stats);
        scale_bad_entries_kernel<<<1, 1, 0, stream>>>(stats, (unsigned long long)p);
        const int64_t rounds = n - 1 + q;
        for (int64_t jr = 0; jr < rounds; ++jr) {
            const int64_t i = plan.x + jr;
            const int k = (int)(i % q);
            const int64_t shift = (i / q) * q - plan.x;
            for (int64_t j0 = 0; j0 < p; j0 += 65535) {
                const unsigned int nj = (unsigned int)(p - j0 < 65535 ? p - j0 : 65535);
                allbroadcast_round_kernel<<<dim3(blocks, nj), kThreads, 0, stream>>>(
                    recv_t + (size_t)k * plan.P, send_t + (size_t)k * plan.P, arrival_dev, (uint32_t)p,
                    (uint32_t)j0, n, plan.skip[k], shift, (int32_t)(jr + 1), stats);
            }
        }
    }
    const size_t cells = (size_t)p * (size_t)n * (size_t)p;
    const size_t want_blocks = (cells + kThreads - 1) / kThreads;
    const size_t most = (size_t)device_sm_count() * 16;
    count_missing_kernel<<<(unsigned int)(want_blocks < most ? want_blocks : most), kThreads, 0, stream>>>(
        arrival_dev, cells, stats);
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return q;
}

int bcast_simulate_allreduce(int32_t p, int64_t n,
                             const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                             uint64_t *value_dev, uint64_t *result_dev, uint64_t *stats_dev,
                             void *scratch_dev, int64_t scratch_bytes, void *cuda_stream)
{
    const int rc = check_common(p, 0, n, recvblock_dev, sendblock_dev, value_dev, stats_dev);
    if (rc != BCAST_OK) return rc;
    if (result_dev == nullptr) return BCAST_ENULL;
    if (((uintptr_t)value_dev & 7u) || ((uintptr_t)result_dev & 7u)) return BCAST_EALIGN;
    const Plan plan = make_plan(p, n);
    const int q = plan.q;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long *stats = reinterpret_cast<unsigned long long *>(stats_dev);
    if (cudaMemsetAsync(stats_dev, 0, 8 * sizeof(uint64_t), stream) != cudaSuccess) return BCAST_ECUDA;
    if (q == 0) {
        copy_row_kernel<<<(unsigned int)((n + 255) / 256), 256, 0, stream>>>(value_dev, result_dev, n);
        return cudaGetLastError() == cudaSuccess ? 0 : BCAST_ECUDA;
    }
    if (scratch_dev == nullptr) return BCAST_ENULL;
    if ((uintptr_t)scratch_dev & 15u) return BCAST_EALIGN;
    if (scratch_bytes < bcast_simulate_all_scratch_bytes(p, n, 1)) return BCAST_ESCRATCH;
    int8_t *recv_t = reinterpret_cast<int8_t *>(scratch_dev) + kHeaderBytes;
    int8_t *send_t = recv_t + (size_t)q * plan.P;
    uint8_t *sent = reinterpret_cast<uint8_t *>(send_t + (size_t)q * plan.P);
    if (cudaMemsetAsync(sent, 0, (size_t)p * (size_t)n * (size_t)p, stream) != cudaSuccess) return BCAST_ECUDA;
    const unsigned int blocks = (unsigned int)(((int64_t)p + kThreads - 1) / kThreads);
    transpose_tables_kernel<<<dim3(blocks, 2), kThreads, 0, stream>>>(
        recvblock_dev, sendblock_dev, recv_t, send_t, (uint32_t)p, q, (size_t)plan.P, stats);
    scale_bad_entries_kernel<<<1, 1, 0, stream>>>(stats, (unsigned long long)p);
    const int64_t rounds = n - 1 + q;
    for (int64_t jr = rounds - 1; jr >= 0; --jr) {                 // the all-broadcast's rounds, last one first
        const int64_t i = plan.x + jr;
        const int k = (int)(i % q);
        const int64_t shift = (i / q) * q - plan.x;
        for (int64_t j0 = 0; j0 < p; j0 += 65535) {
            const unsigned int nj = (unsigned int)(p - j0 < 65535 ? p - j0 : 65535);
            allreduce_round_kernel<<<dim3(blocks, nj), kThreads, 0, stream>>>(
                recv_t + (size_t)k * plan.P, send_t + (size_t)k * plan.P, value_dev, sent, (uint32_t)p, (uint32_t)j0,
                n, plan.skip[k], shift, stats);
        }
    }
    for (int64_t j0 = 0; j0 < p; j0 += 65535) {
        const unsigned int nj = (unsigned int)(p - j0 < 65535 ? p - j0 : 65535);
        allreduce_finish_kernel<<<dim3(blocks, nj), kThreads, 0, stream>>>(value_dev, sent, result_dev, (uint32_t)p,
                                                                           (uint32_t)j0, n, stats);
    }
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return q;
}

}  // extern "C"
