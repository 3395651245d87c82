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
//   * One thread per processor, one launch per round, all on the caller's stream.  Nothing
//     waits on another block inside a launch.
//   * Broadcast state is arrival[b][a], the round in which processor a got block b.  A
//     sender "held the block before the round" iff its arrival is in [0, round); a value
//     written during the round is >= round, so concurrent readers decide the same way
//     whether or not they see it: one buffer, no race in the outcome.
//   * Reduction state is value[b][a] plus a saturating count sent[b][a]; a receiver reads its
//     to-processor's partial result in place (see reduce_round_kernel for why the outcome
//     does not depend on the order of the threads).
//   * Counters are summed per warp with redux, per block in shared memory, and added to the
//     64-bit statistics with one atomic per block and counter that is not zero.
#include <cuda_runtime.h>
#include <stdint.h>

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
    for (int i = threadIdx.x; i < n_entries; i += kThreads) {
        const int v = src[i];
        const bool ok = v >= -q && v <= q - 1;
        bad += ok ? 0u : 1u;
        const int row = i / q;
        tile[row * 33 + (i - row * q)] = ok ? (int8_t)v : kInvalid;
    }
    __syncthreads();
    if (threadIdx.x < rows)
        for (int k = 0; k < q; ++k) out[(size_t)k * P + first + threadIdx.x] = tile[threadIdx.x * 33 + k];
    add_stat(bstats, 5, bad);
    stats_end(bstats, stats);
}

__global__ void __launch_bounds__(kThreads)
init_arrival_kernel(int32_t *__restrict__ arrival, uint32_t p, uint32_t root)
{
    const uint32_t a = blockIdx.x * kThreads + threadIdx.x;
    if (a < p) arrival[(size_t)blockIdx.y * p + a] = a == root ? 0 : -1;
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
__global__ void __launch_bounds__(kThreads)
broadcast_round_kernel(const int8_t *__restrict__ recv_k, const int8_t *__restrict__ send_k,
                       int32_t *arrival, unsigned long long *held, size_t P, uint32_t p, uint32_t root,
                       int last, uint32_t skip_k, int shift, int32_t round, unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0, c6 = 0;
    // a resident grid strides over the processors: a few thousand blocks would each add their
    // counters to the same statistics words, and those atomics would set the pace of the round
    for (uint32_t a = blockIdx.x * kThreads + threadIdx.x; a < p; a += gridDim.x * kThreads) {
        if (a == root) continue;
        const uint32_t f = a >= skip_k ? a - skip_k : a + (p - skip_k);     // from-processor
        const int want = block32(recv_k[a], shift, last);
        // f's to-processor is a, which is not the root, so f's send is not suppressed
        const int sent = block32(send_k[f], shift, last);
        if (want < 0) {
            c3 += sent >= 0 ? 1u : 0u;
        } else if (sent != want) {
            c0 += 1;
        } else {
            unsigned long long *words = held + (size_t)(want >> 6) * P;
            const unsigned long long bit = 1ull << (want & 63);
            bool f_held = (words[f] & bit) != 0ull;
            if (f_held && f != root && block32(recv_k[f], shift, last) == want) {
                const int32_t at_f = arrival[(size_t)want * p + f];          // f may be getting it only now
                f_held = at_f >= 0 && at_f < round;
            }
            const unsigned long long mine = words[a];
            if (!f_held) c1 += 1;                                            // not held before the round
            else if ((mine & bit) != 0ull) c2 += 1;
            else {
                words[a] = mine | bit;
                arrival[(size_t)want * p + a] = round;
                c6 += 1;
            }
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
__global__ void __launch_bounds__(kThreads)
reduce_round_kernel(const int8_t *__restrict__ recv_k, const int8_t *__restrict__ send_k,
                    uint64_t *value, unsigned long long *once, unsigned long long *twice, size_t P,
                    uint32_t p, uint32_t root, int last, uint32_t skip_k, int shift,
                    unsigned long long *stats)
{
    __shared__ BlockStats bstats;
    stats_begin(bstats);
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0, c6 = 0;
    for (uint32_t a = blockIdx.x * kThreads + threadIdx.x; a < p; a += gridDim.x * kThreads) {
        uint32_t t = a + skip_k;                           // < 2^32: p, skip_k < 2^31
        if (t >= p) t -= p;
        const int mine = a == root ? -1 : block32(recv_k[a], shift, last);         // what a sends
        const int got = t == root ? -1 : block32(recv_k[t], shift, last);          // what t sends to a
        const int want = t == root ? -1 : block32(send_k[a], shift, last);
        // how often a has sent a block: bit in once[] after the first time, in twice[] after the second;
        // thread a alone reads and writes a's words
        bool sent_mine = false;
        if (mine >= 0) {
            sent_mine = (once[(size_t)(mine >> 6) * P + a] >> (mine & 63)) & 1ull;
            if (sent_mine) c2 += 1;
        }
        if (want < 0) {
            if (got >= 0) c3 += 1;
        } else if (got != want) {
            c0 += 1;
        } else if (a != root && (mine == want || ((once[(size_t)(want >> 6) * P + a] >> (want & 63)) & 1ull))) {
            c1 += 1;                                       // it would never be passed on
        } else {
            value[(size_t)want * p + a] += value[(size_t)want * p + t];
            c6 += 1;
        }
        if (mine >= 0) {
            unsigned long long *set = sent_mine ? twice : once;
            set[(size_t)(mine >> 6) * P + a] |= 1ull << (mine & 63);
        }
    }
    add_stat(bstats, 0, c0);
    add_stat(bstats, 1, c1);
    add_stat(bstats, 2, c2);
    add_stat(bstats, 3, c3);
    add_stat(bstats, 6, c6);
    stats_end(bstats, stats);
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

}  // namespace bcast_sim

using namespace bcast_sim;

extern "C" {

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
    // blocks of the arrival table go in slices of at most 65535 (the grid's y limit)
    for (int64_t b0 = 0; b0 < n; b0 += 65535) {
        const unsigned int nb = (unsigned int)(n - b0 < 65535 ? n - b0 : 65535);
        init_arrival_kernel<<<dim3(blocks, nb), kThreads, 0, stream>>>(arrival_dev + (size_t)b0 * p, (uint32_t)p,
                                                                       (uint32_t)root);
    }
    if (q > 0) {
        int8_t *recv_t = reinterpret_cast<int8_t *>(scratch_dev) + kHeaderBytes;
        int8_t *send_t = recv_t + (size_t)q * plan.P;
        unsigned long long *held = reinterpret_cast<unsigned long long *>(send_t + (size_t)q * plan.P);
        const unsigned int pblocks = (unsigned int)(plan.P / kThreads + (plan.P % kThreads != 0));
        for (int64_t w0 = 0; w0 < set_words(n); w0 += 65535) {
            const unsigned int nw = (unsigned int)(set_words(n) - w0 < 65535 ? set_words(n) - w0 : 65535);
            init_block_sets_kernel<<<dim3(pblocks, nw), kThreads, 0, stream>>>(
                held + (size_t)w0 * plan.P, (size_t)plan.P, (uint32_t)p, (uint32_t)root, n - 64 * w0, 1);
        }
        transpose_tables_kernel<<<dim3(blocks, 2), kThreads, 0, stream>>>(
            recvblock_dev, sendblock_dev, recv_t, send_t, (uint32_t)p, q, (size_t)plan.P, stats);
        const int64_t rounds = n - 1 + q;
        const unsigned int resident = (unsigned int)device_sm_count() * 8u;
        const unsigned int round_blocks = blocks < resident ? blocks : resident;
        for (int64_t j = 0; j < rounds; ++j) {
            const int64_t i = plan.x + j;
            const int k = (int)(i % q);
            const int64_t shift = (i / q) * q - plan.x;            // Theorem 1
            broadcast_round_kernel<<<round_blocks, kThreads, 0, stream>>>(
                recv_t + (size_t)k * plan.P, send_t + (size_t)k * plan.P, arrival_dev, held, (size_t)plan.P,
                (uint32_t)p, (uint32_t)root, (int)(n - 1), plan.skip[k], (int)shift, (int32_t)(j + 1), stats);
        }
    }
    if (q > 0) {
        const unsigned long long *held = reinterpret_cast<const unsigned long long *>(
            reinterpret_cast<const int8_t *>(scratch_dev) + kHeaderBytes + 2 * (size_t)q * plan.P);
        const unsigned int resident = (unsigned int)device_sm_count() * 8u;
        for (int64_t w0 = 0; w0 < set_words(n); w0 += 65535) {
            const unsigned int nw = (unsigned int)(set_words(n) - w0 < 65535 ? set_words(n) - w0 : 65535);
            count_missing_sets_kernel<<<dim3(blocks < resident ? blocks : resident, nw), kThreads, 0, stream>>>(
                held + (size_t)w0 * plan.P, (size_t)plan.P, (uint32_t)p, n - 64 * w0, stats);
        }
    }
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
    for (int64_t j = rounds - 1; j >= 0; --j) {                    // the broadcast's rounds, last one first
        const int64_t i = plan.x + j;
        const int k = (int)(i % q);
        const int64_t shift = (i / q) * q - plan.x;
        reduce_round_kernel<<<round_blocks, kThreads, 0, stream>>>(recv_t + (size_t)k * plan.P, send_t + (size_t)k * plan.P,
                                                             value_dev, once, twice, (size_t)plan.P, (uint32_t)p,
                                                             (uint32_t)root, (int)(n - 1), plan.skip[k], (int)shift,
                                                             stats);
    }
    for (int64_t b0 = 0; b0 < n; b0 += 65535) {
        const unsigned int nb = (unsigned int)(n - b0 < 65535 ? n - b0 : 65535);
        reduce_finish_kernel<<<dim3(blocks, nb), kThreads, 0, stream>>>(
            value_dev, once, twice, (size_t)plan.P, result_dev, (uint32_t)p, (uint32_t)root, b0, stats);
    }
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
