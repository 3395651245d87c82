/*
 * bcast_sched.h -- C ABI of the broadcast-schedule library (CUDA, sm_100a).
 *
 * Computes, for p processors on the ceil(log2 p)-regular circulant graph, the
 * round-optimal n-block broadcast schedule of J. L. Traff, "Optimal Broadcast
 * Schedules in Logarithmic Time with Applications to Broadcast, All-Broadcast,
 * Reduction and All-Reduction" (arXiv 2407.18004): the skips, and for each
 * processor its recvblock[] and sendblock[] arrays of q = ceil(log2 p) entries.
 *
 * Conventions for every entry point
 *  - Plain C types only.  "host" pointers are ordinary process memory; "device"
 *    pointers are CUDA global memory of the current device.  The caller owns
 *    every buffer and the library allocates nothing.  It is thread-safe and
 *    keeps no state between calls, with three documented exceptions: the
 *    process-wide overrides of bcast_set_launch_shape and
 *    bcast_set_simulate_rounds, and the built-in scratch array of
 *    bcast_verify_sweep_static.
 *  - cuda_stream is a cudaStream_t passed as void* (NULL = default stream).
 *    Device work is enqueued on it and the call returns without synchronising.
 *  - Return value: >= 0 on success (where stated, the value of q), otherwise a
 *    negative BCAST_E* code.  Bad arguments are detected on the host before
 *    anything is launched; nothing is thrown across the ABI.
 *  - 1 <= p <= 2^31-1.  Processors are numbered 0..p-1.  A root other than 0 is
 *    handled by renumbering (Section 2): the row of actual rank a holds the
 *    schedule of virtual rank (a - root + p) mod p.
 *  - Schedule entries are int32 in [-q, q-1] for rounds k = 0..q-1.  A negative
 *    entry names a block of an earlier phase (Algorithm 1 adds q per phase).
 *  - The search of Algorithms 4 and 5 runs as a loop with an iteration cap far
 *    above the bound of Lemma 6.  No p is known to reach the cap; should a
 *    search ever do so, the entries it still owed read BCAST_UNRESOLVED in the
 *    tables of bcast_schedule / bcast_allbroadcast_schedule / bcast_schedule_host
 *    (BCAST_PAD in the rows of bcast_schedule_batch; bcast_schedule_shifted adds
 *    its shift to the marker byte and does not preserve it), and
 *    bcast_verify_sweep counts the event in fail_counts[7].
 */
#ifndef BCAST_SCHED_H
#define BCAST_SCHED_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BCAST_OK            0
#define BCAST_EINVAL_P     -1   /* p < 1 or p > 2^31-1                                  */
#define BCAST_EINVAL_ROOT  -2   /* root outside [0, p)                                  */
#define BCAST_EINVAL_RANGE -3   /* not 0 <= rank_begin <= rank_end <= p, or p_lo > p_hi */
#define BCAST_ENULL        -4   /* a required pointer is NULL                           */
#define BCAST_EALIGN       -5   /* a device pointer is not aligned as documented        */
#define BCAST_EINVAL_N     -6   /* n < 1, q < 1 or nq < 0                               */
#define BCAST_EINVAL_ROUND -7   /* round j outside [0, n-1+q)                           */
#define BCAST_ECUDA        -8   /* a CUDA runtime call failed (launch, attribute query) */
#define BCAST_ESTRIDE      -9   /* row_stride below 31                                  */
#define BCAST_ESCRATCH     -10  /* scratch buffer too small for a single p of the range */
#define BCAST_ETOOBIG      -11  /* p_hi above BCAST_STATIC_SWEEP_MAX_P                  */
#define BCAST_EINVAL_SHAPE -12  /* not one of BCAST_SHAPE_*                             */

#define BCAST_NONE         (-1)         /* bcast_round_block: nothing moves in this round */
#define BCAST_PAD          INT32_MIN    /* filler of unused row entries in the batch form */
#define BCAST_UNRESOLVED   (-128)       /* table entry a capped search never reached (see above) */
#define BCAST_MAX_Q        31

/* Launch shapes of the table kernel (bcast_set_launch_shape). */
#define BCAST_SHAPE_AUTO     (-1)       /* chosen per call from an estimate (the default)          */
#define BCAST_SHAPE_BLOCK      0        /* a block per tile, undecided entries searched per tile   */
#define BCAST_SHAPE_WARPS      1        /* warps on their own, searches deferred to the block's end */
#define BCAST_SHAPE_LOWFRAME   2        /* the same, low rounds looked up in a table of low states */
#define BCAST_SHAPE_WARPS_TIGHT 3       /* BCAST_SHAPE_WARPS with next to no queue space: for tests */
                                        /* of the path that recomputes a group whose queues ran full */

/* How bcast_simulate_broadcast / bcast_simulate_reduce launch their rounds (bcast_set_simulate_rounds). */
#define BCAST_ROUNDS_AUTO      0        /* fused where the device has cooperative launches (default) */
#define BCAST_ROUNDS_LAUNCHES  1        /* one kernel launch per communication round                  */
#define BCAST_ROUNDS_FUSED     2        /* all rounds in cooperative launches, blocks meet per round   */
#define BCAST_ROUNDS_FUSED_MISS 3       /* for tests of the bounded wait: BCAST_ROUNDS_FUSED whose blocks */
                                        /* wait for one block more than there are; every call with more   */
                                        /* than one round ends, after a second or two, with all eight   */
                                        /* statistics words UINT64_MAX                                     */

#define BCAST_STATIC_SWEEP_BYTES  (8u << 20)   /* built-in scratch of bcast_verify_sweep_static */
#define BCAST_STATIC_SWEEP_MAX_P  65536        /* largest p_hi it accepts                       */

/* Text for a BCAST_E* code (static storage, never NULL). */
const char *bcast_strerror(int code);

/*
 * q = ceil(log2 p), the number of skips, of rounds per phase and of entries
 * per schedule row (Section 2).  p = 1 gives 0.  Host only.
 */
int bcast_q(int32_t p);

/*
 * Algorithm 2: the skips of the circulant graph, skip[q] = p and
 * skip[k-1] = ceil(skip[k] / 2), so skip[0] = 1 and skip[1] = 2 for p > 1.
 * skip_host: host array of q+1 (at most 32) int32, written by the call.
 * Returns q.  Host only, O(q).
 */
int bcast_skips(int32_t p, int32_t *skip_host);

/*
 * Algorithms 3-6 for every actual rank a in [rank_begin, rank_end):
 * row a - rank_begin of recvblock_dev receives Algorithm 5's receive schedule
 * and the same row of sendblock_dev the send schedule (Section 2.3:
 * sendblock[k] of r equals recvblock[k] of (r + skip[k]) mod p) of virtual rank
 * (a - root + p) mod p.
 * Layout: device memory, int32, row-major, (rank_end - rank_begin) rows of
 * exactly q entries, no padding; 4-byte aligned (16-byte aligned pointers take
 * the vector-store path).  Either table pointer may be NULL to skip that table,
 * not both.  An empty rank range and p = 1 (q = 0) succeed without a launch.
 * Asynchronous on cuda_stream.  Returns q.
 * The kernel has three launch shapes, chosen per call from an estimate of how
 * many entries of this p the closed forms leave to the search of Algorithms 4
 * and 5 (bcast_set_launch_shape forces one).  The tables are the same in all.
 */
int bcast_schedule(int32_t p, int32_t root, int64_t rank_begin, int64_t rank_end,
                   int32_t *recvblock_dev, int32_t *sendblock_dev, void *cuda_stream);

/*
 * Force a launch shape of the table kernel for all later calls of this process
 * (tuning, and tests that run every shape on the same p): one of BCAST_SHAPE_*;
 * BCAST_SHAPE_AUTO restores the per-call choice.  A shape a call cannot take
 * (shifted tables, small q) falls back to one it can.  Until the first call of
 * this function the environment variable BCAST_LAUNCH_SHAPE=block|warps|lowframe|tight,
 * read once, has the same effect.  Results never depend on the shape.  (No
 * counterpart in the paper.)  Returns BCAST_OK or BCAST_EINVAL_SHAPE.
 */
int bcast_set_launch_shape(int shape);

/*
 * bcast_schedule with the rows already prepared for n blocks, i.e. after the
 * preamble of Algorithm 1: with x = (q - (n-1) mod q) mod q virtual rounds in
 * front, every entry has x subtracted, and the entries of the rounds k < x
 * (already "done" when communication starts) have q added, so that the loop of
 * Algorithm 1 can use entry k = i mod q as it is and add q after each use.
 * Entries lie in [-2q+1, 2q-2].  n >= 1 (BCAST_EINVAL_N otherwise); everything
 * else as for bcast_schedule.  n - 1 a multiple of q gives x = 0 and the
 * unshifted tables.  Returns q; x is what bcast_round reports as -shift for
 * round j = 0.
 */
int bcast_schedule_shifted(int32_t p, int32_t root, int64_t n, int64_t rank_begin, int64_t rank_end,
                           int32_t *recvblock_dev, int32_t *sendblock_dev, void *cuda_stream);

/*
 * The schedule part of Algorithm 7 (all-broadcast, Appendix A) for one processor
 * `rank`: with every processor j as root in turn, row j - root_begin of
 * recvblocks_dev receives recvschedule((rank - j + p) mod p) and the same row of
 * sendblocks_dev the send schedule for that root, which Algorithm 7 defines as
 * sendblocks[j][k] = recvblocks[(j - skip[k] + p) mod p][k], for the roots j in
 * [root_begin, root_end).  These are the rows of bcast_schedule's tables listed
 * by descending virtual rank; layout, alignment, NULL rules, asynchrony and
 * return value are those of bcast_schedule (BCAST_EINVAL_ROOT stands for a rank
 * outside [0, p)).
 */
int bcast_allbroadcast_schedule(int32_t p, int32_t rank, int64_t root_begin, int64_t root_end,
                                int32_t *recvblocks_dev, int32_t *sendblocks_dev, void *cuda_stream);

/*
 * bcast_schedule with HOST output tables: the rank range is cut into chunks that
 * fit the caller's device staging buffer (staging_dev, staging_bytes, 16-byte
 * aligned; it must hold at least 32 rows of each requested table); each chunk
 * is computed on the device and then copied into recvblock_host /
 * sendblock_host (same layout as above, rows of the whole range) with
 * cudaMemcpyAsync on cuda_stream.  Pinned host memory makes the copies
 * asynchronous; pageable memory works and is slower.  The tables are complete
 * once the stream has been synchronised.  Returns q, or BCAST_ESCRATCH when the
 * staging buffer is too small.
 */
int bcast_schedule_host(int32_t p, int32_t root, int64_t rank_begin, int64_t rank_end,
                        int32_t *recvblock_host, int32_t *sendblock_host,
                        void *staging_dev, int64_t staging_bytes, void *cuda_stream);

/*
 * The same computation for nq independent queries (p_i, rank_i, root_i), all in
 * device memory (int32, 4-byte aligned).  Row i of each output (int32,
 * row-major, row_stride >= 31 entries per row) holds q_i = ceil(log2 p_i)
 * schedule entries followed by BCAST_PAD up to row_stride.  A query with
 * p_i < 1 or rank_i / root_i outside [0, p_i) gets a row of BCAST_PAD only and
 * is counted in *bad_count_dev (device int32, may be NULL; the caller zeroes
 * it).  Either output may be NULL, not both.  Asynchronous on cuda_stream.
 */
int bcast_schedule_batch(const int32_t *p_dev, const int32_t *rank_dev, const int32_t *root_dev,
                         int64_t nq, int32_t row_stride,
                         int32_t *recvblock_dev, int32_t *sendblock_dev,
                         int32_t *bad_count_dev, void *cuda_stream);

/*
 * Fused verification sweep (the exhaustive check of Section 2.3 / Appendix B)
 * for every p in [p_lo, p_hi], root 0, all ranks, without writing tables to
 * the caller: per p it computes all receive and send rows with the same
 * device code as bcast_schedule, then checks on the device
 *   [0] condition 1: recvblock[k]_r = sendblock[k] of (r - skip[k]) mod p
 *   [1] condition 2: sendblock[k]_r = recvblock[k] of (r + skip[k]) mod p
 *   [2] condition 3: the q received blocks are {-1..-q} \ {b-q} U {b}
 *                    (the root: exactly {-1..-q})
 *   [3] condition 4: sendblock[k] was received in a round j < k or is b - q
 *   [4] Theorem 3:   more than 4 violations in Algorithm 6
 *   [5] Lemmas 5, 6: more than q-1 descents or 2q+R list steps in the search
 *   [6] root row sendblock[k] = k and sendblock[0] = b - q for the others
 *   [7] internal:    the search ran into its iteration cap
 * and adds the number of failing (rank, round) pairs to fail_counts_dev[0..7]
 * (device uint32[8]; the caller zeroes it; all zero means every check passed).
 * checksum_dev[p - p_lo] (device uint64, 8-byte aligned) receives the wrapping
 * sum over all (r, k) of mix(r*2^32 + k*2^16 + (recv & 255)*2^8 + (send & 255)),
 * mix being the SplitMix64 output finaliser; p = 1 gives 0.
 * scratch_dev: device memory of scratch_bytes bytes, 16-byte aligned, used for
 * the per-p tables while they are checked; bcast_verify_sweep_scratch_bytes()
 * gives the size that lets every SM work; any size of at least
 * 256 + (2 * q(p_hi) * (p_hi + 1) rounded up to a multiple of 256) bytes is accepted
 * and uses fewer blocks.  Contents after the call are unspecified.
 * Asynchronous on cuda_stream; two sweeps that share a scratch buffer must not
 * overlap on the device.
 */
int64_t bcast_verify_sweep_scratch_bytes(int32_t p_lo, int32_t p_hi);
int bcast_verify_sweep(int32_t p_lo, int32_t p_hi, uint64_t *checksum_dev,
                       uint32_t *fail_counts_dev, void *scratch_dev, int64_t scratch_bytes,
                       void *cuda_stream);

/*
 * bcast_verify_sweep for callers that cannot allocate device memory.  (The paper
 * has no counterpart; this is a packaging variant of the sweep above.)
 *
 * Some hosts of this library may not call cudaMalloc at the point where they
 * want a sweep: code running inside a memory-pool or real-time section that
 * forbids allocation, a plug-in that is handed output buffers but no allocator,
 * a process whose allocator is owned by another runtime.  For them the per-p
 * tables go into a fixed array of BCAST_STATIC_SWEEP_BYTES (8 MiB) that is part
 * of the library's device image; each GPU that loads the library holds it until
 * the process ends.  The caller still owns and passes checksum_dev and
 * fail_counts_dev (same meaning, alignment and zeroing rules as above).
 *
 * Limits and rules
 *  - p_hi <= BCAST_STATIC_SWEEP_MAX_P (65536), else BCAST_ETOOBIG; nothing is
 *    launched.  The array holds three blocks' worth of tables at that size, so
 *    large ranges run with less parallelism than bcast_verify_sweep with the
 *    scratch size it recommends; results are identical.
 *  - The call itself performs no cudaMalloc/cudaFree and uses no allocating
 *    library routine.
 *  - The first call on each device looks the array's device address up
 *    (cudaGetSymbolAddress, with that device current) and remembers it; make
 *    that first call before any stream capture is started.
 *  - All calls on a device share the one array and it keeps whatever the last
 *    call left; the sweep clears its work-queue counter itself at the start of
 *    each call and reads nothing else before writing it.  Two calls whose device
 *    work overlaps (different streams, different host threads) race on the
 *    array: serialise them.
 * Asynchronous on cuda_stream.  Returns BCAST_OK or a BCAST_E* code.
 */
int bcast_verify_sweep_static(int32_t p_lo, int32_t p_hi, uint64_t *checksum_dev,
                              uint32_t *fail_counts_dev, void *cuda_stream);

/*
 * Algorithm 1 carried out by all p processors at once on given tables (Section 2;
 * the exceptions are those the paper leaves to its Send||Recv operation): in
 * communication round j = 0 .. n-2+q, with i = x + j, k = i mod q, processor a
 * sends block sendblock[a][k] + q*floor(i/q) - x to (a + skip[k]) mod p and
 * receives block recvblock[a][k] + q*floor(i/q) - x from (a - skip[k]) mod p; a
 * negative block moves nothing, a block above n-1 stands for block n-1, nothing
 * is sent to the root and the root receives nothing.  A stronger check than the
 * conditions of bcast_verify_sweep: the blocks really travel.
 *
 * recvblock_dev, sendblock_dev: device int32 tables [p][q] of ALL actual ranks
 * as bcast_schedule(p, root, 0, p, ...) writes them (not modified; NULL allowed
 * only for p = 1).
 * arrival_dev: device int32 [n][p], written by the call: arrival[b*p + a] is the
 * round, counted from 1, in which processor a received block b; 0 for the root;
 * -1 if the block never arrived.  A block is delivered only when the sender
 * sends exactly the block the receiver expects, held it before the round, and
 * the receiver does not hold it yet.
 * stats_dev: device uint64[8], 8-byte aligned, zeroed and filled by the call:
 *   [0] receiver expects a block, its from-processor sends another one or nothing
 *   [1] matching block that the sender did not hold before the round
 *   [2] matching block that the receiver already holds
 *   [3] a block sent to a processor (not the root) that expects nothing
 *   [4] (processor, block) pairs still missing after the last round
 *   [5] table entries outside [-q, q-1] (they move nothing in any round)
 *   [6] blocks delivered                    (correct tables: (p-1)*n)
 *   [7] last round that delivered a block   (correct tables: n-1+q)
 * Correct tables give zeros in [0..5].
 * scratch_dev: device memory, 16-byte aligned, at least
 * bcast_simulate_scratch_bytes(p, n, 0) bytes; it receives round-major byte
 * copies of the tables and a bit per (processor, block) for who holds what.
 * Contents after the call are unspecified.
 * Asynchronous on cuda_stream.  Returns q.
 * Limits: n < 2^31 - 64; n * p int32 cells must fit the caller's memory.
 *
 * The n-1+q rounds run either as one small launch each or, by default where the
 * device has cooperative launches (and grants this one), inside cooperative launches of up to 65536
 * rounds whose blocks meet at a counter in the scratch between two rounds (a
 * round of 2^20 processors is too short to pay for a launch of its own).  That
 * wait is bounded: should a block see no progress for a second or two (all
 * blocks of a cooperative launch are resident, so this is not expected), every
 * block stops and ALL EIGHT statistics words are set to UINT64_MAX; arrival_dev
 * is then unspecified.  Both forms give the same arrival table and statistics.
 */
int64_t bcast_simulate_scratch_bytes(int32_t p, int64_t n, int reduction);

/*
 * Not from the paper: forces how the two single-root simulators launch their
 * rounds from now on, process-wide (tuning, and tests that run both forms on the
 * same tables): one of BCAST_ROUNDS_*.  BCAST_ROUNDS_FUSED on a device without
 * cooperative launches makes those calls return BCAST_ECUDA.  The environment
 * variable BCAST_SIMULATE_ROUNDS=launches|fused, read once at the first
 * simulation, does the same until this is called.  Host only.  Returns BCAST_OK
 * or BCAST_EINVAL_SHAPE.
 */
int bcast_set_simulate_rounds(int mode);

int bcast_simulate_broadcast(int32_t p, int32_t root, int64_t n,
                             const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                             int32_t *arrival_dev, uint64_t *stats_dev,
                             void *scratch_dev, int64_t scratch_bytes, void *cuda_stream);

/*
 * The reduction of Observation 1, item 3: the rounds of Algorithm 1 taken from
 * the last to the first with every communication reversed.  In the round that
 * is broadcast round i, processor a sends its partial result of block
 * recvblock[a][k] + q*floor(i/q) - x to its from-processor (a - skip[k]) mod p
 * and receives a partial result of block sendblock[a][k] + q*floor(i/q) - x from
 * its to-processor (a + skip[k]) mod p, which it combines with its own.  The
 * root sends nothing, a processor whose to-processor is the root receives
 * nothing; negative blocks and blocks above n-1 as in the broadcast.  The
 * operator is the wrapping sum of uint64.
 *
 * value_dev: device uint64 [n][p], 8-byte aligned: value[b*p + a] is processor
 * a's contribution to block b on entry and its partial result on return.
 * result_dev: device uint64 [n]: the root's value of each block after the last
 * round (correct tables: the sum over all processors).
 * A partial result is combined only when the receiver expects exactly the block
 * the sender sends and has not sent (and is not sending) its own partial result
 * of that block.
 * stats_dev: device uint64[8], zeroed and filled by the call:
 *   [0] receiver expects a block, its to-processor sends another one or nothing
 *   [1] matching block whose partial result the receiver has already passed on
 *   [2] a processor sends a block it has sent before
 *   [3] a block sent to a processor that expects nothing
 *   [4] (non-root processor, block) pairs not sent exactly once
 *   [5] table entries outside [-q, q-1]
 *   [6] partial results combined            (correct tables: (p-1)*n)
 *   [7] unused, 0
 * scratch_dev: at least bcast_simulate_scratch_bytes(p, n, 1) bytes, 16-byte
 * aligned.  Tables, limits, asynchrony, the two ways of launching the rounds
 * (statistics all UINT64_MAX if the bounded wait ran out; value_dev and
 * result_dev then unspecified) and return value as for bcast_simulate_broadcast.
 */
int bcast_simulate_reduce(int32_t p, int32_t root, int64_t n,
                          const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                          uint64_t *value_dev, uint64_t *result_dev, uint64_t *stats_dev,
                          void *scratch_dev, int64_t scratch_bytes, void *cuda_stream);

/*
 * Algorithm 7 carried out by all p processors at once (Observation 1, item 2):
 * every processor is the root of a broadcast of its own n blocks and all p
 * broadcasts share the n-1+q rounds.  In round i = x + j (k = i mod q) processor
 * a packs, for every root but its to-processor (a + skip[k]) mod p, block
 * sendblocks[root][k] + q*floor(i/q) - x, and unpacks, for every root but
 * itself, block recvblocks[root][k] + q*floor(i/q) - x from what its
 * from-processor (a - skip[k]) mod p packed for that root; negative blocks are
 * neither packed nor unpacked, a block above n-1 stands for block n-1.
 *
 * recvblock_dev, sendblock_dev: device int32 tables [p][q] of the broadcast from
 * root 0 as bcast_schedule(p, 0, 0, p, ...) writes them.  One pair serves every
 * processor: its rows for root j (what bcast_allbroadcast_schedule would write
 * for it) are the rows of rank (a - j) mod p of these tables.
 * arrival_dev: device int32 [p][n][p], written by the call:
 * arrival[(root*n + b)*p + a] is the round, counted from 1, in which processor a
 * received block b of that root; 0 for a = root; -1 if it never arrived.
 * stats_dev, delivery rule: as for bcast_simulate_broadcast, the statistics
 * summed over all roots (correct tables: [6] = p*(p-1)*n, [7] = n-1+q).
 * scratch_dev: at least bcast_simulate_all_scratch_bytes(p, n, 0) bytes, 16-byte
 * aligned.  The state has p*p*n cells: sizes are the caller's to keep within
 * its memory (p = 4096, n = 8: 512 MiB of arrival cells).
 * Launches n-1+q small kernels per 65535 roots on cuda_stream.  Returns q.
 */
int64_t bcast_simulate_all_scratch_bytes(int32_t p, int64_t n, int reduction);
int bcast_simulate_allbroadcast(int32_t p, int64_t n,
                                const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                                int32_t *arrival_dev, uint64_t *stats_dev,
                                void *scratch_dev, int64_t scratch_bytes, void *cuda_stream);

/*
 * The all-reduction of Observation 1, item 4 (the reduce-scatter use of the
 * schedules): Algorithm 7's rounds from the last to the first with every
 * communication reversed, p reductions sharing the rounds, each processor the
 * root of the reduction of its own n blocks.  In the round that is all-broadcast
 * round i, processor a sends to its from-processor, for every root but itself,
 * its partial result of block recvblocks[root][k] + q*floor(i/q) - x, and
 * receives from its to-processor t, for every root but t, a partial result of
 * block sendblocks[root][k] + q*floor(i/q) - x, which it adds to its own.  The
 * operator is the wrapping sum of uint64.
 *
 * Tables as for bcast_simulate_allbroadcast.
 * value_dev: device uint64 [p][n][p]: value[(root*n + b)*p + a] is processor a's
 * contribution to block b of that root on entry, partial results on return.
 * result_dev: device uint64 [p][n]: result[root*n + b] is that root's value of
 * its block b after the last round (correct tables: the sum over all
 * processors; every processor ends with the n sums that are its own).
 * stats_dev, combining rule: as for bcast_simulate_reduce, summed over all roots
 * (correct tables: [6] = p*(p-1)*n, zeros in [0..5]).
 * scratch_dev: at least bcast_simulate_all_scratch_bytes(p, n, 1) bytes (it
 * holds a byte per state cell besides the byte tables), 16-byte aligned.
 * Asynchrony, limits and return value as for bcast_simulate_allbroadcast.
 */
int bcast_simulate_allreduce(int32_t p, int64_t n,
                             const int32_t *recvblock_dev, const int32_t *sendblock_dev,
                             uint64_t *value_dev, uint64_t *result_dev, uint64_t *stats_dev,
                             void *scratch_dev, int64_t scratch_bytes, void *cuda_stream);

/*
 * Measurement aid (no counterpart in the paper): fills buffer_dev (device,
 * 16-byte aligned; bytes rounded down to a multiple of 16) with the store
 * pattern of the table kernel and nothing else -- one block of 256 threads per
 * contiguous chunk of bytes_per_block bytes (0: the bytes a block of
 * bcast_schedule writes at q = 27), 16-byte streaming stores.  Its rate is the
 * write-only ceiling the table kernel's HBM fraction can be read against.
 * Asynchronous on cuda_stream.  Returns BCAST_OK or a BCAST_E* code.
 */
int bcast_store_ceiling(void *buffer_dev, int64_t bytes, int64_t bytes_per_block, void *cuda_stream);

/*
 * The table of the search's low states that bcast_schedule hands to its kernel
 * for p whose closed forms leave many entries undecided (no counterpart in the
 * paper as a table: it is Algorithms 4 and 5 memoised on the search's state).
 * Let u be what is left of p + r after the greedy digits of p + r over the
 * skips at the levels >= BCAST_LOW_LEVELS (skip[q] = p first).  For u >= 2 the
 * first rounds of the receive schedule of virtual rank r depend on u alone:
 * nibble k (bits 4k..4k+3, k = 0..7) of states_host[u] is the skip index e the
 * search accepts in round k, i.e. recvblock[k] = e - q; 14 where the search
 * returns past the low levels and accepts the lowest digit j >= BCAST_LOW_LEVELS
 * of p + r (recvblock[k] = j - q, or the baseblock of r when j = q); 15 for the
 * rounds after that one, which the table does not hold.  Entries 0 and 1 are
 * all-ones.  Fills min(skip[BCAST_LOW_LEVELS], capacity) words of states_host
 * (host memory, capacity >= 0) and returns that count; 0 for q < BCAST_LOW_LEVELS + 2,
 * where the kernels do not use it.
 * Pure host computation, no CUDA call.  Errors: BCAST_EINVAL_P, BCAST_ENULL,
 * BCAST_EINVAL_N (capacity < 0).
 */
#define BCAST_LOW_LEVELS 9
int bcast_low_states(int32_t p, uint32_t *states_host, int32_t capacity);

/*
 * Algorithm 1's use of a schedule row, O(1) per round.  For n >= 1 blocks and
 * communication round j in [0, n-1+q): x = (q - (n-1) mod q) mod q virtual
 * rounds come first, so i = x + j, k = i mod q is the skip index of the round
 * (peers (r +- skip[k]) mod p) and shift = q * floor(i/q) - x is what
 * Theorem 1 adds to the row entry.  Host only.
 */
int bcast_round(int32_t q, int64_t n, int64_t j, int32_t *k_out, int64_t *shift_out);

/*
 * The block a processor moves in round j given its row (host, q entries):
 * sched_row[k] + shift, capped to n-1, or BCAST_NONE when negative.  The rules
 * "nothing is sent to the root" and "the root receives nothing" are the
 * caller's.  Returns the block (>= 0), BCAST_NONE, or a BCAST_E* code (< -1).
 */
int64_t bcast_round_block(int32_t q, int64_t n, int64_t j, const int32_t *sched_row_host);

#ifdef __cplusplus
}
#endif

/*
 * The same lookup as bcast_round_block for use inside the caller's own code,
 * host or device (a kernel that moves the blocks reads its row from the table
 * and calls this once per round): Theorem 1's block sched_row[k] + q*floor(i/q) - x
 * with i = x + j, k = i mod q.  No argument checks: q >= 1, n >= 1,
 * 0 <= j < n-1+q are the caller's duty.  *k_out (may be NULL) receives the skip
 * index of the round.  Returns the block, capped to n-1, or BCAST_NONE.
 */
#if defined(__CUDACC__)
#define BCAST_INLINE static __host__ __device__ __forceinline__
#else
#define BCAST_INLINE static inline
#endif
BCAST_INLINE int64_t bcast_round_block_inline(int32_t q, int64_t n, int64_t j, const int32_t *sched_row,
                                              int32_t *k_out)
{
    const int64_t x = (q - (n - 1) % q) % q;
    const int64_t i = x + j;
    const int32_t k = (int32_t)(i % q);
    const int64_t raw = (int64_t)sched_row[k] + (i / q) * q - x;
    if (k_out) *k_out = k;
    if (raw < 0) return BCAST_NONE;
    return raw > n - 1 ? n - 1 : raw;
}

#endif /* BCAST_SCHED_H */
