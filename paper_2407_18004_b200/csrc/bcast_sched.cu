// C ABI of the broadcast-schedule library (see include/bcast_sched.h): host entry points, the
// launch of the table kernel (schedule_tile.cuh, instantiated per q in table_q_*.cu) and the
// kernel for independent queries.
//
//   schedule_batch_kernel   independent (p, rank, root) queries, one per thread, sorted by q within
//                           a block so that a warp's lanes run loops of like length: receive row
//                           by the search, send row by Algorithm 6; rows padded to row_stride.
#include <cuda_runtime.h>
#include <stdint.h>

#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "../../include/bcast_sched.h"
#include "host_util.h"
#include "table_kernel.cuh"

namespace bcast {

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

// ------------------------------------------------------------------ write-only ceiling
// Nothing but the table kernel's store pattern: every block streams out one contiguous chunk
// with 16-byte st.global.cs, a warp covering 512 contiguous bytes per instruction.
__global__ void __launch_bounds__(kThreads)
store_ceiling_kernel(int4 *__restrict__ out, int64_t n_vec, int64_t vec_per_block)
{
    const int64_t begin = (int64_t)blockIdx.x * vec_per_block;
    const int64_t end = min(begin + vec_per_block, n_vec);
    const int4 v = make_int4((int)blockIdx.x, (int)threadIdx.x, -1, -2);
    for (int64_t i = begin + threadIdx.x; i < end; i += kThreads) __stcs(out + i, v);
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
    case BCAST_EINVAL_SHAPE:  return "launch shape must be one of BCAST_SHAPE_*";
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

// Algorithm 6's violations per rank, estimated on a fixed sample of ranks: the density of entries
// the closed forms leave undecided.  Returns true when it is at most `most` per rank.
static bool undecided_at_most(const LevelTables &tab, int64_t p, int q, double most)
{
    if (q < 2) return true;
    const int kSamples = 80;
    const int limit = (int)(kSamples * most);
    int total = 0;
    uint64_t state = 0x9e3779b97f4a7c15ull ^ (uint64_t)p;
    for (int i = 0; i < kSamples && total <= limit; ++i) {
        state = state * 6364136223846793005ull + 1442695040888963407ull;
        const int64_t r = 1 + (int64_t)((state >> 33) % (uint64_t)(p - 1));
        total += host_violations(tab, p, q, r);
    }
    return total <= limit;
}

// A forced launch shape of the table kernel (tuning, and the tests, which run every shape on the
// same p): process-wide, BCAST_SHAPE_AUTO unless bcast_set_launch_shape() or, at its first use, the
// environment variable BCAST_LAUNCH_SHAPE=block|warps|lowframe|tight says otherwise.
static std::atomic<int> &forced_shape()
{
    static std::atomic<int> forced([] {
        const char *v = getenv("BCAST_LAUNCH_SHAPE");
        if (v == nullptr) return BCAST_SHAPE_AUTO;
        if (strcmp(v, "block") == 0) return BCAST_SHAPE_BLOCK;
        if (strcmp(v, "warps") == 0) return BCAST_SHAPE_WARPS;
        if (strcmp(v, "lowframe") == 0) return BCAST_SHAPE_LOWFRAME;
        if (strcmp(v, "tight") == 0) return BCAST_SHAPE_WARPS_TIGHT;
        return BCAST_SHAPE_AUTO;
    }());
    return forced;
}

// Which launch shape suits p.  With next to no undecided entries (at most 0.05 of Algorithm 6's
// violations per rank; p = 2^27-1 has none) the warps go through the tiles on their own and the block
// runs the few searches at the end.  With more, the launch carries the low rounds of the search
// tabulated for every low state (low_frame_fill), which settles most undecided entries by a lookup and
// leaves few enough searches for the same shape.  The block-per-tile shape, which meets after every
// tile and drains its queues there, serves the shifted tables, small q and descending rows below
// kDescWarpsFromQ.  A wrong estimate costs time, never correctness.
static int choose_shape(const LevelTables &tab, int64_t p, int q, int descending, int shift_x)
{
    if (shift_x != 0) return kShapeBlockPerTile;
    int shape = forced_shape().load(std::memory_order_relaxed);
    if (shape < 0) {
        if (undecided_at_most(tab, p, q, 0.05)) shape = kShapeWarps;
        else shape = q >= kSharedFrom + 2 ? kShapeWarpsLowFrame : kShapeBlockPerTile;
    }
    if (shape == kShapeWarpsLowFrame && q < kSharedFrom + 2) shape = kShapeWarps;
    if (descending && q < kDescWarpsFromQ) shape = kShapeBlockPerTile;
    return shape;
}

// Launch of the table kernel for n_rows output rows starting at global row index row_begin.
static int launch_table(int32_t p, int q, int32_t anchor, int64_t row_begin, int64_t n_rows, int descending,
                        int32_t *recv_dev, int32_t *send_dev, void *cuda_stream, int shift_x = 0)
{
    const int sms = sm_count();
    if (sms <= 0) return BCAST_ECUDA;
    const int64_t n_tiles = (n_rows + kThreads - 1) / kThreads;
    const LevelTables tab = host_tables(p, q);
    const int shape = choose_shape(tab, p, q, descending, shift_x);
    // up to kWarpsPerBlock consecutive tiles per block, fewer while the grid would have less than
    // kBlocksPerSmWanted blocks per SM (short launches want many small blocks).  A block that works with
    // the table of the search's low states copies it to shared memory first and gathers its deferred
    // searches over several groups of tiles, so it takes more: up to kLowFrameTiles.
    int64_t tiles_per_block = n_tiles / ((int64_t)sms * kBlocksPerSmWanted);
    if (tiles_per_block < 1) tiles_per_block = 1;
    if (tiles_per_block > kWarpsPerBlock) tiles_per_block = kWarpsPerBlock;
    if (shape == kShapeWarpsLowFrame) {
        // one wave of resident blocks while that keeps a block within kLowFrameTiles tiles, else blocks of
        // kLowFrameTiles (measured: p = 2^20+1 best at 4 tiles, 2^22+1 at 8 to 16, 2^24+3 and 1.2e8 at 16
        // to 32; fewer than 4 or more than 32 is slower everywhere)
        const int64_t slots = (int64_t)sms * kTableBlocksPerSm;
        tiles_per_block = (n_tiles + slots - 1) / slots;
        if (tiles_per_block > kLowFrameTiles) tiles_per_block = kLowFrameTiles;
        if (tiles_per_block < kWarpsPerBlock / 2) tiles_per_block = kWarpsPerBlock / 2;
    }
    const int grid = (int)((n_tiles + tiles_per_block - 1) / tiles_per_block);
    const int recv_vec = ((uintptr_t)recv_dev & 15u) == 0, send_vec = ((uintptr_t)send_dev & 15u) == 0;
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
    launch.shape = shape;
    memset(&launch.low_states, 0xff, sizeof(launch.low_states));
    if (shape == kShapeWarpsLowFrame) {
        Geometry g;
        g.p = (uint32_t)p;
        g.pm1 = (uint32_t)p - 1u;
        g.q = q;
        low_frame_fill(g, kSharedFrom, launch.low_states.word, (uint32_t)kLowFrameStates);
    }
    launch.grid = grid;
    launch.stream = (cudaStream_t)cuda_stream;
    if (!(launch_table_q_low(launch, q) || launch_table_q_mid(launch, q) || launch_table_q_high(launch, q) ||
          launch_table_q_top(launch, q)))
        return BCAST_EINVAL_P;
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return q;
}

int bcast_set_launch_shape(int shape)
{
    if (shape < BCAST_SHAPE_AUTO || shape > BCAST_SHAPE_WARPS_TIGHT) return BCAST_EINVAL_SHAPE;
    static_assert(BCAST_SHAPE_BLOCK == kShapeBlockPerTile && BCAST_SHAPE_WARPS == kShapeWarps &&
                  BCAST_SHAPE_LOWFRAME == kShapeWarpsLowFrame && BCAST_SHAPE_WARPS_TIGHT == kShapeWarpsTight,
                  "public and internal shape numbers agree");
    forced_shape().store(shape, std::memory_order_relaxed);
    return BCAST_OK;
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

int bcast_store_ceiling(void *buffer_dev, int64_t bytes, int64_t bytes_per_block, void *cuda_stream)
{
    if (buffer_dev == nullptr) return BCAST_ENULL;
    if ((uintptr_t)buffer_dev & 15u) return BCAST_EALIGN;
    if (bytes < 0 || bytes_per_block < 0) return BCAST_EINVAL_N;
    if (bytes_per_block == 0) bytes_per_block = (int64_t)kWarpsPerBlock * kThreads * 27 * 8;   // 8 tiles of both tables at q = 27
    const int64_t n_vec = bytes / 16;
    const int64_t vec_per_block = (bytes_per_block + 15) / 16;
    if (n_vec == 0) return BCAST_OK;
    const int64_t grid = (n_vec + vec_per_block - 1) / vec_per_block;
    if (grid > 0x7fffffff) return BCAST_EINVAL_N;
    store_ceiling_kernel<<<(int)grid, kThreads, 0, (cudaStream_t)cuda_stream>>>(
        reinterpret_cast<int4 *>(buffer_dev), n_vec, vec_per_block);
    if (cudaGetLastError() != cudaSuccess) return BCAST_ECUDA;
    return BCAST_OK;
}

int bcast_low_states(int32_t p, uint32_t *states_host, int32_t capacity)
{
    static_assert(BCAST_LOW_LEVELS == kSharedFrom, "public and internal number of low levels agree");
    if (p < 1) return BCAST_EINVAL_P;
    if (states_host == nullptr) return BCAST_ENULL;
    if (capacity < 0) return BCAST_EINVAL_N;
    const int q = host_q(p);
    if (q < kSharedFrom + 2) return 0;
    Geometry g;
    g.p = (uint32_t)p;
    g.pm1 = (uint32_t)p - 1u;
    g.q = q;
    low_frame_fill(g, kSharedFrom, states_host, (uint32_t)capacity);
    const uint32_t states = skip_of(g, kSharedFrom);
    return (int)(states < (uint32_t)capacity ? states : (uint32_t)capacity);
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

}  // extern "C"
