// Verification sweep (see include/bcast_sched.h): persistent blocks pull values of p from a
// queue, build the tables of one p in scratch memory with the table kernel's device
// functions, then check the paper's correctness conditions against them and reduce a checksum.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/bcast_sched.h"
#include "host_util.h"
#include "schedule_tile.cuh"

namespace bcast {

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
            __syncthreads();                               // every thread has read the queue's counters before the reset
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

static int64_t sweep_bytes_per_block(int32_t p_hi)
{
    return round_up((int64_t)2 * host_q(p_hi) * ((int64_t)p_hi + 1), 256);
}

constexpr int64_t kSweepHeaderBytes = 256;             // the work-queue counter lives here

}  // namespace bcast

using namespace bcast;

extern "C" {

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
