// Host-side helpers shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "schedule_fast.cuh"

namespace bcast {

inline int host_q(int64_t p)
{
    int q = 0;
    while (((int64_t)1 << q) < p) ++q;
    return q;
}

inline int sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    return sms;
}

// Algorithm 2 and the prefix sums of the skips.
inline LevelTables host_tables(int64_t p, int q)
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

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

}  // namespace bcast
