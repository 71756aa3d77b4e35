// Weight prefetch into the L2 from the kernels that run BETWEEN two projections.
//
// While a normalisation, rotation, gating or attention kernel runs, the HBM is nearly idle, and the projection that
// follows can keep only a few tiles per SM in flight before its own dependency wait.  Those in-between kernels
// therefore ask the L2 for the first weight tiles of the next projection: every thread issues a few L2 prefetches
// before it waits for its own predecessor (weights never depend on a predecessor).  A prefetch moves no data into
// the SM and cannot change a result; a line that has been evicted again by the time it is wanted costs nothing but
// the read it would have cost anyway.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_tc.h"

namespace medusa {

// For every CTA c of the next projection launch (c < G): the first `units` (tile, k block) pairs of its range, each
// a 128-row x 128-byte box of its weight matrix, one prefetch per row.
__device__ __forceinline__ void prefetch_weights(const WeightPrefetch &p, long long tid, long long n_threads)
{
    if (p.units <= 0)
        return;
    const long long items = (long long)p.G * p.units * 128;
    for (long long i = tid; i < items; i += n_threads) {
        const int r = (int)(i & 127);
        const int cu = (int)(i >> 7);
        const int c = cu / p.units, j = cu - c * p.units;
        long long x0, x1;
        if (p.whole_tiles) {  // CTA c owns tiles c, c + G, ...: its first tile
            x0 = (long long)c * p.KB;
            x1 = x0 + p.KB;
        } else {
            x0 = ((long long)c * p.total) / p.G;
            x1 = ((long long)(c + 1) * p.total) / p.G;
        }
        const long long x = x0 + j;
        if (x >= x1 || x >= p.total)
            continue;
        const int tile = (int)(x / p.KB), kb = (int)(x - (long long)tile * p.KB);
        const int rest = tile - p.seg0_tiles;
        const int seg = rest < 0 ? 0 : 1 + rest / p.seg_tiles;
        const int row = (rest < 0 ? tile : rest % p.seg_tiles) * 128 + r;
        if (row >= (seg == 0 ? p.seg0_rows : p.seg_rows))
            continue;
        const char *addr = (const char *)p.W[seg] + ((size_t)row * p.K + (size_t)kb * 64) * 2;
        asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(addr));
    }
}

}  // namespace medusa
