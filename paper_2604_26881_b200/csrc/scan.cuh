// Block-wide exclusive scan in shared memory, used by the dispatch and plan kernels.
#pragma once

#include <stdint.h>

namespace faasmoe {

// Exclusive scan of data[0..n) (shared memory) by the whole block; every thread owns a contiguous
// run of entries, the per-thread sums are scanned with warp shuffles.  s_warp needs 33 entries.
// Returns the total.  Ends with a block barrier.
__device__ __forceinline__ int block_scan_exclusive(int32_t* data, int n, int32_t* s_warp)
{
    const int tid = threadIdx.x, nth = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = (nth + 31) >> 5;
    const int per = (n + nth - 1) / nth;
    const int b0 = min(n, tid * per), b1 = min(n, b0 + per);
    int sum = 0;
    for (int b = b0; b < b1; ++b) sum += data[b];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = lane < nw ? s_warp[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += v;
        }
        s_warp[lane] = wi - w;              // exclusive prefix of the warp totals
        if (lane == 31) s_warp[32] = wi;    // grand total
    }
    __syncthreads();
    int run = s_warp[warp] + incl - sum;
    for (int b = b0; b < b1; ++b) { const int c = data[b]; data[b] = run; run += c; }
    const int total = s_warp[32];
    __syncthreads();
    return total;
}

}  // namespace faasmoe
