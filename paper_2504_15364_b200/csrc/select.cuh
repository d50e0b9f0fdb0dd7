// Block-level exact top-N selection over orderable u32 keys held in shared memory, and the
// ordered compaction plan that follows it.  Used by the staged select kernel and by the fused
// cluster kernel.
//
// Total order (paper silent on ties; the reading used everywhere in this library):
//   key descending, token index ascending -- among equal scores the older token is kept.
#pragma once
#include "common.cuh"

namespace kd {

struct Threshold {
    uint32_t key;   // key of the N-th ranked token
    int need_eq;    // how many tokens with key == threshold are kept (the oldest ones), >= 1
};

struct SelectSmem {
    int hist[256];
    int warp_gt[32];
    int warp_eq[32];
    int bcast[2];
    int first_evicted;
};

// MSB-first radix select, 4 passes of 8 bits.  Histogram updates are aggregated per warp with
// match_any so that heavily tied inputs (all scores equal) cost one atomic per warp, not one
// per key.  Requires 1 <= N <= n.  All threads of the block must call; result is uniform.
template <int THREADS>
__device__ Threshold block_radix_select(const uint32_t* __restrict__ keys, int n, int N, SelectSmem& sm) {
    const int tid = threadIdx.x, lane = tid & 31;
    uint32_t prefix = 0, mask = 0;
    int want = N;   // rank (1 = largest) of the wanted key among keys matching the prefix
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int b = tid; b < 256; b += THREADS) sm.hist[b] = 0;
        __syncthreads();
        for (int base = 0; base < n; base += THREADS) {
            const int i = base + tid;
            uint32_t k = 0;
            bool valid = false;
            if (i < n) { k = keys[i]; valid = (k & mask) == prefix; }
            const unsigned active = __ballot_sync(0xffffffffu, valid);
            if (valid) {
                const int digit = (k >> shift) & 0xff;
                const unsigned peers = __match_any_sync(active, digit);
                if (lane == __ffs(peers) - 1) atomicAdd(&sm.hist[digit], __popc(peers));
            }
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns bins 255-8l .. 248-8l (descending); find the bin holding rank `want`
            int c[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = sm.hist[255 - 8 * lane - j]; tot += c[j]; }
            int incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const int excl = incl - tot;
            if (excl < want && want <= incl) {
                int above = excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (above < want && want <= above + c[j]) {
                        sm.bcast[0] = 255 - 8 * lane - j;
                        sm.bcast[1] = want - above;
                    }
                    above += c[j];
                }
            }
        }
        __syncthreads();
        prefix |= static_cast<uint32_t>(sm.bcast[0]) << shift;
        mask |= 0xffu << shift;
        want = sm.bcast[1];
    }
    return Threshold{prefix, want};
}

// Exclusive block scan of two counters per thread.  Returns this thread's exclusive prefixes;
// the block totals are returned through tot_gt/tot_eq.
template <int THREADS>
__device__ void block_exclusive_scan2(int gt, int eq, SelectSmem& sm, int& pre_gt, int& pre_eq,
                                      int& tot_gt, int& tot_eq) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int igt = gt, ieq = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, igt, o);
        const int b = __shfl_up_sync(0xffffffffu, ieq, o);
        if (lane >= o) { igt += a; ieq += b; }
    }
    if (lane == 31) { sm.warp_gt[warp] = igt; sm.warp_eq[warp] = ieq; }
    __syncthreads();
    if (warp == 0) {
        constexpr int W = THREADS / 32;
        int a = lane < W ? sm.warp_gt[lane] : 0, b = lane < W ? sm.warp_eq[lane] : 0;
        int ia = a, ib = b;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xffffffffu, ia, o);
            const int y = __shfl_up_sync(0xffffffffu, ib, o);
            if (lane >= o) { ia += x; ib += y; }
        }
        if (lane < W) { sm.warp_gt[lane] = ia - a; sm.warp_eq[lane] = ib - b; }
        if (lane == 31) { sm.bcast[0] = ia; sm.bcast[1] = ib; }
    }
    __syncthreads();
    pre_gt = sm.warp_gt[warp] + igt - gt;
    pre_eq = sm.warp_eq[warp] + ieq - eq;
    tot_gt = sm.bcast[0];
    tot_eq = sm.bcast[1];
}

}  // namespace kd
