// Fall-back of the one-pass top-k (Methodology, "Top-k Sparsification"): segments whose sampled
// bracket missed, or whose lists overflowed, are selected again by an exact multi-pass radix
// select on p = gamma g + e, which the streaming pass has parked in the residual buffer.
//
// ONE persistent kernel per top-k call, launched cooperatively (all its CTAs are resident), which
// returns in its first instructions unless some segment failed.  (It also hosts the rare second half
// of the emit step, the tiles that admit tie-key elements, so that the emit kernel proper keeps its
// registers for the common case.)  Its phases are separated by
// grid-wide barriers:
//   A  put back the values the streaming pass had zeroed, clear the failed segments' histograms
//   B  histogram of key bits 30..20         C  bucket of the k-th key
//   D  histogram of bits 19..10             E  bucket
//   F  histogram of bits 9..0               G  threshold key T and number of ties kept
//   H  ordered pack (chained scan over groups of tiles) and residual writeback
// The grid barrier counts arrivals in one global word; a CTA that has waited poll_limit polls gives
// up, records ST_TIMEOUT in the status word and leaves the kernel (so do, in turn, the others).
#pragma once
#include "sc_pack.cuh"
#include "sc_topk.cuh"
#include "sc_topk_fast.cuh"

namespace sc {

constexpr uint32_t BARRIER_POLL_LIMIT = 1u << 24;      // about 64 ns each: a second at the very least

struct FallbackParams {
    FastParams F;
    PackParams K;
    uint32_t* hist;                // [W * nseg][HIST_WORDS]
    TopkState* rstate;             // [W * nseg]
    WorkList tiles;                // tiles of the large segments, the same list for every worker
    uint32_t W;
    uint32_t poll_limit;           // of the grid barrier
    unsigned int* barrier;         // arrivals so far (zeroed before the launch)
};

// All CTAs of a cooperative launch meet here.  Returns false when the wait ran out.
__device__ inline bool grid_barrier(unsigned int* counter, unsigned int& target, uint32_t limit, int* status) {
    __shared__ int s_ok;
    target += gridDim.x;
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        __threadfence();
        atomicAdd(counter, 1u);
        uint32_t polls = 0;
        while (*reinterpret_cast<volatile unsigned int*>(counter) < target) {
            if (++polls > limit) { atomicMin(status, ST_TIMEOUT); ok = 0; break; }
            __nanosleep(64);
        }
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0;
}

__global__ void __launch_bounds__(THREADS)
topk_fallback_kernel(const __grid_constant__ FallbackParams P) {
    if (__ldcg(P.F.counters + 1) != 0u) emit_tie_tiles(P.F);          // some segment's threshold is its tie key
    if (__ldcg(P.F.counters) == 0u) return;                            // no segment failed: the usual case
    const Layout& L = P.F.L;
    const uint32_t nprob = P.W * L.nseg;
    const uint32_t items = P.W * P.tiles.len;
    unsigned int target = 0;
    // ---- A
    restore_failed_segments(P.F);
    for (uint32_t prob = blockIdx.x; prob < nprob; prob += gridDim.x) {
        if (__ldcg(&P.F.state[prob].path) != PATH_FAILED) continue;
        for (uint32_t b = threadIdx.x; b < HIST_WORDS; b += THREADS) P.hist[(size_t)prob * HIST_WORDS + b] = 0u;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) *P.K.ticket = 0ull;
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    // ---- B .. G
    radix_histogram<0>(L, P.F.residuals, P.hist, P.rstate, P.F.state, P.tiles, items);
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    radix_resolve<0>(L, P.hist, P.rstate, P.F.state, nprob, P.F.status);
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    radix_histogram<1>(L, P.F.residuals, P.hist, P.rstate, P.F.state, P.tiles, items);
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    radix_resolve<1>(L, P.hist, P.rstate, P.F.state, nprob, P.F.status);
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    radix_histogram<2>(L, P.F.residuals, P.hist, P.rstate, P.F.state, P.tiles, items);
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    radix_resolve<2>(L, P.hist, P.rstate, P.F.state, nprob, P.F.status);
    if (!grid_barrier(P.barrier, target, P.poll_limit, P.F.status)) return;
    // ---- H
    pack_failed_segments(P.K);
}

// Instrumentation: runs the two bounded waits of the fall-back kernel in a situation where what they
// wait for never comes (a barrier that expects one arrival more than the grid has CTAs; a look-back on
// a descriptor that nobody publishes), with a short limit.  Both must give up, record ST_TIMEOUT and
// return.
__global__ void __launch_bounds__(THREADS)
wait_probe_kernel(const __grid_constant__ PackParams K, unsigned int* barrier, uint32_t limit, int which) {
    if (which == 0) {
        unsigned int target = 1;                                       // gridDim.x + 1 arrivals expected
        grid_barrier(barrier, target, limit, K.status);
    } else if (threadIdx.x < 32) {
        uint32_t ex0 = 0, ex1 = 0;
        lookback(K, 1u, 0u, false, ex0, ex1);                          // descriptor 0 carries an old tag for ever
    }
}

}  // namespace sc
