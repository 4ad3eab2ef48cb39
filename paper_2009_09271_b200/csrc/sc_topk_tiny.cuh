// Top-k of short segments (layer-wise scope: the many small tensors of a network -- biases,
// normalisation parameters, small convolutions), Methodology "Top-k Sparsification" with the
// accumulate and residual lines of Algorithm 1 fused in.
//
// One CTA (up to 4096 elements) or one cluster of eight CTAs (up to 65,535) serves one (worker,
// segment) pair and keeps the whole segment in shared memory:
//   1. p = gamma g + e is computed once and parked in shared memory (12 bytes per element of HBM
//      traffic in total: g and e read once, e' written once);
//   2. a radix select over the 31-bit magnitude keys (8 + 8 + 8 + 7 bits, one shared-memory
//      histogram per pass, runs of equal bins counted in registers before the atomic) yields the exact
//      threshold key T and how many of the elements equal to T are kept;
//   3. an ordered compaction (block scans over 1024 coordinates at a time) writes values and
//      coordinates in ascending order; among equal keys the lowest coordinates win;
//   4. e' = p with the kept entries set to +0.0 goes back to the residual.
// One launch replaces the seven launches (and three histogram round trips through global
// memory) of the multi-pass radix select for these segments.
#pragma once
#include <cooperative_groups.h>

#include "sc_common.cuh"

namespace sc {

struct TinyParams {
    Layout L;
    const float* grads;
    float* residuals;
    float* out_vals;
    uint32_t* out_idx;
    FastState* state;          // [W * nseg]: the path word records who served the segment
    const uint32_t* list;      // segment indices served by this launch
    uint32_t count;            // entries of `list`
    uint32_t W;
    int* status;
};

constexpr uint32_t TINY_CHUNK = THREADS * 4;     // coordinates ranked per block scan
constexpr uint32_t TINY_CTAS = 8;                // CTAs of the cluster that shares a longer segment

// C = 1: one CTA holds the whole segment.  C = TINY_CTAS: a thread-block cluster shares it, CTA r holding
// the r-th contiguous part; the per-pass histograms and the per-part kept counts are read from the peers'
// shared memory (distributed shared memory) between two hardware cluster barriers, and every CTA derives
// the same bin, threshold and offsets from them, so nothing has to be broadcast.
template <uint32_t C>
__global__ void __launch_bounds__(THREADS)
topk_tiny_kernel(TinyParams P) {
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) float s_p[];                       // this CTA's part of the segment's p values
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_scan[WARPS + 1];
    __shared__ uint32_t s_sel[3];
    __shared__ uint32_t s_tot[2];                                      // keys > T and keys == T in this CTA's part
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = C > 1 ? cluster.block_rank() : 0u;
    const Layout& L = P.L;
    const float gamma = L.gamma;
    const uint32_t nclusters = gridDim.x / C;
    for (uint32_t pi = blockIdx.x / C; pi < P.count * P.W; pi += nclusters) {
        const uint32_t w = pi / P.count;
        const uint32_t s = P.list[pi - w * P.count];
        const SegEntry seg = L.segs[s];
        const uint32_t n_seg = seg.n, k = seg.k;
        // this CTA's part [lo, lo + n) of the segment
        const uint32_t per = ((n_seg + C - 1) / C + 3u) & ~3u;
        const uint32_t lo = min(rank * per, n_seg), n = min(per, n_seg - lo);
        const size_t row = (size_t)w * L.n_total + seg.offset + lo;
        const float* g = P.grads + row;
        float* e = P.residuals + row;
        __syncthreads();                                               // the previous segment is done with shared memory
        for (uint32_t i = threadIdx.x; i < n; i += THREADS) s_p[i] = accumulate(gamma, __ldcs(g + i), e[i]);
        if (rank == 0 && threadIdx.x == 0) P.state[(size_t)w * L.nseg + s].path = PATH_TINY;
        __syncthreads();
        if (k > 0) {
            // ---- radix select: after the last pass `prefix` is the k-th largest key ----------------------
            uint32_t prefix = 0, mask = 0, need = k, ties = 0;
#pragma unroll 1
            for (int pass = 0; pass < 4; ++pass) {
                const uint32_t shift = pass == 0 ? 23u : pass == 1 ? 15u : pass == 2 ? 7u : 0u;
                const uint32_t field = pass == 3 ? 0x7Fu : 0xFFu;
                s_hist[threadIdx.x] = 0;
                __syncthreads();
                // a thread counts runs of equal bins among its own elements before it touches the histogram:
                // in the first passes nearly all keys of a segment share their leading bits
                {
                    uint32_t run_bin = 0xFFFFFFFFu, run_cnt = 0;
                    for (uint32_t i = threadIdx.x; i < n; i += THREADS) {
                        const uint32_t key = key_of(s_p[i]);
                        if ((key & mask) != prefix) continue;
                        const uint32_t bin = (key >> shift) & field;
                        if (bin == run_bin) { ++run_cnt; continue; }
                        if (run_cnt) atomicAdd(&s_hist[run_bin], run_cnt);
                        run_bin = bin; run_cnt = 1;
                    }
                    if (run_cnt) atomicAdd(&s_hist[run_bin], run_cnt);
                }
                if constexpr (C > 1) cluster.sync(); else __syncthreads();
                // walk the bins from the top: thread t looks at bin 255 - t (summed over the cluster)
                uint32_t v = 0;
                if constexpr (C > 1) {
                    for (uint32_t r = 0; r < C; ++r) v += cluster.map_shared_rank(s_hist, r)[255u - threadIdx.x];
                } else {
                    v = s_hist[255u - threadIdx.x];
                }
                uint32_t total;
                const uint32_t before = block_exclusive_scan(v, s_scan, &total);
                if (before < need && need <= before + v) {
                    s_sel[0] = 255u - threadIdx.x; s_sel[1] = need - before; s_sel[2] = v;
                }
                if constexpr (C > 1) cluster.sync(); else __syncthreads();   // peers have read this histogram
                prefix |= s_sel[0] << shift;
                mask |= field << shift;
                need = s_sel[1];
                ties = s_sel[2];
                __syncthreads();
            }
            const uint32_t T = prefix;                                 // elements with key == T: `ties`, of which `need` are kept
            const bool rank_ties = need < ties;                        // otherwise every element equal to T is kept
            // ---- kept and equal elements in the parts before this one -----------------------------------
            uint32_t kept_before = 0, eq_before = 0;
            if constexpr (C > 1) {
                uint32_t gt = 0, eq = 0;
                for (uint32_t i = threadIdx.x; i < n; i += THREADS) {
                    const uint32_t key = key_of(s_p[i]);
                    gt += key > T ? 1u : 0u;
                    eq += key == T ? 1u : 0u;
                }
                uint32_t tg, te;
                block_exclusive_scan(gt, s_scan, &tg);
                block_exclusive_scan(eq, s_scan, &te);
                if (threadIdx.x == 0) { s_tot[0] = tg; s_tot[1] = te; }
                cluster.sync();
                for (uint32_t r = 0; r < rank; ++r) {
                    const uint32_t* t = cluster.map_shared_rank(s_tot, r);
                    const uint32_t g_r = t[0], e_r = t[1];
                    const uint32_t room = need > eq_before ? need - eq_before : 0u;     // equal keys still to be kept
                    kept_before += g_r + min(e_r, room);
                    eq_before += e_r;
                }
            }
            // ---- ordered compaction: thread t ranks coordinates base + 4 t .. base + 4 t + 3 ---------------
            float* ovals = P.out_vals + (size_t)w * L.K_total + seg.msg_off;
            uint32_t* oidx = P.out_idx + (size_t)w * L.K_total + seg.msg_off;
            const uint32_t idx0 = (uint32_t)seg.offset + lo;
            for (uint32_t base = 0; base < n; base += TINY_CHUNK) {
                const uint32_t i0 = base + threadIdx.x * 4u;
                uint32_t gt = 0, eq = 0;                               // bit c: element i0 + c
#pragma unroll
                for (uint32_t c = 0; c < 4; ++c) {
                    if (i0 + c < n) {
                        const uint32_t key = key_of(s_p[i0 + c]);
                        gt |= (key > T ? 1u : 0u) << c;
                        eq |= (key == T ? 1u : 0u) << c;
                    }
                }
                uint32_t keep = gt | eq, total;
                if (rank_ties) {                                       // only the first `need` of the equal keys are kept
                    uint32_t r = eq_before + block_exclusive_scan((uint32_t)__popc(eq), s_scan, &total);
                    eq_before += total;
                    keep = gt;
#pragma unroll
                    for (uint32_t c = 0; c < 4; ++c)
                        if ((eq >> c) & 1u) { if (r < need) keep |= 1u << c; ++r; }
                }
                uint32_t pos = kept_before + block_exclusive_scan((uint32_t)__popc(keep), s_scan, &total);
                kept_before += total;
#pragma unroll
                for (uint32_t c = 0; c < 4; ++c) {
                    if (((keep >> c) & 1u) && pos < k) {
                        ovals[pos] = s_p[i0 + c];
                        oidx[pos] = idx0 + i0 + c;
                        s_p[i0 + c] = 0.0f;                            // e' = p - q^w: kept entries become +0.0
                        ++pos;
                    }
                }
            }
            if (rank == C - 1 && threadIdx.x == 0 && kept_before != k) atomicMin(P.status, ST_DEVICE_CHECK);   // counts and k disagree
            __syncthreads();
        }
        for (uint32_t i = threadIdx.x; i < n; i += THREADS) e[i] = s_p[i];
        if constexpr (C > 1) cluster.sync();                           // peers may still read this CTA's totals
    }
}

}  // namespace sc
