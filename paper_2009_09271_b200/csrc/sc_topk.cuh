// Fall-back top-k threshold search: a three-level radix select on the bit pattern of |p|
// (Methodology, "Top-k Sparsification"), for segments whose sampled bracket missed.  The streaming
// pass has already parked p = gamma g + e in the residual buffer.
//
// The k-th largest key and the number of ties to admit are found exactly:
//   level 0  histogram of key bits 30..20 over the whole segment,
//   level 1  histogram of bits 19..10 over the elements that share the level-0 bucket,
//   level 2  histogram of bits 9..0 over the elements that share the level-1 bucket.
// After each level one CTA per (worker, segment) walks the histogram from the top and
// narrows (prefix, need).  A level is skipped as soon as the whole bucket is taken.
// These are the phases of ONE kernel (sc_topk_fallback.cuh), separated by grid-wide barriers.
#pragma once
#include "sc_common.cuh"

namespace sc {

// flush a CTA-private histogram into the global one of a problem and clear it
template <uint32_t BINS>
__device__ inline void flush_hist(uint32_t* sh, uint32_t* __restrict__ gh) {
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < BINS; b += THREADS) {
        uint32_t c = sh[b];
        if (c) { atomicAdd(gh + b, c); sh[b] = 0; }
    }
    __syncthreads();
}

// Histogram of one level over the tiles of the failed segments.  LEVEL 0: bits 30..20 of every key;
// LEVEL 1, 2: the next ten bits of the keys whose higher bits equal the prefix found so far.
template <int LEVEL>
__device__ inline void radix_histogram(const Layout& L, const float* __restrict__ residuals, uint32_t* __restrict__ hist,
                                       const TopkState* __restrict__ state, const FastState* __restrict__ fstate,
                                       const WorkList& wl, uint32_t total_items) {
    constexpr uint32_t BINS = (LEVEL == 0) ? HIST0_BINS : 1024u;
    constexpr uint32_t SHIFT = (LEVEL == 0) ? 20u : (LEVEL == 1) ? 10u : 0u;
    constexpr uint32_t HOFF = (LEVEL == 0) ? 0u : (LEVEL == 1) ? HIST0_BINS : HIST0_BINS + HIST1_BINS;
    __shared__ uint32_t sh[BINS];
    __shared__ uint32_t s_dec[4];
    for (uint32_t b = threadIdx.x; b < BINS; b += THREADS) sh[b] = 0;
    __syncthreads();
    long long cur_prob = -1;
    for (uint32_t item = blockIdx.x; item < total_items; item += gridDim.x) {
        if (threadIdx.x == 0) {
            const uint32_t w = item / wl.len;
            const uint32_t lt = wl.ids[item - w * wl.len];
            const uint32_t s = find_by_tile(L, lt);
            const size_t prob = (size_t)w * L.nseg + s;
            s_dec[0] = w; s_dec[1] = s; s_dec[2] = lt - L.segs[s].tile_begin;
            s_dec[3] = (__ldcg(&fstate[prob].path) == PATH_FAILED && (LEVEL == 0 || __ldcg(&state[prob].active))) ? 1u : 0u;
        }
        __syncthreads();
        const uint32_t w = s_dec[0], s = s_dec[1], t = s_dec[2], live = s_dec[3];
        if (live) {                                                      // uniform over the CTA
            const long long prob = (long long)w * L.nseg + s;
            if (prob != cur_prob) {
                if (cur_prob >= 0) flush_hist<BINS>(sh, hist + (size_t)cur_prob * HIST_WORDS + HOFF);
                cur_prob = prob;
            }
            const SegEntry seg = L.segs[s];
            const float* e = residuals + (size_t)w * L.n_total + seg.offset;
            const uint32_t mis = misalign_of(e);
            const uint32_t want = LEVEL == 0 ? 0u : (__ldcg(&state[prob].prefix) >> (SHIFT + 10u));
            uint32_t run_bin = 0xFFFFFFFFu, run_cnt = 0;
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const long long base = (long long)t * TILE + (long long)(j * THREADS + threadIdx.x) * 4 - mis;
                float p[4];
                const uint32_t m = load_quad(e, base, seg.n, p);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t key = key_of(p[c]);
                    if (((m >> c) & 1u) && (LEVEL == 0 || (key >> (SHIFT + 10u)) == want)) {
                        const uint32_t bin = LEVEL == 0 ? key >> 20 : (key >> SHIFT) & 1023u;
                        if (bin == run_bin) ++run_cnt;
                        else {
                            if (run_cnt) atomicAdd(&sh[run_bin], run_cnt);
                            run_bin = bin; run_cnt = 1;
                        }
                    }
                }
            }
            if (run_cnt) atomicAdd(&sh[run_bin], run_cnt);
        }
        __syncthreads();   // s_dec is rewritten by the next iteration
    }
    if (cur_prob >= 0) flush_hist<BINS>(sh, hist + (size_t)cur_prob * HIST_WORDS + HOFF);
}

// One CTA per failed (worker, segment): walk the level's histogram from the highest bin
// down to the bucket that holds the need-th largest key.
template <int LEVEL>
__device__ inline void radix_resolve(const Layout& L, const uint32_t* __restrict__ hist, TopkState* __restrict__ state,
                                     const FastState* __restrict__ fstate, uint32_t nprob, int* __restrict__ status) {
    constexpr uint32_t BINS = (LEVEL == 0) ? HIST0_BINS : 1024u;
    constexpr uint32_t SHIFT = (LEVEL == 0) ? 20u : (LEVEL == 1) ? 10u : 0u;
    constexpr uint32_t HOFF = (LEVEL == 0) ? 0u : (LEVEL == 1) ? HIST0_BINS : HIST0_BINS + HIST1_BINS;
    constexpr uint32_t BPT = BINS / THREADS;
    __shared__ uint32_t scan_smem[WARPS + 1];
    __shared__ uint32_t s_found;
    for (uint32_t prob = blockIdx.x; prob < nprob; prob += gridDim.x) {
        const uint32_t s = prob % L.nseg;
        if (__ldcg(&fstate[prob].path) != PATH_FAILED) continue;       // uniform over the CTA
        uint32_t need, prefix;
        if (LEVEL == 0) {
            need = L.segs[s].k;
            prefix = 0;
            if (need == 0) {                       // nothing kept: no key reaches the threshold
                if (threadIdx.x == 0) {
                    TopkState st = {0u, 0u, 0u, 0xFFFFFFFFu, 0u, 0u, 0u, 0u};
                    state[prob] = st;
                }
                continue;
            }
        } else {
            if (!__ldcg(&state[prob].active)) continue;
            need = __ldcg(&state[prob].need);
            prefix = __ldcg(&state[prob].prefix);
        }
        __syncthreads();
        if (threadIdx.x == 0) s_found = 0;
        const uint32_t* h = hist + (size_t)prob * HIST_WORDS + HOFF;
        uint32_t local[BPT];
        uint32_t sum = 0;
#pragma unroll
        for (uint32_t c = 0; c < BPT; ++c) {       // thread i owns bins BINS-1-i*BPT-c, descending
            local[c] = __ldcg(h + BINS - 1u - (threadIdx.x * BPT + c));
            sum += local[c];
        }
        uint32_t total;
        uint32_t before = block_exclusive_scan(sum, scan_smem, &total);   // has a barrier after s_found = 0
        if (before < need && need <= before + sum) {
            uint32_t acc = before;
#pragma unroll
            for (uint32_t c = 0; c < BPT; ++c) {
                if (need <= acc + local[c]) {
                    const uint32_t bin = BINS - 1u - (threadIdx.x * BPT + c);
                    const uint32_t take = need - acc;          // elements of this bucket that are kept
                    const uint32_t cnt = local[c];
                    TopkState st;
                    st.prefix = prefix | (bin << SHIFT);
                    st.need = take;
                    st.pad0 = st.pad1 = 0;
                    if (take == cnt) {                         // the whole bucket is kept
                        st.active = 0; st.T = st.prefix; st.r = cnt; st.dual = 0;
                    } else if (LEVEL == 2) {                   // bucket == one key value: ties
                        st.active = 0; st.T = st.prefix; st.r = take; st.dual = 1;
                    } else {
                        st.active = 1; st.T = 0; st.r = 0; st.dual = 0;
                    }
                    state[prob] = st;
                    s_found = 1;
                    break;
                }
                acc += local[c];
            }
        }
        __syncthreads();
        if (threadIdx.x == 0 && !s_found) {        // histogram inconsistent with need: report, keep nothing
            TopkState st = {0u, 0u, 0u, 0xFFFFFFFFu, 0u, 0u, 0u, 0u};
            state[prob] = st;
            atomicMin(status, ST_DEVICE_CHECK);
        }
    }
}

}  // namespace sc
