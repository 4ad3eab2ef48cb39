// Top-k of a large segment in ONE pass over g and e (Methodology, "Top-k Sparsification";
// Algorithm 1 accumulate / compress / residual lines).
//
// A radix select has to see every key before it knows the threshold, which costs extra
// passes over HBM.  Here a small systematic sample of |g + e| brackets the threshold first:
//   sample   m keys per (worker, segment); two order statistics of the sample, six standard
//            deviations either side of rank k m / n, give [lo, hi] with
//            count(key > hi) <= k <= count(key >= lo) except with negligible probability;
//   main     the streaming pass forms p = g + e and writes the residual at once: 0 for the
//            "sure" elements (key > hi), p for the rest.  Every element with key >= lo is
//            appended, in coordinate order inside its tile, to a "flagged" list (value,
//            coordinate); the few candidates (lo <= key <= hi) also go to a candidate list
//            and into a 2048-bin histogram;
//   resolve  the candidate histogram pins the bin of the k-th key, the candidates of that
//            bin are sorted in shared memory: exact threshold T and the coordinate cut for
//            ties.  Every count is exact, so the result equals the plain definition; the
//            sample only decides how much work that takes.  If the bracket is wrong (counts
//            prove it) or a list overflows, the segment falls back to the radix select on
//            the parked p;
//   emit     per-tile kept counts -> exclusive scan -> a pass over the flagged list only:
//            kept entries go to the message in ascending coordinate order, kept candidates
//            are zeroed in the residual.  On a fall-back the sure values are first written
//            back from the flagged list.
// No CTA polls for another anywhere on this path; the bracket and the row scan use thread-block
// clusters, whose CTAs meet at hardware cluster barriers only.
#pragma once
#include <cooperative_groups.h>

#include "sc_common.cuh"

namespace sc {

struct FastParams {
    Layout L;
    const float* grads;
    float* residuals;
    float* out_vals;
    uint32_t* out_idx;
    FastState* state;          // [W * nseg]
    uint32_t* sample;          // [W][sample_per_worker]
    uint32_t* cand_hist;       // [W * fast_per_worker][CAND_BINS]
    uint2* list2;              // [W * fast_per_worker][LIST2_CAP]
    uint2* flagged;            // [W][flag_per_worker] (value bits, coordinate inside the segment)
    uint2* cand;               // [W][cand_per_worker] (key, coordinate) of the candidates, any order inside a tile
    uint32_t* tile_sure;       // [W * tiles_per_worker] sure elements of the tile (zeroed before the pass)
    uint32_t* tile_cbase;      // first candidate slot of the tile
    uint32_t* tile_ccnt;       // candidates of the tile
    uint32_t* tile_csum;       // candidates above the threshold's bin (low half) and inside it (high half)
    uint32_t* tile_fbase;      // first flagged slot of the tile (0xFFFFFFFF: the list was full, nothing written)
    uint32_t* tile_fcnt;       // flagged elements of the tile
    uint32_t* n_failed;        // segments whose bracket missed
    uint32_t* offsets;         // [W][tiles_per_worker + 1]
    uint32_t* n_slow;          // segments that need the radix-select path
    int* status;
    uint32_t total_items;
};

// The per-segment kernels of this path are launched over the fast segments only: block index
// f = w * fast_per_worker + fast_index, mapped to the segment through the layout's fast list.
__device__ inline uint32_t fast_problem(const Layout& L, uint32_t f, uint32_t& w, uint32_t& s) {
    w = f / L.fast_per_worker;
    s = L.fast_list[f - w * L.fast_per_worker];
    return w * L.nseg + s;
}

// ---- shared helper: walk a histogram from its highest bin down to the bin that holds the
// need-th largest element.  All THREADS threads call it; results are uniform.
template <uint32_t BINS, typename HistPtr>
__device__ inline bool find_from_top(HistPtr h, uint32_t need, uint32_t* s_tmp /*WARPS+4*/, uint32_t& bin,
                                     uint32_t& need_in, uint32_t& cnt) {
    constexpr uint32_t BPT = BINS / THREADS;
    uint32_t local[BPT], sum = 0;
#pragma unroll
    for (uint32_t c = 0; c < BPT; ++c) {
        local[c] = h[BINS - 1u - (threadIdx.x * BPT + c)];
        sum += local[c];
    }
    if (threadIdx.x == 0) s_tmp[WARPS + 1] = 0xFFFFFFFFu;
    uint32_t total;
    const uint32_t before = block_exclusive_scan(sum, s_tmp, &total);
    if (need >= 1 && before < need && need <= before + sum) {
        uint32_t acc = before;
#pragma unroll
        for (uint32_t c = 0; c < BPT; ++c) {
            if (need <= acc + local[c]) {
                s_tmp[WARPS + 1] = BINS - 1u - (threadIdx.x * BPT + c);
                s_tmp[WARPS + 2] = need - acc;
                s_tmp[WARPS + 3] = local[c];
                break;
            }
            acc += local[c];
        }
    }
    __syncthreads();
    bin = s_tmp[WARPS + 1]; need_in = s_tmp[WARPS + 2]; cnt = s_tmp[WARPS + 3];
    __syncthreads();
    return bin != 0xFFFFFFFFu;
}

// ---- sample: one 32-byte sector (8 elements) of g and e per thread ----------------------
__global__ void __launch_bounds__(THREADS)
topk_sample_kernel(FastParams P) {
    const Layout& L = P.L;
    const uint32_t w = blockIdx.y;
    const uint64_t pos = ((uint64_t)blockIdx.x * THREADS + threadIdx.x) * 8u;   // first key of this thread's sector
    if (pos >= L.sample_per_worker) return;
    // the samples of a worker's large segments lie one after the other, in fast-list order: find the segment
    uint32_t f0 = 0, f1 = L.fast_per_worker - 1u;
    while (f0 < f1) {
        const uint32_t mid = (f0 + f1 + 1u) >> 1;
        if (L.segs[L.fast_list[mid]].sample_begin <= pos) f0 = mid; else f1 = mid - 1u;
    }
    const SegEntry seg = L.segs[L.fast_list[f0]];
    const uint32_t c = (uint32_t)((pos - seg.sample_begin) / 8u);      // sector of the segment's sample
    const size_t row = (size_t)w * L.n_total + seg.offset;
    const float* g = P.grads + row;
    const float* e = P.residuals + row;
    const uint32_t a0 = (8u - (uint32_t)((reinterpret_cast<uintptr_t>(e) >> 2) & 7u)) & 7u;   // first 32B-aligned element
    const uint32_t sectors = (seg.n - a0) / 8u;
    const uint32_t sidx = (uint32_t)(((uint64_t)c * sectors) / (seg.sample_m / 8u));
    const size_t at = (size_t)a0 + (size_t)sidx * 8u;
    const float4 e0 = *reinterpret_cast<const float4*>(e + at), e1 = *reinterpret_cast<const float4*>(e + at + 4);
    const float4 g0 = *reinterpret_cast<const float4*>(g + at), g1 = *reinterpret_cast<const float4*>(g + at + 4);
    uint4 k0, k1;
    const float4 p0 = accumulate(L.gamma, g0, e0), p1 = accumulate(L.gamma, g1, e1);
    k0.x = key_of(p0.x); k0.y = key_of(p0.y); k0.z = key_of(p0.z); k0.w = key_of(p0.w);
    k1.x = key_of(p1.x); k1.y = key_of(p1.y); k1.z = key_of(p1.z); k1.w = key_of(p1.w);
    uint4* out = reinterpret_cast<uint4*>(P.sample + (size_t)w * L.sample_per_worker + seg.sample_begin + (size_t)c * 8u);
    out[0] = k0; out[1] = k1;
}

// ---- bracket: two order statistics of the sample, to 21 bits -----------------------------------
// One thread-block cluster of BRACKET_CTAS CTAs per problem: every CTA histograms its share of the
// sample in its own shared memory, CTA 0 adds the shares up through distributed shared memory, walks
// the total and hands the two bins back the same way; a second round refines them by ten more bits.
// The cluster barriers are the hardware's; no CTA leaves before the last one (a peer's shared memory
// must stay alive while it is read).
// Segments with a small sample take one CTA each (C = 1: no cluster calls at all).  `first` and `count`
// select a range of the fast list; the grid covers count problems of every worker.
constexpr uint32_t BRACKET_CTAS = 8;
constexpr uint32_t BRACKET_BIG_SAMPLE = 1u << 15;                      // samples from this size up take a cluster
template <uint32_t C>
__global__ void __launch_bounds__(THREADS)
topk_bracket_kernel(FastParams P, uint32_t first, uint32_t count) {
    namespace cg = cooperative_groups;
    __shared__ uint32_t h0[HIST0_BINS];
    __shared__ uint32_t hA[1024], hB[1024];
    __shared__ uint32_t s_tmp[WARPS + 4];
    __shared__ uint32_t s_bins[4];                                     // binA, binB, needA, needB (valid in CTA 0)
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = C > 1 ? cluster.block_rank() : 0u;
    const Layout& L = P.L;
    uint32_t w, s;
    const uint32_t pidx = blockIdx.x / C;                              // problem of this launch: (worker, position in the range)
    const uint32_t prob = fast_problem(L, (pidx / count) * L.fast_per_worker + first + pidx % count, w, s);
    const SegEntry seg = L.segs[s];
    const uint32_t m = seg.sample_m;
    const uint4* smp = reinterpret_cast<const uint4*>(P.sample + (size_t)w * L.sample_per_worker + seg.sample_begin);
    // this CTA's share of the sample (in groups of four keys)
    const uint32_t per = (m / 4u + C - 1u) / C;
    const uint32_t i_begin = min(rank * per, m / 4u), i_end = min(i_begin + per, m / 4u);
    // ranks (from the top) that bracket the k-th largest of the segment
    const double q = (double)seg.k / (double)seg.n;
    const double centre = q * (double)m;
    const double delta = 6.0 * sqrt((double)m * q * (1.0 - q)) + 2.0;
    const long long j_hi = (long long)floor(centre - delta);          // keys above this rank: surely kept
    const long long j_lo = (long long)ceil(centre + delta);           // keys below this rank: surely dropped
    const bool have_hi = j_hi >= 1, have_lo = j_lo <= (long long)m;

    for (uint32_t b = threadIdx.x; b < HIST0_BINS; b += THREADS) h0[b] = 0;
    for (uint32_t b = threadIdx.x; b < 1024; b += THREADS) { hA[b] = 0; hB[b] = 0; }
    __syncthreads();
    for (uint32_t i = i_begin + threadIdx.x; i < i_end; i += THREADS) {
        const uint4 k = smp[i];
        atomicAdd(&h0[k.x >> 20], 1u); atomicAdd(&h0[k.y >> 20], 1u);
        atomicAdd(&h0[k.z >> 20], 1u); atomicAdd(&h0[k.w >> 20], 1u);
    }
    if (C > 1) cluster.sync();
    // when k is so small that no sample rank lies safely above the threshold there is no "sure"
    // set (hi stays at the largest key); the candidate histogram then spans up to the largest
    // sample key and everything above it shares the last bin
    if (rank == 0) {
        for (uint32_t b = threadIdx.x; b < HIST0_BINS; b += THREADS) {
            uint32_t v = h0[b];
            for (uint32_t r = 1; r < C; ++r) v += cluster.map_shared_rank(h0, r)[b];
            h0[b] = v;
        }
        __syncthreads();
        const uint32_t rankA = have_hi ? (uint32_t)j_hi : 1u;
        uint32_t binA = 0, needA = 0, binB = 0, needB = 0, cnt = 0;
        find_from_top<HIST0_BINS>(h0, rankA, s_tmp, binA, needA, cnt);
        if (have_lo) find_from_top<HIST0_BINS>(h0, (uint32_t)j_lo, s_tmp, binB, needB, cnt);
        if (threadIdx.x == 0) { s_bins[0] = binA; s_bins[1] = binB; s_bins[2] = needA; s_bins[3] = needB; }
    }
    if (C > 1) cluster.sync();
    if (C == 1) __syncthreads();
    const uint32_t* bins0 = C > 1 ? cluster.map_shared_rank(s_bins, 0) : s_bins;
    const uint32_t binA = bins0[0], binB = bins0[1];
    for (uint32_t i = i_begin + threadIdx.x; i < i_end; i += THREADS) {
        const uint4 k = smp[i];
        const uint32_t kk[4] = {k.x, k.y, k.z, k.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if ((kk[c] >> 20) == binA) atomicAdd(&hA[(kk[c] >> 10) & 1023u], 1u);
            if (have_lo && (kk[c] >> 20) == binB) atomicAdd(&hB[(kk[c] >> 10) & 1023u], 1u);
        }
    }
    if (C > 1) cluster.sync();
    if (rank == 0) {
        for (uint32_t b = threadIdx.x; b < 1024; b += THREADS) {
            uint32_t va = hA[b], vb = hB[b];
            for (uint32_t r = 1; r < C; ++r) {
                va += cluster.map_shared_rank(hA, r)[b];
                vb += cluster.map_shared_rank(hB, r)[b];
            }
            hA[b] = va; hB[b] = vb;
        }
        __syncthreads();
        const uint32_t needA = s_bins[2], needB = s_bins[3];
        uint32_t top = 0x7FFFFFFFu, lo = 0u, bin1 = 0, need1 = 0, cnt = 0;
        if (find_from_top<1024>(hA, needA, s_tmp, bin1, need1, cnt)) top = (binA << 20) | (bin1 << 10) | 1023u;
        if (have_lo && find_from_top<1024>(hB, needB, s_tmp, bin1, need1, cnt)) lo = (binB << 20) | (bin1 << 10);
        const uint32_t hi = have_hi ? top : 0x7FFFFFFFu;
        if (lo > top) lo = top;                                        // (cannot happen; keeps the bracket sane)
        if (threadIdx.x == 0) {
            const uint32_t width_m1 = top - lo;
            const uint32_t bits = width_m1 ? 32u - (uint32_t)__clz((int)width_m1) : 0u;
            FastState st = {};
            st.path = PATH_FAST; st.lo = lo; st.hi = hi; st.shift = bits > 11u ? bits - 11u : 0u;
            P.state[prob] = st;
        }
    }
    if (C > 1) cluster.sync();                                                    // peers stay until CTA 0 has read their histograms
}

// ---- main streaming pass ---------------------------------------------------------------
// Mapping: warp w of a tile owns 512 consecutive elements as four rows of 128; lane l holds
// the quad at 128 j + 4 l of row j (coalesced 512-byte accesses).  Four per-row counts ride
// in the bytes of one word, so one 5-step warp scan ranks all rows.
__device__ inline uint32_t pack_counts(uint32_t bits16) {
    return __popc(bits16 & 0xFu) | (__popc(bits16 & 0xF0u) << 8) | (__popc(bits16 & 0xF00u) << 16) |
           (__popc(bits16 & 0xF000u) << 24);
}
__device__ inline uint32_t warp_inclusive_scan(uint32_t v, uint32_t lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= (uint32_t)d) v += t;
    }
    return v;
}
__device__ inline uint32_t bytes_sum(uint32_t v) { return (v & 0xFFu) + ((v >> 8) & 0xFFu) + ((v >> 16) & 0xFFu) + (v >> 24); }

struct MainTile {                  // where a work item lives (uniform over the CTA)
    bool have, fast, full;
    uint32_t w, lt, s;
    SegEntry seg;
    long long first;               // segment-local coordinate of the tile's first element
    const float* g;
    float* e;
};
__device__ inline MainTile main_decode(const FastParams& P, uint32_t item) {
    const Layout& L = P.L;
    MainTile t{};
    t.have = item < P.total_items;
    if (!t.have) return t;
    t.w = item / L.tiles_per_worker;
    t.lt = item - t.w * L.tiles_per_worker;
    t.s = (L.nseg == 1) ? 0u : find_by_tile(L, t.lt);
    t.seg = L.segs[t.s];
    t.fast = t.seg.fast != 0;
    const size_t row = (size_t)t.w * L.n_total + t.seg.offset;
    t.g = P.grads + row;
    t.e = P.residuals + row;
    t.first = (long long)(t.lt - t.seg.tile_begin) * TILE - misalign_of(t.e);
    t.full = t.first >= 0 && t.first + TILE <= (long long)t.seg.n;
    return t;
}
// Two builds of the same code: MINB = 3 holds the kernel to 80 registers (three CTAs per SM), which is what
// many short segments and dense lists want; MINB = 1 lets it take 97 (two CTAs per SM), which streams long
// segments with sparse lists 1.4 % faster (350 M x 16 at 1 %: 10.45 against 10.65 ms; at 10 %: 12.1 against
// 11.6 ms the other way round).  The host picks one per segment table.
template <int MINB>
__global__ void __launch_bounds__(THREADS, MINB)
topk_main_kernel(FastParams P) {
    __shared__ uint32_t sh[CAND_BINS];                                 // candidate histogram
    __shared__ __align__(16) float s_p[TILE];                          // the tile's p values, for the per-element work
    __shared__ uint16_t s_list[WARPS][512];                            // per warp: its flagged elements, in coordinate order
    __shared__ uint32_t s_wflag[2][WARPS];
    __shared__ uint32_t s_cnt[3][2];                                   // per tile in flight: candidates appended, sure elements
    const Layout& L = P.L;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint32_t off0 = warp * 512u + lane * 4u;                     // this thread's quad of row 0 inside a tile
    // A segment's flagged and candidate lists are cut into regions: one per CTA of this kernel when the
    // segment has more tiles than CTAs (a tile's slots then follow from running counters), else one
    // per tile.  Either way no CTA waits for another and the flagged list does not depend on scheduling.
    // Candidates are appended through a shared-memory counter, so their order inside a tile's slice is
    // arbitrary (all later uses count or sort them).  A tile's candidate and sure counts are final once
    // every warp has passed the next barrier; they are written out then ("pending" tile).
    uint32_t run_flag = 0, run_cand = 0, tot_cand = 0, tot_sure = 0, fcap = 0, ccap = 0;
    for (uint32_t b = threadIdx.x; b < CAND_BINS; b += THREADS) sh[b] = 0;
    if (threadIdx.x < 6) s_cnt[threadIdx.x >> 1][threadIdx.x & 1] = 0;
    __syncthreads();
    long long cur_prob = -1;
    size_t cur_fidx = 0;
    uint32_t lo = 0, hi = 0, shift = 0, parity = 0;
    uint32_t slot3 = 0;                                                // counter pair of the current tile
    uint32_t pend_item = 0xFFFFFFFFu, pend_slot = 0, pend_room = 0;    // tile whose counts are not written yet
    bool pend_accumulates = false;
    const float gamma = L.gamma;
    const uint32_t group_step = (gridDim.x - 1u) * MAIN_GROUP + 1u;    // from a group's last tile to the next group's first
    MainTile T{};
    uint32_t seg_tile_end = 0;                                         // first tile after T's segment
    for (uint32_t item = blockIdx.x * MAIN_GROUP, ig = 0; ;
         item += (ig + 1u == MAIN_GROUP ? group_step : 1u), ig = (ig + 1u == MAIN_GROUP ? 0u : ig + 1u)) {
        // inside a group the next tile usually belongs to the same (worker, segment): then only its position
        // changes, and the lookup of the segment (a search over the table) is skipped
        if (ig != 0u && T.have && T.lt + 1u < seg_tile_end) {
            T.lt += 1u;
            T.first += TILE;
            T.full = T.first >= 0 && T.first + TILE <= (long long)T.seg.n;
        } else {
            T = main_decode(P, item);
            seg_tile_end = T.have ? L.segs[T.s + 1].tile_begin : 0u;
        }
        // ---- flush the per-segment accumulators when the segment changes ---------------------------
        const long long prob = T.have ? (long long)T.w * L.nseg + T.s : -2;
        if (prob != cur_prob && cur_prob >= 0) {                       // uniform over the CTA
            __syncthreads();                                           // the last tile's counts are final
            if (pend_item != 0xFFFFFFFFu) {
                const uint32_t c = min(s_cnt[pend_slot][0], pend_room), su = s_cnt[pend_slot][1];
                if (threadIdx.x == 0) { P.tile_ccnt[pend_item] = c; P.tile_sure[pend_item] = su; }
                tot_cand += c; tot_sure += su;
                pend_item = 0xFFFFFFFFu;
            }
            if (threadIdx.x == 0) {
                if (tot_sure) atomicAdd(&P.state[cur_prob].sure_total, tot_sure);
                if (tot_cand) atomicAdd(&P.state[cur_prob].cand_total, tot_cand);
            }
            for (uint32_t b = threadIdx.x; b < CAND_BINS; b += THREADS) {
                const uint32_t c = sh[b];
                if (c) { atomicAdd(P.cand_hist + cur_fidx * CAND_BINS + b, c); sh[b] = 0; }
            }
            __syncthreads();
            if (threadIdx.x < 6) s_cnt[threadIdx.x >> 1][threadIdx.x & 1] = 0;
            __syncthreads();
            tot_sure = 0; run_flag = 0; run_cand = 0; tot_cand = 0;
            cur_prob = -1;
        }
        if (!T.have) break;
        if (!T.fast) continue;                                         // uniform over the CTA
        const SegEntry& seg = T.seg;
        if (prob != cur_prob) {
            cur_prob = prob;
            cur_fidx = (size_t)T.w * L.fast_per_worker + seg.fast_index;
            const FastState st = P.state[prob];
            lo = st.lo; hi = st.hi; shift = st.shift;
            fcap = seg.flag_cap; ccap = seg.cand_cap;                  // region sizes
        }
        parity ^= 1u;
        slot3 = slot3 == 2u ? 0u : slot3 + 1u;
        float* e = T.e;
        const long long mine = T.first + off0;                         // quad of row 0; row j at + 128 j
        float* sp = s_p;
        __syncwarp();                                                  // the warp's reads of the previous tile's p are done

        // ---- stream: p = g + e goes straight back to the residual and stays in shared memory ----------
        uint32_t flag16 = 0;                                           // bit 4 j + c: key >= lo
        if (T.full) {
            float4 ev[QUADS], gv[QUADS];
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                ev[j] = __ldcs(reinterpret_cast<const float4*>(e + mine + 128 * j));
                gv[j] = __ldcs(reinterpret_cast<const float4*>(T.g + mine + 128 * j));
            }
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const float4 p = accumulate(gamma, gv[j], ev[j]);
                *reinterpret_cast<float4*>(e + mine + 128 * j) = p;
                *reinterpret_cast<float4*>(sp + off0 + 128 * j) = p;
                flag16 |= ((uint32_t)(key_of(p.x) >= lo) | (uint32_t)(key_of(p.y) >= lo) << 1 |
                           (uint32_t)(key_of(p.z) >= lo) << 2 | (uint32_t)(key_of(p.w) >= lo) << 3) << (4 * j);
            }
        } else {
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const long long base = mine + 128 * j;
                float p[4], gq[4];
                const uint32_t valid = load_quad(e, base, seg.n, p);
                load_quad_stream(T.g, base, seg.n, gq);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    p[c] = accumulate(gamma, gq[c], p[c]);
                    flag16 |= (((valid >> c) & 1u) & (uint32_t)(key_of(p[c]) >= lo)) << (4 * j + c);
                }
                if (valid) store_quad(e, base, valid, p);
                *reinterpret_cast<float4*>(sp + off0 + 128 * j) = make_float4(p[0], p[1], p[2], p[3]);
            }
        }
        // the loads of this tile have landed: ask L2 for the tile this CTA takes next, so that DRAM stays busy
        // during the per-element work below (measured on 350 M x 16 at 1 %: 12.3 -> 10.85 ms)
        if (SC_PREFETCH_DIST) {
            const uint32_t ahead = ig + 1u == MAIN_GROUP ? group_step : 1u;    // distance to this CTA's next tile
            if (T.full && T.lt + ahead + 1u < seg_tile_end) {
                prefetch_tile_l2(T.g, e, T.first + (long long)ahead * TILE);
            } else {                                                   // the next tile lies in another segment: locate it
                const MainTile N = main_decode(P, item + ahead);
                if (N.have && N.fast && N.full) prefetch_tile_l2(N.g, N.e, N.first);
            }
        }
        // ---- ranks of the flagged elements, in coordinate order ---------------------------------------
        const uint32_t fcnt4 = pack_counts(flag16);
        const uint32_t finc4 = warp_inclusive_scan(fcnt4, lane);
        const uint32_t ftot4 = __shfl_sync(0xFFFFFFFFu, finc4, 31);
        const uint32_t wflag = bytes_sum(ftot4);                       // flagged elements of this warp's 512
        if (lane == 0) s_wflag[parity][warp] = wflag;
        // each lane files its flagged elements (position inside the warp's 512) under their rank, so that the
        // per-element work below is spread evenly over the lanes whatever the lane they came from
        if (flag16) {
            const uint32_t ex4 = finc4 - fcnt4;
            const uint32_t r0 = ftot4 & 0xFFu, r1 = (ftot4 >> 8) & 0xFFu, r2 = (ftot4 >> 16) & 0xFFu;
            // first slot of this lane's quad in each row, relative to the warp's slice (< 512: 16 bits each)
            const uint32_t q01 = (ex4 & 0xFFu) | ((r0 + ((ex4 >> 8) & 0xFFu)) << 16);
            const uint32_t q23 = (r0 + r1 + ((ex4 >> 16) & 0xFFu)) | ((r0 + r1 + r2 + (ex4 >> 24)) << 16);
            uint32_t bits = flag16;
            while (bits) {
                const uint32_t i = (uint32_t)__ffs((int)bits) - 1u;
                bits &= bits - 1u;
                const uint32_t j = i >> 2;
                const uint32_t slot = (((j & 2u) ? q23 : q01) >> (16u * (j & 1u)) & 0xFFFFu) +
                                      __popc(flag16 & ((1u << i) - 1u) & (0xFu << (4u * j)));
                s_list[warp][slot] = (uint16_t)(128u * j + 4u * lane + (i & 3u));
            }
        }
        __syncthreads();
        uint32_t tflag = 0, fwbase = 0;
#pragma unroll
        for (int i = 0; i < WARPS; ++i) {
            const uint32_t f = s_wflag[parity][i];
            fwbase += (i < (int)warp) ? f : 0u;
            tflag += f;
        }
        // the previous tile's counts are final now (every warp has left its per-element loop)
        if (pend_item != 0xFFFFFFFFu) {
            const uint32_t c = min(s_cnt[pend_slot][0], pend_room), su = s_cnt[pend_slot][1];
            if (threadIdx.x == 0) { P.tile_ccnt[pend_item] = c; P.tile_sure[pend_item] = su; }
            if (pend_accumulates) run_cand += c;
            tot_cand += c; tot_sure += su;
        }
        // this CTA's regions of the two lists, and where this tile's entries go inside them
        const uint32_t tseg = T.lt - seg.tile_begin;                   // tile inside the segment
        if (seg.region_per_tile) { run_flag = 0; run_cand = 0; }
        const uint32_t region = seg.region_per_tile ? tseg : blockIdx.x;
        const bool fits = run_flag + tflag <= fcap;
        const uint32_t fbase = region * fcap + run_flag, cbase = region * ccap + run_cand;
        const uint32_t room = ccap - run_cand;                         // candidate slots left for this tile
        if (threadIdx.x == 0) {
            P.tile_fbase[item] = fits ? fbase : 0xFFFFFFFFu;
            P.tile_fcnt[item] = tflag;
            P.tile_cbase[item] = cbase;
            if (!fits) P.state[prob].overflow = 1u;                    // a region is full: the segment falls back
            const uint32_t nxt = slot3 == 2u ? 0u : slot3 + 1u;        // counters of the tile after this one
            s_cnt[nxt][0] = 0; s_cnt[nxt][1] = 0;
        }
        pend_item = item; pend_slot = slot3; pend_room = fits ? room : 0u; pend_accumulates = !seg.region_per_tile;
        if (fits) run_flag += tflag;
        if (fits && wflag) {
            // the tile's entries fit: write them (entry r of the warp's slice by lane r % 32: coalesced), zero
            // the sure ones in the residual (their values stay in the list, from where a fall-back restores
            // them), append the candidates to the tile's slice and histogram them
            uint2* flist = P.flagged + (size_t)T.w * L.flag_per_worker + seg.flag_begin + fbase + fwbase;
            uint2* clist = P.cand + (size_t)T.w * L.cand_per_worker + seg.cand_begin + cbase;
            const uint32_t first32 = (uint32_t)T.first + warp * 512u;
            const float* spw = sp + warp * 512u;
            uint32_t sure_w = 0;
            for (uint32_t r0 = 0; r0 < wflag; r0 += 32) {
                const uint32_t r = r0 + lane;
                const bool active = r < wflag;
                const uint32_t li = active ? (uint32_t)s_list[warp][r] : 0u;
                const float v = spw[li];
                const uint32_t key = key_of(v);
                const uint32_t coord = first32 + li;
                const bool sure = active && key > hi;
                const bool cand = active && key <= hi;
                if (active) flist[r] = make_uint2(__float_as_uint(v), coord);
                if (sure) e[coord] = 0.0f;
                const uint32_t bs = __ballot_sync(0xFFFFFFFFu, sure);
                const uint32_t bc = __ballot_sync(0xFFFFFFFFu, cand);
                sure_w += __popc(bs);
                if (bc) {                                              // uniform over the warp
                    uint32_t base = 0;
                    if (lane == 0) base = atomicAdd(&s_cnt[slot3][0], (uint32_t)__popc(bc));
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    if (cand) {
                        const uint32_t pos = base + __popc(bc & lt_mask);
                        if (pos < room) {
                            clist[pos] = make_uint2(key, coord);
                            atomicAdd(&sh[min((key - lo) >> shift, CAND_BINS - 1u)], 1u);
                        } else {
                            P.state[prob].overflow = 1u;
                        }
                    }
                }
            }
            if (lane == 0 && sure_w) atomicAdd(&s_cnt[slot3][1], sure_w);
        }
    }
}

// ---- resolve 1: validity of the bracket, bin of the threshold (one CTA per problem) ------
__global__ void __launch_bounds__(THREADS)
topk_candbin_kernel(FastParams P) {
    __shared__ uint32_t s_tmp[WARPS + 4];
    const Layout& L = P.L;
    uint32_t w, s;
    const uint32_t prob = fast_problem(L, blockIdx.x, w, s);
    const SegEntry seg = L.segs[s];
    FastState st = P.state[prob];
    if (st.path != PATH_FAST) return;
    const size_t fidx = (size_t)w * L.fast_per_worker + seg.fast_index;
    bool ok = st.overflow == 0u && st.sure_total <= seg.k &&
              (uint64_t)seg.k <= (uint64_t)st.sure_total + st.cand_total;
    uint32_t bin = 0, need_in = 0, cnt = 0;
    const uint32_t need = ok ? seg.k - st.sure_total : 0u;
    if (ok && need) {
        ok = find_from_top<CAND_BINS>(P.cand_hist + fidx * CAND_BINS, need, s_tmp, bin, need_in, cnt);
        ok = ok && cnt <= LIST2_CAP;
    }
    if (threadIdx.x == 0) {
        if (!ok) {
            st.path = PATH_FAILED;
            atomicAdd(P.n_slow, 1u);
            atomicAdd(P.n_failed, 1u);
        } else if (need == 0) {
            st.need2 = 0; st.T = st.hi; st.icut = 0;                   // exactly the sure elements are kept
        } else {
            st.lo2 = st.lo + (bin << st.shift);
            const uint64_t top = (uint64_t)st.lo2 + (1ull << st.shift) - 1ull;
            st.hi2 = bin == CAND_BINS - 1u ? st.hi : (uint32_t)min(top, (uint64_t)st.hi);
            st.need2 = need_in;
            st.T = cnt;                                                // expected length of the short list (checked later)
        }
        st.cnt2 = 0;
        P.state[prob] = st;
    }
}

// ---- per-tile walks over the candidate slices ----------------------------------------------------
// Eight lanes share TILES_PER_GROUP consecutive tiles.  The kernels below are bound by a chain of
// dependent loads (slice length and base, then the slice), so a group first requests the placement
// words of all its tiles, then the first eight candidates of every tile, and only then looks at
// them: four tiles per group cut the number of such chains per launch by four.
constexpr uint32_t TILES_PER_GROUP = 4;
struct CandSlice {                 // one tile's slice as seen by a lane of its group
    const uint2* list;             // nullptr: nothing to do for this tile
    uint32_t cnt, prob, w, lt;
    uint2 first;                   // entry `sub` of the slice (if sub < cnt)
};
template <bool NEED_FILTER>
__device__ inline void cand_slices(const FastParams& P, uint32_t item0, uint32_t sub, CandSlice (&t)[TILES_PER_GROUP]) {
    const Layout& L = P.L;
    uint32_t base[TILES_PER_GROUP];
#pragma unroll
    for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
        const uint32_t item = item0 + u;
        t[u].list = nullptr; t[u].cnt = 0; base[u] = 0;
        if (item < P.total_items) { t[u].cnt = __ldg(P.tile_ccnt + item); base[u] = __ldg(P.tile_cbase + item); }
    }
#pragma unroll
    for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
        const uint32_t item = item0 + u;
        t[u].first = make_uint2(0u, 0u);
        if (item >= P.total_items) continue;
        t[u].w = item / L.tiles_per_worker;
        t[u].lt = item - t[u].w * L.tiles_per_worker;
        const uint32_t s = (L.nseg == 1) ? 0u : find_by_tile(L, t[u].lt);
        const SegEntry& seg = L.segs[s];
        t[u].prob = t[u].w * L.nseg + s;
        if (!seg.fast) { t[u].cnt = 0; continue; }
        const FastState* st = P.state + t[u].prob;
        if (st->path != PATH_FAST || (NEED_FILTER && st->need2 == 0)) { t[u].cnt = 0; continue; }
        t[u].list = P.cand + (size_t)t[u].w * L.cand_per_worker + seg.cand_begin + base[u];
        if (sub < t[u].cnt) t[u].first = __ldg(t[u].list + sub);
    }
}

// ---- filter: copy the candidates of the threshold's bin into the short list ----------------------
__global__ void __launch_bounds__(THREADS)
topk_candfilter_kernel(FastParams P) {
    const Layout& L = P.L;
    const uint32_t sub = threadIdx.x & 7u;
    const uint32_t item0 = ((blockIdx.x * THREADS + threadIdx.x) >> 3) * TILES_PER_GROUP;
    CandSlice t[TILES_PER_GROUP];
    cand_slices<true>(P, item0, sub, t);
#pragma unroll
    for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
        // candidates above the threshold's bin are kept whatever the exact threshold turns out to be; those
        // inside the bin go to the short list.  Both counts are left for the per-tile kept count, which then
        // reads a tile's candidates again only if some of them lie inside the bin (a few thousand tiles at most).
        uint32_t above = 0, inbin = 0;
        if (t[u].list && t[u].cnt) {
            const FastState* stp = P.state + t[u].prob;
            const uint32_t lo2 = stp->lo2, hi2 = stp->hi2;
            const uint32_t s = t[u].prob - t[u].w * L.nseg;
            uint2* out = P.list2 + ((size_t)t[u].w * L.fast_per_worker + L.segs[s].fast_index) * LIST2_CAP;
            for (uint32_t i = sub; i < t[u].cnt; i += 8) {
                const uint2 c = i == sub ? t[u].first : t[u].list[i];
                if (c.x > hi2) ++above;
                else if (c.x >= lo2) {
                    ++inbin;
                    const uint32_t pos = atomicAdd(&P.state[t[u].prob].cnt2, 1u);
                    if (pos < LIST2_CAP) out[pos] = c;
                }
            }
        }
        uint32_t both = above | (inbin << 16);                         // a tile holds at most 4096 candidates
        both += __shfl_xor_sync(0xFFFFFFFFu, both, 1);
        both += __shfl_xor_sync(0xFFFFFFFFu, both, 2);
        both += __shfl_xor_sync(0xFFFFFFFFu, both, 4);
        if (sub == 0u && item0 + u < P.total_items) P.tile_csum[item0 + u] = both;
    }
}

// ---- resolve 2: sort the short list, read off the threshold and the tie cut -------------------
__global__ void __launch_bounds__(THREADS)
topk_final_kernel(FastParams P) {
    __shared__ unsigned long long srt[LIST2_CAP];
    const Layout& L = P.L;
    uint32_t w, s;
    const uint32_t prob = fast_problem(L, blockIdx.x, w, s);
    FastState st = P.state[prob];
    if (st.path != PATH_FAST || st.need2 == 0) return;
    const uint32_t cnt = st.cnt2;
    if (cnt != st.T || cnt > LIST2_CAP || st.need2 > cnt) {            // short list disagrees with the histogram
        if (threadIdx.x == 0) { P.state[prob].path = PATH_FAILED; atomicAdd(P.n_slow, 1u); atomicAdd(P.n_failed, 1u); }
        return;
    }
    uint32_t size = 1;
    while (size < cnt) size <<= 1;
    const uint2* in = P.list2 + ((size_t)w * L.fast_per_worker + L.segs[s].fast_index) * LIST2_CAP;
    for (uint32_t i = threadIdx.x; i < size; i += THREADS) {
        unsigned long long v = 0;                                       // padding sorts last
        if (i < cnt) { const uint2 c = in[i]; v = ((unsigned long long)c.x << 32) | (0xFFFFFFFFu - c.y); }
        srt[i] = v;
    }
    __syncthreads();
    // bitonic sort, descending: larger key first, equal keys: lower coordinate first
    for (uint32_t k2 = 2; k2 <= size; k2 <<= 1) {
        for (uint32_t j = k2 >> 1; j > 0; j >>= 1) {
            for (uint32_t i = threadIdx.x; i < size; i += THREADS) {
                const uint32_t ixj = i ^ j;
                if (ixj > i) {
                    const unsigned long long a = srt[i], b = srt[ixj];
                    const bool desc = (i & k2) == 0;
                    if (desc ? (a < b) : (a > b)) { srt[i] = b; srt[ixj] = a; }
                }
            }
            __syncthreads();
        }
    }
    if (threadIdx.x == 0) {
        const unsigned long long v = srt[st.need2 - 1u];
        st.T = (uint32_t)(v >> 32);
        st.icut = (0xFFFFFFFFu - (uint32_t)v) + 1u;                  // coordinates below this are kept among the ties
        if (st.icut == 0) st.icut = 0xFFFFFFFFu;                      // (coordinate 2^32-1 cannot occur: n < 2^32)
        P.state[prob] = st;
    }
}

__device__ inline bool fast_kept(uint32_t key, uint32_t coord, uint32_t T, uint32_t icut) {
    return key > T || (key == T && coord < icut);
}

// ---- kept count per tile = sure elements + chosen candidates -------------------------------------
__global__ void __launch_bounds__(THREADS)
topk_tilecount_kernel(FastParams P) {                                 // one thread per tile
    const Layout& L = P.L;
    const uint32_t item = blockIdx.x * THREADS + threadIdx.x;
    if (item >= P.total_items) return;
    const uint32_t sure = __ldg(P.tile_sure + item), both = __ldg(P.tile_csum + item);
    const uint32_t w = item / L.tiles_per_worker;
    const uint32_t lt = item - w * L.tiles_per_worker;
    const uint32_t s = (L.nseg == 1) ? 0u : find_by_tile(L, lt);
    const SegEntry& seg = L.segs[s];
    uint32_t kept = 0;
    if (seg.fast) {
        const FastState* st = P.state + (size_t)w * L.nseg + s;
        if (st->path == PATH_FAST) {
            kept = sure + (both & 0xFFFFu);
            if (both >> 16) {                                          // candidates inside the threshold's bin: the exact rule
                const uint32_t T = st->T, icut = st->icut, lo2 = st->lo2, hi2 = st->hi2;
                const uint2* list = P.cand + (size_t)w * L.cand_per_worker + seg.cand_begin + P.tile_cbase[item];
                const uint32_t cnt = P.tile_ccnt[item];
                for (uint32_t i = 0; i < cnt; ++i) {
                    const uint2 c = list[i];
                    if (c.x >= lo2 && c.x <= hi2) kept += fast_kept(c.x, c.y, T, icut) ? 1u : 0u;
                }
            }
        }
    }
    P.offsets[(size_t)w * (L.tiles_per_worker + 1) + lt] = kept;
}

// ---- emit: G lanes per tile walk the tile's slice of the flagged list ----------------------------
// Sparse slices (a few dozen entries) take a part of a warp per tile, i.e. several tiles per warp
// side by side; long slices take the whole warp and more entries per lane.  One batch covers
// G x D entries.  (Loading the placement words two tiles ahead and asking L2 for the next slice
// one tile ahead changed nothing: the kernel is not bound by its chain of dependent loads.)
template <int G, int D>
__global__ void __launch_bounds__(THREADS)
topk_emit_kernel(FastParams P) {
    static_assert(G == 8 || G == 16 || G == 32, "lanes per tile");
    const Layout& L = P.L;
    const uint32_t lane = threadIdx.x & 31u;
    constexpr uint32_t TPW = 32 / G;                                    // tiles per warp
    const uint32_t grp = lane / G, gl = lane % G;
    const uint32_t gshift = grp * G;
    const uint32_t gmask = (G == 32) ? 0xFFFFFFFFu : ((1u << G) - 1u);
    const uint32_t lt_mask = (1u << gl) - 1u;
    const uint32_t stride = gridDim.x * WARPS * TPW;
    const uint32_t rounds = (P.total_items + stride - 1) / stride;      // the same for every lane: ballots stay whole
    // per-(worker, segment) constants stay in registers while the group's tiles belong to the same one
    uint32_t cw = 0xFFFFFFFFu, cs = 0xFFFFFFFFu, c_tile_end = 0;        // cached worker, segment, end of its tile range
    uint32_t T = 0, icut = 0, hi = 0, seg_k = 0, idx0 = 0, tile_begin = 0, off_begin = 0;
    bool live = false;
    const uint2* flist0 = nullptr;
    float* e = nullptr;
    float* ovals = nullptr;
    uint32_t* oidx = nullptr;
    uint32_t item = (blockIdx.x * WARPS + (threadIdx.x >> 5)) * TPW + grp;
    for (uint32_t round = 0; round < rounds; ++round, item += stride) {
        uint32_t cnt = 0, base = 0, running = 0;
        if (item < P.total_items) {
            const uint32_t w = item / L.tiles_per_worker;
            const uint32_t lt = item - w * L.tiles_per_worker;
            if (w != cw || lt < tile_begin || lt >= c_tile_end) {       // another (worker, segment): reload
                cw = w;
                cs = (L.nseg == 1) ? 0u : find_by_tile(L, lt);
                const SegEntry seg = L.segs[cs];
                tile_begin = seg.tile_begin; c_tile_end = L.segs[cs + 1].tile_begin;
                const FastState* st = P.state + (size_t)w * L.nseg + cs;
                live = seg.fast && st->path == PATH_FAST;
                T = st->T; icut = st->icut; hi = st->hi; seg_k = seg.k; idx0 = (uint32_t)seg.offset;
                off_begin = P.offsets[(size_t)w * (L.tiles_per_worker + 1) + tile_begin];
                flist0 = P.flagged + (size_t)w * L.flag_per_worker + seg.flag_begin;
                e = P.residuals + (size_t)w * L.n_total + seg.offset;
                ovals = P.out_vals + (size_t)w * L.K_total + seg.msg_off;
                oidx = P.out_idx + (size_t)w * L.K_total + seg.msg_off;
            }
            if (live) {
                // the four words that place this tile: independent loads, one round trip
                const uint32_t* o = P.offsets + (size_t)w * (L.tiles_per_worker + 1) + lt;
                cnt = __ldg(P.tile_fcnt + item); base = __ldg(P.tile_fbase + item);
                const uint32_t o0 = __ldg(o), o1 = __ldg(o + 1);
                running = o0 - off_begin;                               // kept coordinates of the segment before this tile
                if (cnt && (unsigned long long)running + (o1 - o0) > seg_k) {   // counts and k disagree: write nothing
                    if (gl == 0) atomicMin(P.status, ST_DEVICE_CHECK);
                    cnt = 0;
                }
            }
        }
        const uint32_t maxcnt = __reduce_max_sync(0xFFFFFFFFu, cnt);
        // entry i of the slice belongs to lane i % G of the group; the message position advances with the running rank
        uint32_t pos = running;
        const uint2* fl = flist0 + base + gl;
        for (uint32_t b = 0; b < maxcnt; b += G * D) {                  // D independent loads in flight per lane
            uint2 a[D];
#pragma unroll
            for (int u = 0; u < D; ++u) a[u] = (b + G * u + gl < cnt) ? __ldg(fl + b + G * u) : make_uint2(0u, 0xFFFFFFFFu);
#pragma unroll
            for (int u = 0; u < D; ++u) {
                // a padding entry has key 0 and coordinate 2^32-1: it would be kept only if T == 0 and icut > 2^32-1,
                // which cannot be (a group without a tile has T and icut of its last tile, or 0 and 0)
                const uint32_t key = a[u].x & 0x7FFFFFFFu;
                const bool sel = key > T || (key == T && a[u].y < icut);
                const uint32_t bal = (__ballot_sync(0xFFFFFFFFu, sel) >> gshift) & gmask;
                if (sel) {
                    const uint32_t r = pos + __popc(bal & lt_mask);
                    ovals[r] = __uint_as_float(a[u].x);
                    oidx[r] = idx0 + a[u].y;
                    if (key <= hi) e[a[u].y] = 0.0f;                    // a kept candidate: the main pass left p there
                }
                pos += __popc(bal);
            }
        }
    }
}

// ---- restore: a segment fell back; put the sure values back so that the residual holds p ------
__global__ void __launch_bounds__(THREADS)
topk_restore_kernel(FastParams P) {
    const Layout& L = P.L;
    if (*P.n_failed == 0u) return;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warps_total = gridDim.x * WARPS;
    for (uint32_t item = blockIdx.x * WARPS + (threadIdx.x >> 5); item < P.total_items; item += warps_total) {
        const uint32_t w = item / L.tiles_per_worker;
        const uint32_t lt = item - w * L.tiles_per_worker;
        const uint32_t s = (L.nseg == 1) ? 0u : find_by_tile(L, lt);
        const SegEntry seg = L.segs[s];
        if (!seg.fast) continue;
        const FastState* st = P.state + (size_t)w * L.nseg + s;
        if (st->path != PATH_FAILED) continue;
        const uint32_t base = P.tile_fbase[item], cnt = P.tile_fcnt[item], hi = st->hi;
        if (base == 0xFFFFFFFFu || cnt == 0u) continue;                 // nothing was written, nothing was zeroed
        const uint2* flist = P.flagged + (size_t)w * L.flag_per_worker + seg.flag_begin + base;
        float* e = P.residuals + (size_t)w * L.n_total + seg.offset;
        for (uint32_t i = lane; i < cnt; i += 32) {
            const uint2 a = flist[i];
            if ((a.x & 0x7FFFFFFFu) > hi) e[a.y] = __uint_as_float(a.x);
        }
    }
}

}  // namespace sc
