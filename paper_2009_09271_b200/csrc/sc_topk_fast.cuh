// Top-k of a large segment in ONE pass over g and e (Methodology, "Top-k Sparsification";
// Algorithm 1 accumulate / compress / residual lines).
//
// A radix select has to see every key before it knows the threshold, which costs extra
// passes over HBM.  Here a small systematic sample of |g + e| brackets the threshold first:
//   bracket  m keys per (worker, segment) are read from 32-byte sectors, one per stretch of the segment
//            at a hashed place inside the stretch; two order
//            statistics of the sample, six standard deviations either side of rank k m / n, give
//            [lo, hi] with count(key > hi) <= k <= count(key >= lo) except with negligible
//            probability.  A key value that holds a large share of the sample at the lower order
//            statistic (exact zeros of a sparse gradient, a constant tensor) becomes the "tie key":
//            its elements are counted per tile instead of being listed;
//   main     the streaming pass forms p = g + e and writes the residual at once: 0 for the elements
//            above the sample's own estimate of the threshold, p for the rest.  Every element with key >= lo is
//            appended, in coordinate order inside its tile, to a "flagged" list (value,
//            coordinate); the few candidates (lo <= key <= hi) also go to a candidate list
//            and into a 2048-bin histogram.  The CTA that finishes a segment's last tile reads
//            the histogram and pins the bin of the k-th key (exact counts decide whether the
//            bracket held);
//   resolve  the candidates of that bin are copied to a short list; the CTA that finishes a
//            segment's last tile sorts it in shared memory (exact threshold T and the coordinate
//            cut for ties), admits tie-key elements by coordinate order if the threshold is the
//            tie key, and scans the per-tile kept counts into message offsets;
//   emit     a pass over the flagged list only: kept entries go to the message in ascending
//            coordinate order; the few entries between the estimated and the exact threshold are
//            corrected in the residual (scattered accesses to DRAM cost a row cycle each, so as few
//            as possible are left for this step); tiles that admit tie-key elements are re-read from
//            the residual instead.
// Every count is exact, so the result equals the plain definition; the sample only decides how
// much work that takes.  If the bracket is wrong (counts prove it) or a list overflows, the
// segment falls back to the radix select on the parked p.
// No CTA polls for another anywhere on this path: the bracket uses a thread-block cluster, whose
// CTAs meet at hardware cluster barriers only, and "the CTA that finishes last" is found with one
// atomic counter per segment (nobody waits for it).
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
    uint32_t* tile_sure;       // [W * tiles_per_worker] sure elements of the tile
    uint32_t* tile_cbase;      // first candidate slot of the tile
    uint32_t* tile_ccnt;       // candidates of the tile
    uint32_t* tile_csum;       // kept candidates of the tile (low half), candidates inside the threshold's bin (high
                               // half); after the resolve step of a segment that admits ties: ties admitted in the tile
    uint32_t* tile_fbase;      // first flagged slot of the tile (0xFFFFFFFF: the list was full, nothing written)
    uint32_t* tile_fcnt;       // flagged elements of the tile
    uint32_t* tile_tie;        // elements equal to the tie key (written only for segments that have one)
    uint32_t* counters;        // [0] segments whose bracket missed, [1] segments that admit tie-key elements
    uint32_t* offsets;         // [W][tiles_per_worker + 1]: kept coordinates of the SEGMENT before the tile
    int* status;
    uint32_t total_items;
    uint32_t main_group;       // consecutive tiles a CTA of the streaming pass takes at a time (<= MAIN_GROUP)
};

// The per-segment launches of this path cover the fast segments only: problem index
// f = w * fast_per_worker + fast_index, mapped to the segment through the layout's fast list.
__device__ inline uint32_t fast_problem(const Layout& L, uint32_t f, uint32_t& w, uint32_t& s) {
    w = f / L.fast_per_worker;
    s = L.fast_list[f - w * L.fast_per_worker];
    return w * L.nseg + s;
}

// Reads that must see what other CTAs wrote or added with atomics: straight from L2.
struct L2Words {
    const uint32_t* p;
    __device__ uint32_t operator[](uint32_t i) const { return __ldcg(p + i); }
};
__device__ inline FastState load_state_l2(const FastState* p) {
    FastState st;
    const uint4* src = reinterpret_cast<const uint4*>(p);
    uint4* dst = reinterpret_cast<uint4*>(&st);
#pragma unroll
    for (int i = 0; i < (int)(sizeof(FastState) / 16); ++i) dst[i] = __ldcg(src + i);
    return st;
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

// ---- bracket: sample the segment, take two order statistics of the sample ---------------------
// One thread-block cluster of BRACKET_CTAS CTAs per problem (one CTA for small samples).  Every CTA
// reads its share of the sample: one 32-byte sector (8 elements) of g and e per step and thread, one
// sector per stretch of the segment at a hashed place inside it; the keys are kept in global memory for
// the later histogram passes (each thread reads back only what it wrote itself).  The first pass histograms key bits 30..20 in shared memory, CTA 0 adds the
// shares up through distributed shared memory, walks the total and hands the two bins back the same
// way; the second pass refines them by ten more bits.  If the lower order statistic falls on a key prefix that
// holds a large share of the sample, a third pass resolves the last ten bits: when ONE key value holds that
// share it becomes the tie key (counted, not listed, by the streaming pass).
// The cluster barriers are the hardware's; no CTA leaves before the last one (a peer's shared memory
// must stay alive while it is read).  `first` and `count` select a range of the fast list; the grid
// covers count problems of every worker.
constexpr uint32_t BRACKET_CTAS = 8;
constexpr uint32_t BRACKET_BIG_SAMPLE = 1u << 15;                      // samples from this size up take a cluster
constexpr int SAMPLE_BATCH = 4;                                        // sectors of g and e in flight per thread
// a key value is "massive" when it holds at least 1/256 of the sample (its elements would fill a good
// part of the candidate list, which has room for n/32 entries) and at least 16 keys
__device__ inline bool massive_in_sample(uint32_t cnt, uint32_t m) { return cnt >= 16u && (uint64_t)cnt * 256u >= m; }

template <uint32_t C>
__global__ void __launch_bounds__(THREADS)
topk_bracket_kernel(FastParams P, uint32_t first, uint32_t count) {
    namespace cg = cooperative_groups;
    __shared__ uint32_t h0[HIST0_BINS];
    __shared__ uint32_t hA[1024], hB[1024], hC[1024], hM[1024];
    __shared__ uint32_t s_tmp[WARPS + 4];
    __shared__ uint32_t s_bins[8];                                     // valid in CTA 0: binA, binB, needA, needB, third pass?, prefix B, binM, needM
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = C > 1 ? cluster.block_rank() : 0u;
    const Layout& L = P.L;
    uint32_t w, s;
    const uint32_t pidx = blockIdx.x / C;                              // problem of this launch: (worker, position in the range)
    const uint32_t prob = fast_problem(L, (pidx / count) * L.fast_per_worker + first + pidx % count, w, s);
    const SegEntry seg = L.segs[s];
    const uint32_t m = seg.sample_m;
    uint4* smp = reinterpret_cast<uint4*>(P.sample + (size_t)w * L.sample_per_worker + seg.sample_begin);
    // this CTA's share of the sample, in sectors of eight keys
    const uint32_t S = m / 8u;
    const uint32_t per = (S + C - 1u) / C;
    const uint32_t c_begin = min(rank * per, S), c_end = min(c_begin + per, S);
    // ranks (from the top) that bracket the k-th largest of the segment
    const double q = (double)seg.k / (double)seg.n;
    const double centre = q * (double)m;
    const double delta = 6.0 * sqrt((double)m * q * (1.0 - q)) + 2.0;
    const long long j_hi = (long long)floor(centre - delta);          // keys above this rank: surely kept
    const long long j_lo = (long long)ceil(centre + delta);           // keys below this rank: surely dropped
    const bool have_hi = j_hi >= 1, have_lo = j_lo <= (long long)m;

    for (uint32_t b = threadIdx.x; b < HIST0_BINS; b += THREADS) h0[b] = 0;
    for (uint32_t b = threadIdx.x; b < 1024; b += THREADS) { hA[b] = 0; hB[b] = 0; hC[b] = 0; hM[b] = 0; }
    __syncthreads();
    {   // ---- the sample: sector c of the sample is sector floor(c sectors / S) of the segment's aligned part
        const size_t row = (size_t)w * L.n_total + seg.offset;
        const float* g = P.grads + row;
        const float* e = P.residuals + row;
        const uint32_t a0 = (8u - (uint32_t)((reinterpret_cast<uintptr_t>(e) >> 2) & 7u)) & 7u;   // first 32-byte aligned element
        const uint32_t sectors = (seg.n - a0) / 8u;
        // one sector out of every `stride`, at a hashed place inside its stretch: evenly spread, but not periodic
        // (a tensor whose large entries repeat with the stride, a hot column of a matrix, would otherwise be
        // sampled at its large entries only, or never)
        const uint32_t stride = max(sectors / S, 1u);
        for (uint32_t c0 = c_begin + threadIdx.x; c0 < c_end; c0 += THREADS * SAMPLE_BATCH) {
            float4 ev[SAMPLE_BATCH][2], gv[SAMPLE_BATCH][2];
#pragma unroll
            for (int u = 0; u < SAMPLE_BATCH; ++u) {
                const uint32_t c = c0 + u * THREADS;
                if (c < c_end) {
                    const uint32_t jitter = mix32(c * 0x9E3779B9u + 0x85EBCA6Bu) % stride;
                    const size_t at = (size_t)a0 + ((size_t)(((uint64_t)c * sectors) / S) + jitter) * 8u;
                    ev[u][0] = *reinterpret_cast<const float4*>(e + at); ev[u][1] = *reinterpret_cast<const float4*>(e + at + 4);
                    gv[u][0] = *reinterpret_cast<const float4*>(g + at); gv[u][1] = *reinterpret_cast<const float4*>(g + at + 4);
                }
            }
#pragma unroll
            for (int u = 0; u < SAMPLE_BATCH; ++u) {
                const uint32_t c = c0 + u * THREADS;
                if (c < c_end) {
                    const float4 p0 = accumulate(L.gamma, gv[u][0], ev[u][0]), p1 = accumulate(L.gamma, gv[u][1], ev[u][1]);
                    uint4 k0, k1;
                    k0.x = key_of(p0.x); k0.y = key_of(p0.y); k0.z = key_of(p0.z); k0.w = key_of(p0.w);
                    k1.x = key_of(p1.x); k1.y = key_of(p1.y); k1.z = key_of(p1.z); k1.w = key_of(p1.w);
                    smp[2 * (size_t)c] = k0; smp[2 * (size_t)c + 1] = k1;
                    atomicAdd(&h0[k0.x >> 20], 1u); atomicAdd(&h0[k0.y >> 20], 1u);
                    atomicAdd(&h0[k0.z >> 20], 1u); atomicAdd(&h0[k0.w >> 20], 1u);
                    atomicAdd(&h0[k1.x >> 20], 1u); atomicAdd(&h0[k1.y >> 20], 1u);
                    atomicAdd(&h0[k1.z >> 20], 1u); atomicAdd(&h0[k1.w >> 20], 1u);
                }
            }
        }
    }
    if (C > 1) cluster.sync(); else __syncthreads();
    // when k is so small that no sample rank lies safely above the threshold there is no "sure"
    // set (hi stays at the largest key); the candidate histogram then spans up to the largest
    // sample key and everything above it shares the last bin.  The lower statistic is always
    // located (the smallest sample key when no rank lies safely below the threshold): that is
    // where a massive key value matters.
    if (rank == 0) {
        for (uint32_t b = threadIdx.x; b < HIST0_BINS; b += THREADS) {
            uint32_t v = h0[b];
            for (uint32_t r = 1; r < C; ++r) v += cluster.map_shared_rank(h0, r)[b];
            h0[b] = v;
        }
        __syncthreads();
        const uint32_t rankA = have_hi ? (uint32_t)j_hi : 1u, rankB = have_lo ? (uint32_t)j_lo : m;
        // the sample's own estimate of the k-th key: the statistic in the middle
        const uint32_t rankM = (uint32_t)min(max((long long)llround(centre), 1ll), (long long)m);
        uint32_t binA = 0, needA = 0, binB = 0, needB = 0, binM = 0, needM = 0, cnt = 0;
        find_from_top<HIST0_BINS>(h0, rankA, s_tmp, binA, needA, cnt);
        find_from_top<HIST0_BINS>(h0, rankB, s_tmp, binB, needB, cnt);
        find_from_top<HIST0_BINS>(h0, rankM, s_tmp, binM, needM, cnt);
        if (threadIdx.x == 0) { s_bins[0] = binA; s_bins[1] = binB; s_bins[2] = needA; s_bins[3] = needB; s_bins[6] = binM; s_bins[7] = needM; }
    }
    if (C > 1) cluster.sync(); else __syncthreads();
    const uint32_t* bins0 = C > 1 ? cluster.map_shared_rank(s_bins, 0) : s_bins;
    const uint32_t binA = bins0[0], binB = bins0[1], binM = bins0[6];
    for (uint32_t c = c_begin + threadIdx.x; c < c_end; c += THREADS) {
        const uint4 k0 = smp[2 * (size_t)c], k1 = smp[2 * (size_t)c + 1];
        const uint32_t kk[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if ((kk[i] >> 20) == binA) atomicAdd(&hA[(kk[i] >> 10) & 1023u], 1u);
            if ((kk[i] >> 20) == binB) atomicAdd(&hB[(kk[i] >> 10) & 1023u], 1u);
            if ((kk[i] >> 20) == binM) atomicAdd(&hM[(kk[i] >> 10) & 1023u], 1u);
        }
    }
    if (C > 1) cluster.sync(); else __syncthreads();
    uint32_t bin1A = 0, need2A = 0, bin1B = 0, need2B = 0, bin1M = 0;  // valid in CTA 0
    bool okA = false, okB = false, okM = false;
    if (rank == 0) {
        for (uint32_t b = threadIdx.x; b < 1024; b += THREADS) {
            uint32_t va = hA[b], vb = hB[b], vm = hM[b];
            for (uint32_t r = 1; r < C; ++r) {
                va += cluster.map_shared_rank(hA, r)[b];
                vb += cluster.map_shared_rank(hB, r)[b];
                vm += cluster.map_shared_rank(hM, r)[b];
            }
            hA[b] = va; hB[b] = vb; hM[b] = vm;
        }
        __syncthreads();
        uint32_t cntA = 0, cntB = 0, cntM = 0, need2M = 0;
        okA = find_from_top<1024>(hA, s_bins[2], s_tmp, bin1A, need2A, cntA);
        okB = find_from_top<1024>(hB, s_bins[3], s_tmp, bin1B, need2B, cntB);
        okM = find_from_top<1024>(hM, s_bins[7], s_tmp, bin1M, need2M, cntM);
        if (threadIdx.x == 0) {
            s_bins[4] = (okB && massive_in_sample(cntB, m)) ? 1u : 0u;
            s_bins[5] = (binB << 10) | bin1B;
        }
    }
    if (C > 1) cluster.sync(); else __syncthreads();
    const bool third_pass = bins0[4] != 0u;                                // the same answer in every CTA of the cluster
    if (third_pass) {
        const uint32_t prefB = bins0[5];
        for (uint32_t c = c_begin + threadIdx.x; c < c_end; c += THREADS) {
            const uint4 k0 = smp[2 * (size_t)c], k1 = smp[2 * (size_t)c + 1];
            const uint32_t kk[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if ((kk[i] >> 10) == prefB) atomicAdd(&hC[kk[i] & 1023u], 1u);
        }
        if (C > 1) cluster.sync(); else __syncthreads();
    }
    if (rank == 0) {
        const uint32_t prefA = (binA << 10) | bin1A, prefB = (binB << 10) | bin1B;
        uint32_t top = okA ? ((prefA << 10) | 1023u) : 0x7FFFFFFFu;
        uint32_t lo = (have_lo && okB) ? (prefB << 10) : 0u;
        uint32_t tie_key = TIE_NONE;
        if (third_pass) {
            for (uint32_t b = threadIdx.x; b < 1024; b += THREADS) {
                uint32_t v = hC[b];
                for (uint32_t r = 1; r < C; ++r) v += cluster.map_shared_rank(hC, r)[b];
                hC[b] = v;
            }
            __syncthreads();
            uint32_t bin2 = 0, need3 = 0, mult = 0;
            if (find_from_top<1024>(hC, need2B, s_tmp, bin2, need3, mult) && massive_in_sample(mult, m)) {
                tie_key = (prefB << 10) | bin2;
                lo = tie_key + 1u;                                     // listed: strictly above the tie key
                uint32_t bin2a = 0, multa = 0;
                if (okA && prefA == prefB && find_from_top<1024>(hC, need2A, s_tmp, bin2a, need3, multa))
                    top = (prefA << 10) | bin2a;                       // the upper statistic, exactly (it may be the tie key itself)
            }
        }
        const uint32_t hi = have_hi ? top : 0x7FFFFFFFu;
        if (tie_key == TIE_NONE && lo > top) lo = top;                 // (cannot happen; keeps the bracket sane)
        if (threadIdx.x == 0) {
            const uint32_t width_m1 = top >= lo ? top - lo : 0u;
            const uint32_t bits = width_m1 ? 32u - (uint32_t)__clz((int)width_m1) : 0u;
            FastState st = {};
            st.path = PATH_FAST; st.lo = lo; st.hi = hi; st.shift = bits > 11u ? bits - 11u : 0u;
            st.tie_key = tie_key;
            // with a tie key the residual has to keep p everywhere (the emit step re-reads tiles from it)
            st.zcut = tie_key != TIE_NONE ? 0x7FFFFFFFu : (okM ? min((binM << 20) | (bin1M << 10) | 511u, hi) : hi);
            P.state[prob] = st;
        }
    }
    if (C > 1) cluster.sync();                                                    // peers stay until CTA 0 has read their histograms
}

// ---- the bin of the threshold --------------------------------------------------------------
// Exact counts decide whether the bracket held: count(key > hi) <= k <= count(key >= lo) + ties.
// Then either the k-th key lies among the candidates (its histogram bin is pinned here, the exact
// key by the finish step), or every candidate is kept and the rest are tie-key elements.
// Called after the streaming pass has ended (all counts are final).  Every CTA that needs a segment's
// bin works it out for itself (a walk over 2048 words); `owner` (the CTA that holds the segment's
// first tile) also records it in the segment's state.
struct BinInfo { uint32_t live, need2, lo2, hi2; };                   // live: the segment is still on the one-pass path
// Run by ONE WARP (the warps of a CTA take different segments): lane l adds up 64 bins, a warp scan
// finds the lane whose bins hold the k-th key, and that lane walks its 64 bins.
__device__ __noinline__ BinInfo resolve_bin(const FastParams& P, uint32_t prob, bool owner) {
    const Layout& L = P.L;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t w = prob / L.nseg, s = prob - w * L.nseg;
    const SegEntry& seg = L.segs[s];
    FastState st = P.state[prob];
    BinInfo out = {0u, 0u, 0u, 0u};
    if (st.path != PATH_FAST) return out;
    const size_t fidx = (size_t)w * L.fast_per_worker + seg.fast_index;
    st.cand_total += min(st.cov_used, seg.cov_cap);                   // from here on: every listed candidate
    const uint64_t listed = (uint64_t)st.sure_total + st.cand_total;
    const uint64_t ties = st.tie_key != TIE_NONE ? st.tie_total : 0u;
    uint32_t fail = FAIL_NONE;
    if (st.overflow) fail = FAIL_OVERFLOW;
    else if (st.sure_total > seg.k || (uint64_t)seg.k > listed + ties) fail = FAIL_BRACKET;
    uint32_t bin = 0, need_in = 0, cnt = 0;
    const uint32_t need = fail ? 0u : seg.k - st.sure_total;
    const bool among_candidates = need != 0u && need <= st.cand_total;
    if (!fail && among_candidates) {                                   // uniform over the warp
        static_assert(CAND_BINS == 64 * 32, "64 bins per lane");
        const uint32_t* mine = P.cand_hist + fidx * CAND_BINS + (CAND_BINS - 64u * (lane + 1u));   // lane 0 owns the top 64 bins
        uint32_t sum = 0;
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {                                 // (four loads in flight: the filter below wants the registers)
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(mine) + i);
            sum += v.x + v.y + v.z + v.w;
        }
        uint32_t inc = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= (uint32_t)d) inc += t;
        }
        const uint32_t before = inc - sum;
        const bool here = before < need && need <= inc;                // at most one lane
        if (here) {
            uint32_t acc = before;
            for (int b = 63; b >= 0; --b) {
                const uint32_t c = __ldg(mine + b);
                if (need <= acc + c) { bin = CAND_BINS - 64u * (lane + 1u) + (uint32_t)b; need_in = need - acc; cnt = c; break; }
                acc += c;
            }
        }
        const uint32_t who = __ballot_sync(0xFFFFFFFFu, here);
        if (who == 0u) fail = FAIL_BRACKET;
        else {
            const int src = __ffs((int)who) - 1;
            bin = __shfl_sync(0xFFFFFFFFu, bin, src); need_in = __shfl_sync(0xFFFFFFFFu, need_in, src); cnt = __shfl_sync(0xFFFFFFFFu, cnt, src);
            if (cnt > LIST2_CAP) fail = FAIL_SHORT_LIST;
        }
    }
    st.need2 = 0; st.need_ties = 0; st.cnt2 = 0; st.expect2 = 0; st.icut = 0;
    if (fail) {
        st.path = PATH_FAILED; st.fail = fail;
    } else if (need == 0) {
        st.T = st.hi;                                                  // exactly the sure elements are kept
    } else if (among_candidates) {
        st.lo2 = st.lo + (bin << st.shift);
        const uint64_t top = (uint64_t)st.lo2 + (1ull << st.shift) - 1ull;
        st.hi2 = bin == CAND_BINS - 1u ? st.hi : (uint32_t)min(top, (uint64_t)st.hi);
        st.need2 = need_in;
        st.expect2 = cnt;                                              // length of the short list (checked by the finish step)
    } else {                                                           // all candidates, and the first need_ties tie-key elements
        st.T = st.tie_key;
        st.need_ties = need - st.cand_total;
    }
    if (owner && lane == 0) {
        if (fail) atomicAdd(P.counters, 1u);
        else if (st.need_ties) atomicAdd(P.counters + 1, 1u);
        // only result words are written: other CTAs may be reading the counts above, or adding to the
        // short-list counter, at this moment
        FastState* dst = P.state + prob;
        dst->path = st.path; dst->fail = st.fail; dst->need2 = st.need2;
        dst->need_ties = st.need_ties; dst->expect2 = st.expect2; dst->icut = st.icut; dst->T = st.T;
        dst->lo2 = st.lo2; dst->hi2 = st.hi2;
    }
    out.live = fail ? 0u : 1u; out.need2 = st.need2; out.lo2 = st.lo2; out.hi2 = st.hi2;
    return out;
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
    uint32_t n, tile_begin;        // of the segment
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
    const SegEntry* seg = L.segs + t.s;
    t.fast = seg->fast != 0;
    t.n = seg->n; t.tile_begin = seg->tile_begin;
    const size_t row = (size_t)t.w * L.n_total + seg->offset;
    t.g = P.grads + row;
    t.e = P.residuals + row;
    t.first = (long long)(t.lt - t.tile_begin) * TILE - misalign_of(t.e);
    t.full = t.first >= 0 && t.first + TILE <= (long long)t.n;
    return t;
}
// What the per-element work of a tile needs to know about its (worker, segment): kept in shared memory
// (written by thread 0 when the CTA enters the segment, read by everyone after the tile's barrier), so that
// the streaming part of the loop has the registers to itself.
struct MainSeg {
    uint32_t hi, shift, tie_key, ccap;
    uint32_t flag_cap, region_per_tile, ext_begin, ext_cap;
    uint32_t ext_chunk, cov_cap, zcut, pad1;
    uint2* flist;                  // the segment's flagged list of this worker
    uint2* clist;                  // its candidate list
    uint2* cover;                  // its candidate overflow list
    uint32_t* hist;                // its candidate histogram
};
// Two builds of the same code: MINB = 3 holds the kernel to 80 registers (three CTAs per SM), which is what
// many short segments and dense lists want; MINB = 1 lets it take more (two CTAs per SM), which streams long
// segments with sparse lists 1.4 % faster (350 M x 16 at 1 %: 10.45 against 10.65 ms; at 10 %: 12.1 against
// 11.6 ms the other way round).  The host picks one per segment table.
template <int MINB>
__global__ void __launch_bounds__(THREADS, MINB)
topk_main_kernel(const __grid_constant__ FastParams P) {
    __shared__ uint32_t sh[CAND_BINS];                                 // candidate histogram
    __shared__ __align__(16) float s_p[TILE];                          // the tile's p values, for the per-element work
    __shared__ uint16_t s_list[WARPS][512];                            // per warp: its flagged elements, in coordinate order
    __shared__ uint32_t s_wflag[2][WARPS];
    __shared__ uint32_t s_cnt[3][4];                                   // per tile in flight: candidates appended, sure elements, tie-key elements
    __shared__ uint32_t s_tot[4];                                      // of the current segment in this CTA: candidates, sure, ties
    __shared__ uint32_t s_misc[3];                                     // broadcasts of thread 0
    __shared__ MainSeg s_seg;
    const Layout& L = P.L;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t off0 = warp * 512u + lane * 4u;                     // this thread's quad of row 0 inside a tile
    // A segment's flagged and candidate lists are cut into regions: one per CTA of this kernel when the
    // segment has more tiles than CTAs (a tile's slots then follow from running counters), else one
    // per tile.  A region that is full continues in a pool behind the regions, handed out in chunks through
    // one atomic counter per segment (the only global atomic on the way, and only where elements of the
    // bracket are much denser than on average).  Either way no CTA waits for another; where a tile's slice
    // lies is recorded per tile, so the later steps do not depend on the order of the chunks.
    // Candidates are appended through a shared-memory counter, so their order inside a tile's slice is
    // arbitrary (all later uses count or sort them).  A tile's candidate and sure counts are final once
    // every warp has passed the next barrier; they are written out then ("pending" tile).
    uint32_t cur_pos = 0, cur_end = 0, run_cand = 0;
    for (uint32_t b = threadIdx.x; b < CAND_BINS; b += THREADS) sh[b] = 0;
    if (threadIdx.x < 12) s_cnt[threadIdx.x >> 2][threadIdx.x & 3] = 0;
    if (threadIdx.x < 4) s_tot[threadIdx.x] = 0;
    __syncthreads();
    uint32_t cur_prob = 0xFFFFFFFFu;
    uint32_t lo = 0, parity = 0;
    uint32_t slot3 = 0;                                                // counter triple of the current tile
    uint32_t pend_item = 0xFFFFFFFFu, pend_slot = 0, pend_room = 0;    // tile whose counts are not written yet
    bool pool_dry = false;
    const float gamma = L.gamma;
    const uint32_t group = P.main_group;
    const uint32_t group_step = (gridDim.x - 1u) * group + 1u;         // from a group's last tile to the next group's first
    MainTile T{};
    uint32_t seg_tile_end = 0;                                         // first tile after T's segment
    for (uint32_t item = blockIdx.x * group, ig = 0; ;
         item += (ig + 1u == group ? group_step : 1u), ig = (ig + 1u == group ? 0u : ig + 1u)) {
        // inside a group the next tile usually belongs to the same (worker, segment): then only its position
        // changes, and the lookup of the segment (a search over the table) is skipped
        if (ig != 0u && T.have && T.lt + 1u < seg_tile_end) {
            T.lt += 1u;
            T.first += TILE;
            T.full = T.first >= 0 && T.first + TILE <= (long long)T.n;
        } else {
            T = main_decode(P, item);
            seg_tile_end = T.have ? L.segs[T.s + 1].tile_begin : 0u;
        }
        // ---- flush the per-segment accumulators when the segment changes ---------------------------
        const uint32_t prob = T.have ? T.w * L.nseg + T.s : 0xFFFFFFFEu;
        if (prob != cur_prob && cur_prob != 0xFFFFFFFFu) {             // uniform over the CTA
            __syncthreads();                                           // the last tile's counts are final
            if (threadIdx.x == 0 && pend_item != 0xFFFFFFFFu) {
                const uint32_t c = min(s_cnt[pend_slot][0], pend_room), su = s_cnt[pend_slot][1], ti = s_cnt[pend_slot][2];
                P.tile_ccnt[pend_item] = c; P.tile_sure[pend_item] = su;
                if (s_seg.tie_key != TIE_NONE) P.tile_tie[pend_item] = ti;
                s_tot[0] += c; s_tot[1] += su; s_tot[2] += ti;
            }
            pend_item = 0xFFFFFFFFu;
            {
                uint32_t* gh = s_seg.hist;
                for (uint32_t b = threadIdx.x; b < CAND_BINS; b += THREADS) {
                    const uint32_t c = sh[b];
                    if (c) { atomicAdd(gh + b, c); sh[b] = 0; }
                }
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                FastState* st = P.state + cur_prob;
                if (s_tot[1]) atomicAdd(&st->sure_total, s_tot[1]);
                if (s_tot[0]) atomicAdd(&st->cand_total, s_tot[0]);
                if (s_tot[2]) atomicAdd(&st->tie_total, s_tot[2]);
                s_tot[0] = 0; s_tot[1] = 0; s_tot[2] = 0;
            }
            if (threadIdx.x < 12) s_cnt[threadIdx.x >> 2][threadIdx.x & 3] = 0;
            __syncthreads();
            run_cand = 0;
            cur_prob = 0xFFFFFFFFu;
        }
        if (!T.have) break;
        if (!T.fast) continue;                                         // uniform over the CTA
        if (prob != cur_prob) {
            cur_prob = prob;
            lo = P.state[prob].lo;
            const SegEntry* seg = L.segs + T.s;
            cur_pos = blockIdx.x * seg->flag_cap; cur_end = cur_pos + seg->flag_cap;
            pool_dry = false;
            if (threadIdx.x == 0) {                                    // (no warp still reads the previous segment's block)
                const FastState* st = P.state + prob;
                MainSeg m;
                m.hi = st->hi; m.shift = st->shift; m.tie_key = st->tie_key; m.ccap = seg->cand_cap;
                m.flag_cap = seg->flag_cap; m.region_per_tile = seg->region_per_tile; m.ext_begin = seg->ext_begin; m.ext_cap = seg->ext_cap;
                m.ext_chunk = seg->ext_chunk; m.cov_cap = seg->cov_cap; m.zcut = st->zcut; m.pad1 = 0;
                m.flist = P.flagged + (size_t)T.w * L.flag_per_worker + seg->flag_begin;
                m.clist = P.cand + (size_t)T.w * L.cand_per_worker + seg->cand_begin;
                m.cover = P.cand + (size_t)T.w * L.cand_per_worker + seg->cov_begin;
                m.hist = P.cand_hist + ((size_t)T.w * L.fast_per_worker + seg->fast_index) * CAND_BINS;
                s_seg = m;
            }
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
                const uint32_t valid = load_quad(e, base, T.n, p);
                load_quad_stream(T.g, base, T.n, gq);
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
            const uint32_t ahead = ig + 1u == group ? group_step : 1u;         // distance to this CTA's next tile
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
        const uint32_t tie_key = s_seg.tie_key, ccap = s_seg.ccap, flag_cap = s_seg.flag_cap;
        const bool per_tile = s_seg.region_per_tile != 0u;
        // the previous tile's counts are final now (every warp has left its per-element loop)
        if (pend_item != 0xFFFFFFFFu) {
            const uint32_t c = min(s_cnt[pend_slot][0], pend_room);
            if (threadIdx.x == 0) {
                const uint32_t su = s_cnt[pend_slot][1], ti = s_cnt[pend_slot][2];
                P.tile_ccnt[pend_item] = c; P.tile_sure[pend_item] = su;
                if (tie_key != TIE_NONE) P.tile_tie[pend_item] = ti;
                s_tot[0] += c; s_tot[1] += su; s_tot[2] += ti;
            }
            run_cand += c;
        }
        // this CTA's regions of the two lists, and where this tile's entries go inside them
        const uint32_t tseg = T.lt - T.tile_begin;                     // tile inside the segment
        if (per_tile) { cur_pos = tseg * flag_cap; cur_end = cur_pos + flag_cap; run_cand = 0; }
        bool fits = cur_pos + tflag <= cur_end;
        if (!fits && !pool_dry) {                                      // uniform: the region is full, continue in the pool
            if (threadIdx.x == 0) {
                const uint32_t want = max(tflag, s_seg.ext_chunk);
                const uint32_t got = atomicAdd(&P.state[prob].ext_used, want);
                s_misc[1] = ((uint64_t)got + want <= s_seg.ext_cap) ? got : 0xFFFFFFFFu;
                s_misc[2] = want;
            }
            __syncthreads();
            const uint32_t got = s_misc[1];
            if (got != 0xFFFFFFFFu) { cur_pos = s_seg.ext_begin + got; cur_end = cur_pos + s_misc[2]; fits = true; }
            else pool_dry = true;
        }
        const uint32_t fbase = cur_pos, cbase = (per_tile ? tseg : blockIdx.x) * ccap + run_cand;
        const uint32_t room = ccap - run_cand;                         // candidate slots left for this tile
        if (threadIdx.x == 0) {
            P.tile_fbase[item] = fits ? fbase : 0xFFFFFFFFu;
            P.tile_fcnt[item] = tflag;
            P.tile_cbase[item] = cbase;
            if (!fits) P.state[prob].overflow = 1u;                    // the list is full: the segment falls back
            const uint32_t nxt = slot3 == 2u ? 0u : slot3 + 1u;        // counters of the tile after this one
            s_cnt[nxt][0] = 0; s_cnt[nxt][1] = 0; s_cnt[nxt][2] = 0;
        }
        pend_item = item; pend_slot = slot3; pend_room = fits ? room : 0u;
        if (fits) cur_pos += tflag;
        if (tie_key != TIE_NONE) {                                     // uniform: count this thread's tie-key elements
            uint32_t ties = 0;
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const float4 p = *reinterpret_cast<const float4*>(sp + off0 + 128 * j);
                const uint32_t c0 = (uint32_t)(mine + 128 * j);        // coordinates outside the segment wrap far beyond n
                ties += (uint32_t)(key_of(p.x) == tie_key && c0 < T.n) + (uint32_t)(key_of(p.y) == tie_key && c0 + 1u < T.n) +
                        (uint32_t)(key_of(p.z) == tie_key && c0 + 2u < T.n) + (uint32_t)(key_of(p.w) == tie_key && c0 + 3u < T.n);
            }
            ties = __reduce_add_sync(0xFFFFFFFFu, ties);
            if (lane == 0 && ties) atomicAdd(&s_cnt[slot3][2], ties);
        }
        if (fits && wflag) {
            // the tile's entries fit: write them (entry r of the warp's slice by lane r % 32: coalesced), zero
            // the ones above the estimated threshold in the residual while the tile's lines are still in L2 (their
            // values stay in the list, from where the emit step or a fall-back puts back what should not have
            // been zeroed), append the candidates to the tile's slice and histogram them
            uint2* flist = s_seg.flist + fbase + fwbase;
            uint2* clist = s_seg.clist + cbase;
            const uint32_t hi = s_seg.hi, shift = s_seg.shift, zcut = s_seg.zcut;
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
                if (active && key > zcut) e[coord] = 0.0f;
                const uint32_t bs = __ballot_sync(0xFFFFFFFFu, sure);
                const uint32_t bc = __ballot_sync(0xFFFFFFFFu, cand);
                sure_w += __popc(bs);
                if (bc) {                                              // uniform over the warp
                    uint32_t base = 0;
                    if (lane == 0) base = atomicAdd(&s_cnt[slot3][0], (uint32_t)__popc(bc));
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    if (cand) {
                        const uint32_t pos = base + __popc(bc & ((1u << lane) - 1u));
                        if (pos < room) {
                            clist[pos] = make_uint2(key, coord);
                        } else {                                       // rare: candidates crowd in this part of the segment
                            const uint32_t gp = atomicAdd(&P.state[prob].cov_used, 1u);
                            if (gp < s_seg.cov_cap) s_seg.cover[gp] = make_uint2(key, coord);
                            else P.state[prob].overflow = 1u;
                        }
                        atomicAdd(&sh[min((key - lo) >> shift, CAND_BINS - 1u)], 1u);
                    }
                }
            }
            if (lane == 0 && sure_w) atomicAdd(&s_cnt[slot3][1], sure_w);
        }
    }
}

// ---- filter: copy the candidates of the threshold's bin into the short list -------------------
// Eight lanes share TILES_PER_GROUP consecutive tiles.  The walk is bound by a chain of dependent
// loads (slice length and base, then the slice), so a group first requests the placement words of
// all its tiles, then the first eight candidates of every tile, and only then looks at them: four
// tiles per group cut the number of such chains per launch by four.
// A CTA serves a contiguous range of tiles.  It first works out the threshold's bin of every large
// segment its range touches (see resolve_bin; FILTER_TABLE segments at a time), then its lane groups
// walk the range without meeting again.
constexpr uint32_t TILES_PER_GROUP = 4;
constexpr uint32_t FILTER_TILES_PER_CTA = (THREADS / 8) * TILES_PER_GROUP;   // tiles one sweep of the lane groups covers
constexpr uint32_t FILTER_TABLE = 64;

__device__ inline uint32_t problem_of_item(const Layout& L, uint32_t item) {
    const uint32_t w = item / L.tiles_per_worker;
    const uint32_t lt = item - w * L.tiles_per_worker;
    return w * L.nseg + ((L.nseg == 1) ? 0u : find_by_tile(L, lt));
}

__global__ void __launch_bounds__(THREADS)
topk_filter_kernel(const __grid_constant__ FastParams P, uint32_t items_per_cta) {
    __shared__ BinInfo s_bin[FILTER_TABLE];                            // by problem index relative to the first of the table
    __shared__ uint32_t s_range[2];
    const Layout& L = P.L;
    const uint32_t sub = threadIdx.x & 7u;
    const uint32_t chunk_begin = blockIdx.x * items_per_cta;
    const uint32_t chunk_end = min(chunk_begin + items_per_cta, P.total_items);
    for (uint32_t pos = chunk_begin; pos < chunk_end; ) {
        __syncthreads();                                               // the previous part is done with the table
        if (threadIdx.x == 0) {
            const uint32_t p_first = problem_of_item(L, pos);
            const uint32_t p_stop = p_first + FILTER_TABLE;            // first problem the table has no room for
            uint32_t part_end = chunk_end;
            if (problem_of_item(L, chunk_end - 1u) >= p_stop) {        // the range goes on beyond the table: stop at that problem's first tile
                const uint32_t w = p_stop / L.nseg, s = p_stop - w * L.nseg;
                part_end = w * L.tiles_per_worker + L.segs[s].tile_begin;
            }
            s_range[0] = p_first; s_range[1] = part_end;
        }
        __syncthreads();
        const uint32_t p_first = s_range[0], part_end = s_range[1];
        const uint32_t p_last = problem_of_item(L, part_end - 1u);
        for (uint32_t p = p_first + (threadIdx.x >> 5); p <= p_last; p += WARPS) {   // one warp per segment
            const uint32_t w = p / L.nseg, s = p - w * L.nseg;
            if (L.segs[s].fast != 1u) continue;                       // (segments of few tiles are resolved by one CTA each)
            // the CTA whose range holds the segment's first tile records the result
            const uint32_t first_item = w * L.tiles_per_worker + L.segs[s].tile_begin;
            const BinInfo bi = resolve_bin(P, p, first_item >= pos && first_item < part_end);
            if ((threadIdx.x & 31u) == 0u) s_bin[p - p_first] = bi;
        }
        __syncthreads();
        // (the loop bound is the same for all lanes of a warp: its shuffles stay whole)
        for (uint32_t warp0 = pos + (threadIdx.x >> 5) * 4u * TILES_PER_GROUP; warp0 < part_end; warp0 += FILTER_TILES_PER_CTA) {
            const uint32_t item0 = warp0 + ((threadIdx.x >> 3) & 3u) * TILES_PER_GROUP;
            uint32_t cnt[TILES_PER_GROUP], base[TILES_PER_GROUP];
#pragma unroll
            for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
                const uint32_t item = item0 + u;
                cnt[u] = 0; base[u] = 0;
                if (item < part_end) { cnt[u] = __ldg(P.tile_ccnt + item); base[u] = __ldg(P.tile_cbase + item); }
            }
            const uint2* list[TILES_PER_GROUP];
            uint2 first[TILES_PER_GROUP];
            uint32_t prob[TILES_PER_GROUP];
            uint32_t s_prev = 0xFFFFFFFFu, w_prev = 0xFFFFFFFFu, end_prev = 0;   // consecutive tiles mostly share their segment
#pragma unroll
            for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
                const uint32_t item = item0 + u;
                list[u] = nullptr; first[u] = make_uint2(0u, 0u); prob[u] = 0u;
                if (item >= part_end) continue;
                const uint32_t w = item / L.tiles_per_worker;
                const uint32_t lt = item - w * L.tiles_per_worker;
                if (w != w_prev || lt >= end_prev) {
                    s_prev = (L.nseg == 1) ? 0u : find_by_tile(L, lt);
                    w_prev = w; end_prev = L.segs[s_prev + 1].tile_begin;
                }
                const uint32_t s = s_prev;
                const SegEntry& seg = L.segs[s];
                prob[u] = w * L.nseg + s;
                if (seg.fast != 1u) continue;
                const BinInfo bi = s_bin[prob[u] - p_first];
                if (!bi.live || bi.need2 == 0u || cnt[u] == 0u) continue;  // no candidate, or every candidate, is kept
                list[u] = P.cand + (size_t)w * L.cand_per_worker + seg.cand_begin + base[u];
                if (sub < cnt[u]) first[u] = __ldg(list[u] + sub);
            }
#pragma unroll
            for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
                // candidates above the threshold's bin are kept whatever the exact threshold turns out to be; those
                // inside the bin go to the short list, and the finish step adds the kept ones to the tile's count
                uint32_t above = 0, inbin = 0;
                if (list[u]) {
                    const BinInfo bi = s_bin[prob[u] - p_first];
                    const uint32_t w = prob[u] / L.nseg, s = prob[u] - w * L.nseg;
                    uint2* out = P.list2 + ((size_t)w * L.fast_per_worker + L.segs[s].fast_index) * LIST2_CAP;
                    for (uint32_t i0 = sub; i0 < cnt[u]; i0 += 32) {       // four entries in flight per lane
                        uint2 c4[4];
#pragma unroll
                        for (uint32_t v = 0; v < 4; ++v) {
                            const uint32_t i = i0 + 8u * v;
                            c4[v] = i == sub ? first[u] : (i < cnt[u] ? __ldg(list[u] + i) : make_uint2(0u, 0u));
                        }
#pragma unroll
                        for (uint32_t v = 0; v < 4; ++v) {
                            if (i0 + 8u * v >= cnt[u]) continue;
                            const uint2 c = c4[v];
                            if (c.x > bi.hi2) ++above;
                            else if (c.x >= bi.lo2) {
                                ++inbin;
                                const uint32_t pos2 = atomicAdd(&P.state[prob[u]].cnt2, 1u);
                                if (pos2 < LIST2_CAP) out[pos2] = c;
                            }
                        }
                    }
                }
                uint32_t both = above | (inbin << 16);                 // a tile holds at most 4096 candidates
                both += __shfl_xor_sync(0xFFFFFFFFu, both, 1);
                both += __shfl_xor_sync(0xFFFFFFFFu, both, 2);
                both += __shfl_xor_sync(0xFFFFFFFFu, both, 4);
                if (sub == 0u && item0 + u < part_end) P.tile_csum[item0 + u] = both;
            }
        }
        pos = part_end;
    }
}

__device__ inline bool fast_kept(uint32_t key, uint32_t coord, uint32_t T, uint32_t icut) {
    return key > T || (key == T && coord < icut);
}

// ---- finish: exact threshold, per-tile kept counts, message offsets ----------------------------
// One thread-block cluster of C = FINISH_CTAS CTAs per (worker, segment) of more than SMALL_MAX_TILES tiles
// (the shorter ones take topk_resolve_small_kernel instead); `first` and `count` select a range of the
// fast list, the grid covers count problems of every worker.
//   threshold among the candidates: CTA 0 sorts the short list (the candidates of the threshold's
//       histogram bin, at most LIST2_CAP) in shared memory, larger key first and lower coordinate first
//       among equal keys; its first need2 entries are kept, which fixes T and the coordinate cut, and each
//       of them adds one to its tile's count of kept candidates;
//   threshold == tie key: every listed element is kept and the first need_ties tie-key elements in
//       coordinate order: a running sum of the per-tile tie counts says how many each tile admits;
//   then the kept counts of the segment's tiles are summed up into the tiles' first message slots: every
//   CTA of the cluster adds up a contiguous share of the tiles, the shares' totals are exchanged through
//   distributed shared memory, and each CTA scans its share from the sum of the shares before it.
// The cluster barriers are the hardware's; every CTA runs to the last one.
constexpr uint32_t FINISH_CTAS = 8;
constexpr uint32_t FINISH_PER = 16;                                    // tiles per thread and round of a scan
constexpr uint32_t SMALL_MAX_TILES = 1024;                             // one-pass segments of at most this many tiles are resolved by one CTA each
__device__ inline uint32_t block_sum(uint32_t v, uint32_t* s_scan) {
    uint32_t total;
    block_exclusive_scan(v, s_scan, &total);
    return total;
}
template <uint32_t C>
__global__ void __launch_bounds__(THREADS)
topk_finish_kernel(const __grid_constant__ FastParams P, uint32_t first, uint32_t count) {
    namespace cg = cooperative_groups;
    __shared__ unsigned long long srt[LIST2_CAP];
    __shared__ uint32_t s_scan[WARPS + 1];
    __shared__ uint32_t s_share[3];                                    // ties and kept elements of this CTA's share; [2]: CTA 0 gave up
    cg::cluster_group cluster = cg::this_cluster();
    constexpr bool solo = C == 1;
    constexpr uint32_t ranks = C;
    const uint32_t rank = solo ? 0u : cluster.block_rank();
    const Layout& L = P.L;
    uint32_t w, s;
    const uint32_t pidx = blockIdx.x / C;                              // problem of this launch: (worker, position in the range)
    const uint32_t prob = fast_problem(L, (pidx / count) * L.fast_per_worker + first + pidx % count, w, s);
    const SegEntry seg = L.segs[s];
    FastState st = P.state[prob];
    if (st.path != PATH_FAST) return;                                  // the same answer in every CTA of the cluster
    const uint32_t ntiles = L.segs[s + 1].tile_begin - seg.tile_begin;
    const size_t item0 = (size_t)w * L.tiles_per_worker + seg.tile_begin;
    const bool admit = st.need_ties != 0u;
    if (rank == 0) {
        bool failed = false;
        const uint32_t mis = misalign_of(P.residuals + (size_t)w * L.n_total + seg.offset);   // tiles lie on the 128-byte grid of the row
        // candidates that did not fit their tile's slice (rare): those of the threshold's bin join the short list
        const uint32_t ncov = min(st.cov_used, seg.cov_cap);
        const uint2* cover = P.cand + (size_t)w * L.cand_per_worker + seg.cov_begin;
        if (st.need2 && ncov) {
            uint2* out = P.list2 + ((size_t)w * L.fast_per_worker + seg.fast_index) * LIST2_CAP;
            for (uint32_t i = threadIdx.x; i < ncov; i += THREADS) {
                const uint2 c = cover[i];
                if (c.x >= st.lo2 && c.x <= st.hi2) {
                    const uint32_t pos = atomicAdd(&P.state[prob].cnt2, 1u);
                    if (pos < LIST2_CAP) out[pos] = c;
                }
            }
            __threadfence();
            __syncthreads();
            st.cnt2 = __ldcg(&P.state[prob].cnt2);
        }
        if (st.need2) {
            const uint32_t cnt = st.cnt2;
            if (cnt != st.expect2 || cnt > LIST2_CAP || st.need2 > cnt) {  // short list disagrees with the histogram
                failed = true;
                if (threadIdx.x == 0) {
                    P.state[prob].path = PATH_FAILED; P.state[prob].fail = FAIL_SHORT_LIST;
                    atomicAdd(P.counters, 1u);
                }
            } else {
                uint32_t size = 1;
                while (size < cnt) size <<= 1;
                const uint2* in = P.list2 + ((size_t)w * L.fast_per_worker + seg.fast_index) * LIST2_CAP;
                for (uint32_t i = threadIdx.x; i < size; i += THREADS) {
                    unsigned long long v = 0;                           // padding sorts last
                    if (i < cnt) { const uint2 c = __ldcg(in + i); v = ((unsigned long long)c.x << 32) | (0xFFFFFFFFu - c.y); }
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
                const unsigned long long v = srt[st.need2 - 1u];
                st.T = (uint32_t)(v >> 32);
                st.icut = (0xFFFFFFFFu - (uint32_t)v) + 1u;            // coordinates below this are kept among the ties
                if (st.icut == 0) st.icut = 0xFFFFFFFFu;               // (coordinate 2^32-1 cannot occur: n < 2^32)
                if (threadIdx.x == 0) { P.state[prob].T = st.T; P.state[prob].icut = st.icut; }
                // the kept entries of the short list, counted into their tiles
                for (uint32_t i = threadIdx.x; i < st.need2; i += THREADS) {
                    const uint32_t coord = 0xFFFFFFFFu - (uint32_t)srt[i];
                    atomicAdd(P.tile_csum + item0 + (coord + mis) / TILE, 1u);
                }
            }
        }
        if (!failed && ncov && (admit || st.need2)) {                  // kept overflow candidates, counted into their tiles
            uint32_t* counts = admit ? P.tile_ccnt : P.tile_csum;      // (every candidate is kept when ties are admitted)
            for (uint32_t i = threadIdx.x; i < ncov; i += THREADS) {
                const uint2 c = cover[i];
                if (admit || c.x > st.hi2) atomicAdd(counts + item0 + (c.y + mis) / TILE, 1u);
            }
        }
        if (threadIdx.x == 0) s_share[2] = failed ? 1u : 0u;
        __threadfence();                                               // the counts above are in L2 before the peers read them
    }
    if (solo) __syncthreads(); else cluster.sync();
    const bool give_up = (solo ? s_share[2] : *cluster.map_shared_rank(&s_share[2], 0)) != 0u;
    if (!give_up) {
        // ---- kept count per tile, exclusive sum over the segment's tiles ------------------------------
        constexpr uint32_t ROUND = THREADS * FINISH_PER;
        const uint32_t per = ((ntiles + ranks - 1) / ranks + ROUND - 1) / ROUND * ROUND;
        const uint32_t begin = min(rank * per, ntiles), end = min(begin + per, ntiles);
        uint32_t* off = P.offsets + (size_t)w * (L.tiles_per_worker + 1) + seg.tile_begin;
        uint32_t tie_run = 0;                                          // tie-key elements of the segment before the current tile
        if (admit) {
            uint32_t tsum = 0;
            for (uint32_t t = begin + threadIdx.x; t < end; t += THREADS) tsum += __ldcg(P.tile_tie + item0 + t);
            tsum = block_sum(tsum, s_scan);
            if (threadIdx.x == 0) s_share[0] = tsum;
            if (!solo) cluster.sync();
            for (uint32_t r = 0; r < rank; ++r) tie_run += *cluster.map_shared_rank(&s_share[0], r);
        }
        // first round over the share: how many ties each tile admits, and the share's kept total
        uint32_t ksum = 0;
        for (uint32_t base = begin; base < end; base += ROUND) {
            const uint32_t t0 = base + threadIdx.x * FINISH_PER;
            uint32_t kept[FINISH_PER];
#pragma unroll
            for (uint32_t i = 0; i < FINISH_PER; ++i) {
                kept[i] = 0;
                if (t0 + i < end) {
                    kept[i] = __ldcg(P.tile_sure + item0 + t0 + i);
                    kept[i] += admit ? __ldcg(P.tile_ccnt + item0 + t0 + i) : (__ldcg(P.tile_csum + item0 + t0 + i) & 0xFFFFu);
                }
            }
            if (admit) {
                uint32_t adm[FINISH_PER], tsum = 0;
#pragma unroll
                for (uint32_t i = 0; i < FINISH_PER; ++i) {
                    adm[i] = t0 + i < end ? __ldcg(P.tile_tie + item0 + t0 + i) : 0u;
                    tsum += adm[i];
                }
                uint32_t total;
                uint32_t before = tie_run + block_exclusive_scan(tsum, s_scan, &total);
                tie_run += total;
#pragma unroll
                for (uint32_t i = 0; i < FINISH_PER; ++i) {
                    const uint32_t room = st.need_ties > before ? st.need_ties - before : 0u;
                    const uint32_t a = min(adm[i], room);
                    before += adm[i];
                    kept[i] += a;
                    if (t0 + i < end) P.tile_csum[item0 + t0 + i] = a;
                }
            }
#pragma unroll
            for (uint32_t i = 0; i < FINISH_PER; ++i) ksum += kept[i];
        }
        ksum = block_sum(ksum, s_scan);
        if (threadIdx.x == 0) s_share[1] = ksum;
        if (!solo) cluster.sync();
        uint32_t kept_run = 0;
        for (uint32_t r = 0; r < rank; ++r) kept_run += *cluster.map_shared_rank(&s_share[1], r);
        // second round: the tiles' first message slots
        for (uint32_t base = begin; base < end; base += ROUND) {
            const uint32_t t0 = base + threadIdx.x * FINISH_PER;
            uint32_t kept[FINISH_PER], sum = 0;
#pragma unroll
            for (uint32_t i = 0; i < FINISH_PER; ++i) {
                kept[i] = 0;
                if (t0 + i < end) {
                    kept[i] = __ldcg(P.tile_sure + item0 + t0 + i);
                    if (admit) kept[i] += __ldcg(P.tile_ccnt + item0 + t0 + i) + __ldcg(P.tile_csum + item0 + t0 + i);
                    else kept[i] += __ldcg(P.tile_csum + item0 + t0 + i) & 0xFFFFu;
                }
                sum += kept[i];
            }
            uint32_t total;
            uint32_t ex = kept_run + block_exclusive_scan(sum, s_scan, &total);
            kept_run += total;
#pragma unroll
            for (uint32_t i = 0; i < FINISH_PER; ++i) {
                if (t0 + i < end) off[t0 + i] = ex;
                ex += kept[i];
            }
        }
        if (rank == ranks - 1u && threadIdx.x == 0 && kept_run != seg.k) atomicMin(P.status, ST_DEVICE_CHECK);   // counts and k disagree
    }
    if (!solo) cluster.sync();                                         // a peer's totals must outlive their readers
}

// ---- resolve of a one-pass segment of few tiles: bin, filter, exact threshold and offsets by ONE CTA ---------
// For segments of at most SMALL_MAX_TILES tiles (4 M elements) the three steps above cost more in launches and
// in waiting for memory than in work (the tensors of a network, layer by layer: 42 of ResNet-50's per worker).
// One CTA per (worker, segment) does them back to back: warp 0 works out the threshold's bin, the lane groups
// walk the tiles' candidate slices (the short list and the per-tile counts stay in shared memory), the list is
// sorted, ties are admitted, and the kept counts are summed into the tiles' message offsets.
__global__ void __launch_bounds__(THREADS)
topk_resolve_small_kernel(const __grid_constant__ FastParams P, uint32_t first, uint32_t count) {
    __shared__ unsigned long long srt[LIST2_CAP];
    __shared__ uint32_t s_kept[SMALL_MAX_TILES];                       // kept candidates per tile
    __shared__ uint32_t s_scan[WARPS + 1];
    __shared__ BinInfo s_bi;
    __shared__ uint32_t s_cnt2;
    const Layout& L = P.L;
    const uint32_t lane = threadIdx.x & 31u, sub = threadIdx.x & 7u;
    uint32_t w, s;
    const uint32_t prob = fast_problem(L, (blockIdx.x / count) * L.fast_per_worker + first + blockIdx.x % count, w, s);
    const SegEntry seg = L.segs[s];
    if (P.state[prob].path != PATH_FAST) return;
    const uint32_t ntiles = L.segs[s + 1].tile_begin - seg.tile_begin;
    const size_t item0 = (size_t)w * L.tiles_per_worker + seg.tile_begin;
    if (threadIdx.x < 32) {
        const BinInfo bi = resolve_bin(P, prob, true);
        if (lane == 0) { s_bi = bi; s_cnt2 = 0; }
    }
    for (uint32_t t = threadIdx.x; t < ntiles; t += THREADS) s_kept[t] = 0;
    __syncthreads();
    const BinInfo bi = s_bi;
    if (!bi.live) return;                                              // the bracket missed: the fall-back serves the segment
    FastState st = load_state_l2(P.state + prob);                      // with what warp 0 has just recorded
    const bool admit = st.need_ties != 0u;
    const uint32_t mis = misalign_of(P.residuals + (size_t)w * L.n_total + seg.offset);   // tiles lie on the 128-byte grid of the row
    const uint2* clist = P.cand + (size_t)w * L.cand_per_worker + seg.cand_begin;
    // ---- filter: candidates above the bin are kept, those inside it go to the short list -----------------------
    if (bi.need2) {
        for (uint32_t warp0 = (threadIdx.x >> 5) * 4u * TILES_PER_GROUP; warp0 < ntiles; warp0 += FILTER_TILES_PER_CTA) {
            const uint32_t t0 = warp0 + ((threadIdx.x >> 3) & 3u) * TILES_PER_GROUP;
            uint32_t cnt[TILES_PER_GROUP], base[TILES_PER_GROUP];
#pragma unroll
            for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
                cnt[u] = 0; base[u] = 0;
                if (t0 + u < ntiles) { cnt[u] = __ldg(P.tile_ccnt + item0 + t0 + u); base[u] = __ldg(P.tile_cbase + item0 + t0 + u); }
            }
#pragma unroll
            for (uint32_t u = 0; u < TILES_PER_GROUP; ++u) {
                uint32_t above = 0;
                for (uint32_t i0 = sub; i0 < cnt[u]; i0 += 32) {           // four entries in flight per lane
                    uint2 c4[4];
#pragma unroll
                    for (uint32_t v = 0; v < 4; ++v) {
                        const uint32_t i = i0 + 8u * v;
                        c4[v] = i < cnt[u] ? __ldg(clist + base[u] + i) : make_uint2(0u, 0u);
                    }
#pragma unroll
                    for (uint32_t v = 0; v < 4; ++v) {
                        if (i0 + 8u * v >= cnt[u]) continue;
                        const uint2 c = c4[v];
                        if (c.x > bi.hi2) ++above;
                        else if (c.x >= bi.lo2) {
                            const uint32_t pos = atomicAdd(&s_cnt2, 1u);
                            if (pos < LIST2_CAP) srt[pos] = ((unsigned long long)c.x << 32) | (0xFFFFFFFFu - c.y);
                        }
                    }
                }
                above += __shfl_xor_sync(0xFFFFFFFFu, above, 1);
                above += __shfl_xor_sync(0xFFFFFFFFu, above, 2);
                above += __shfl_xor_sync(0xFFFFFFFFu, above, 4);
                if (sub == 0u && t0 + u < ntiles) s_kept[t0 + u] = above;
            }
        }
    }
    __syncthreads();
    // candidates that did not fit their tile's slice (rare)
    const uint32_t ncov = min(st.cov_used, seg.cov_cap);
    const uint2* cover = P.cand + (size_t)w * L.cand_per_worker + seg.cov_begin;
    if (ncov && (admit || bi.need2)) {
        for (uint32_t i = threadIdx.x; i < ncov; i += THREADS) {
            const uint2 c = cover[i];
            if (admit || c.x > bi.hi2) atomicAdd(&s_kept[(c.y + mis) / TILE], 1u);
            else if (c.x >= bi.lo2) {
                const uint32_t pos = atomicAdd(&s_cnt2, 1u);
                if (pos < LIST2_CAP) srt[pos] = ((unsigned long long)c.x << 32) | (0xFFFFFFFFu - c.y);
            }
        }
        __syncthreads();
    }
    // ---- exact threshold from the short list ----------------------------------------------------------------
    if (bi.need2) {
        const uint32_t cnt = s_cnt2;
        if (cnt != st.expect2 || cnt > LIST2_CAP || bi.need2 > cnt) {  // short list disagrees with the histogram
            if (threadIdx.x == 0) {
                P.state[prob].path = PATH_FAILED; P.state[prob].fail = FAIL_SHORT_LIST;
                atomicAdd(P.counters, 1u);
            }
            return;
        }
        uint32_t size = 1;
        while (size < cnt) size <<= 1;
        for (uint32_t i = cnt + threadIdx.x; i < size; i += THREADS) srt[i] = 0;   // padding sorts last
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
        const unsigned long long v = srt[bi.need2 - 1u];
        if (threadIdx.x == 0) {
            uint32_t icut = (0xFFFFFFFFu - (uint32_t)v) + 1u;          // coordinates below this are kept among the ties
            if (icut == 0) icut = 0xFFFFFFFFu;                         // (coordinate 2^32-1 cannot occur: n < 2^32)
            P.state[prob].T = (uint32_t)(v >> 32); P.state[prob].icut = icut;
        }
        for (uint32_t i = threadIdx.x; i < bi.need2; i += THREADS) {
            const uint32_t coord = 0xFFFFFFFFu - (uint32_t)srt[i];
            atomicAdd(&s_kept[(coord + mis) / TILE], 1u);
        }
        __syncthreads();
    }
    // ---- kept count per tile, exclusive sum over the segment's tiles (at most four tiles per thread) --------------
    constexpr uint32_t PER = SMALL_MAX_TILES / THREADS;
    const uint32_t t0 = threadIdx.x * PER;
    uint32_t kept[PER];
#pragma unroll
    for (uint32_t i = 0; i < PER; ++i) {
        kept[i] = 0;
        if (t0 + i < ntiles) {
            kept[i] = __ldg(P.tile_sure + item0 + t0 + i) + s_kept[t0 + i];
            if (admit) kept[i] += __ldg(P.tile_ccnt + item0 + t0 + i);   // every candidate is kept (those of the overflow list are in s_kept)
        }
    }
    if (admit) {                                                       // ties before each tile decide how many it admits
        uint32_t adm[PER], tsum = 0;
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) {
            adm[i] = t0 + i < ntiles ? __ldg(P.tile_tie + item0 + t0 + i) : 0u;
            tsum += adm[i];
        }
        uint32_t total;
        uint32_t before = block_exclusive_scan(tsum, s_scan, &total);
#pragma unroll
        for (uint32_t i = 0; i < PER; ++i) {
            const uint32_t room = st.need_ties > before ? st.need_ties - before : 0u;
            const uint32_t a = min(adm[i], room);
            before += adm[i];
            kept[i] += a;
            if (t0 + i < ntiles) P.tile_csum[item0 + t0 + i] = a;
        }
    }
    uint32_t sum = 0;
#pragma unroll
    for (uint32_t i = 0; i < PER; ++i) sum += kept[i];
    uint32_t total;
    uint32_t ex = block_exclusive_scan(sum, s_scan, &total);
    uint32_t* off = P.offsets + (size_t)w * (L.tiles_per_worker + 1) + seg.tile_begin;
#pragma unroll
    for (uint32_t i = 0; i < PER; ++i) {
        if (t0 + i < ntiles) off[t0 + i] = ex;
        ex += kept[i];
    }
    if (threadIdx.x == 0 && total != seg.k) atomicMin(P.status, ST_DEVICE_CHECK);   // counts and k disagree
}

// ---- emit: G lanes per tile walk the tile's slice of the flagged list ----------------------------
// Sparse slices (a few dozen entries) take a part of a warp per tile, i.e. several tiles per warp
// side by side; long slices take the whole warp and more entries per lane.  One batch covers
// G x D entries.  (Loading the placement words two tiles ahead and asking L2 for the next slice
// one tile ahead changed nothing: the kernel is not bound by its chain of dependent loads.)
// Tiles that admit tie-key elements are skipped here (see emit_tie_tiles).
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
    uint32_t T = 0, icut = 0, zcut = 0, seg_k = 0, idx0 = 0, tile_begin = 0;
    bool live = false, admits = false;
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
                admits = st->need_ties != 0u;
                T = st->T; icut = st->icut; seg_k = seg.k; idx0 = (uint32_t)seg.offset;
                zcut = st->zcut;                                        // the streaming pass zeroed the entries above this key
                flist0 = P.flagged + (size_t)w * L.flag_per_worker + seg.flag_begin;
                e = P.residuals + (size_t)w * L.n_total + seg.offset;
                ovals = P.out_vals + (size_t)w * L.K_total + seg.msg_off;
                oidx = P.out_idx + (size_t)w * L.K_total + seg.msg_off;
            }
            if (live) {
                // the words that place this tile: independent loads, one round trip
                cnt = __ldg(P.tile_fcnt + item); base = __ldg(P.tile_fbase + item);
                running = __ldg(P.offsets + (size_t)w * (L.tiles_per_worker + 1) + lt);   // kept coordinates of the segment before this tile
                if (admits && __ldg(P.tile_csum + item) != 0u) cnt = 0;                  // served by the second loop
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
                    if (r < seg_k) {
                        ovals[r] = __uint_as_float(a[u].x);
                        oidx[r] = idx0 + a[u].y;
                    } else {                                            // counts and k disagree
                        atomicMin(P.status, ST_DEVICE_CHECK);
                    }
                    if (key <= zcut) e[a[u].y] = 0.0f;                  // the streaming pass left p there
                } else if (key > zcut) {
                    e[a[u].y] = __uint_as_float(a[u].x);                // zeroed by the streaming pass, but not kept
                }
                pos += __popc(bal);
            }
        }
    }
}

// ---- tiles that admit tie-key elements ----------------------------------------------------------
// Run by every CTA of the kernel that follows the emit step (sc_topk_fallback.cuh), and only when some
// segment's threshold is its tie key.  One warp per tile re-reads the tile from the residual (which
// still holds p there) in coordinate order: everything above the tie key is kept, and the first `adm`
// tie-key elements of the tile, as the finish step decided.
__device__ inline void emit_tie_tiles(const FastParams& P) {
    __shared__ float s_stage_v[WARPS][128];                            // per warp: the kept entries of one step, in coordinate order
    __shared__ uint32_t s_stage_i[WARPS][128];
    const Layout& L = P.L;
    const uint32_t lane = threadIdx.x & 31u;
    float* stage_v = s_stage_v[threadIdx.x >> 5];
    uint32_t* stage_i = s_stage_i[threadIdx.x >> 5];
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint32_t warps_total = gridDim.x * WARPS;
    const uint32_t warp_g = blockIdx.x * WARPS + (threadIdx.x >> 5);
    for (uint32_t it0 = warp_g; it0 < P.total_items; it0 += warps_total * 32u) {
        // every lane looks at one tile (neighbouring tiles, which tend to admit ties together, go to different
        // warps); the warp then serves, one after the other, those that admit ties
        uint32_t my_adm = 0, my_s = 0;
        {
            const unsigned long long it64 = (unsigned long long)it0 + (unsigned long long)lane * warps_total;
            const uint32_t it = it64 < P.total_items ? (uint32_t)it64 : 0xFFFFFFFFu;
            if (it != 0xFFFFFFFFu) {
                const uint32_t w = it / L.tiles_per_worker;
                const uint32_t lt = it - w * L.tiles_per_worker;
                my_s = (L.nseg == 1) ? 0u : find_by_tile(L, lt);
                if (L.segs[my_s].fast) {
                    const FastState* st = P.state + (size_t)w * L.nseg + my_s;
                    if (st->path == PATH_FAST && st->need_ties != 0u) my_adm = P.tile_csum[it];
                }
            }
        }
        uint32_t todo = __ballot_sync(0xFFFFFFFFu, my_adm != 0u);
        while (todo) {
            const uint32_t src = (uint32_t)__ffs((int)todo) - 1u;
            todo &= todo - 1u;
            const uint32_t it = it0 + src * warps_total;
            const uint32_t adm = __shfl_sync(0xFFFFFFFFu, my_adm, src), s = __shfl_sync(0xFFFFFFFFu, my_s, src);
            const uint32_t w = it / L.tiles_per_worker;
            const uint32_t lt = it - w * L.tiles_per_worker;
            const SegEntry& seg = L.segs[s];
            const uint32_t tkey = P.state[(size_t)w * L.nseg + s].T;   // == tie key
            float* er = P.residuals + (size_t)w * L.n_total + seg.offset;
            float* ov = P.out_vals + (size_t)w * L.K_total + seg.msg_off;
            uint32_t* oi = P.out_idx + (size_t)w * L.K_total + seg.msg_off;
            const long long first = (long long)(lt - seg.tile_begin) * TILE - misalign_of(er);
            const bool full = first >= 0 && first + TILE <= (long long)seg.n;
            uint32_t pos = P.offsets[(size_t)w * (L.tiles_per_worker + 1) + lt];
            uint32_t ties_seen = 0;
            for (uint32_t r0 = 0; r0 < TILE / 128; r0 += 8) {           // 128 coordinates per step, a quad per lane; eight steps' loads together
                float pb[8][4];
                uint32_t vb[8];
                if (full) {                                               // uniform: eight independent 128-bit loads
#pragma unroll
                    for (uint32_t u = 0; u < 8; ++u) {
                        const float4 q = *reinterpret_cast<const float4*>(er + first + 128 * (r0 + u) + 4 * lane);
                        pb[u][0] = q.x; pb[u][1] = q.y; pb[u][2] = q.z; pb[u][3] = q.w;
                        vb[u] = 0xFu;
                    }
                } else {
#pragma unroll
                    for (uint32_t u = 0; u < 8; ++u) vb[u] = load_quad(er, first + 128 * (r0 + u) + 4 * lane, seg.n, pb[u]);
                }
#pragma unroll
                for (uint32_t u = 0; u < 8; ++u) {
                    const long long qb = first + 128 * (r0 + u) + 4 * lane;
                    float* p = pb[u];
                    const uint32_t valid = vb[u];
                    uint32_t above = 0, tie = 0;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t key = key_of(p[c]), v = (valid >> c) & 1u;
                        above |= (v & (uint32_t)(key > tkey)) << c;
                        tie |= (v & (uint32_t)(key == tkey)) << c;
                    }
                    // ranks by four independent ballots (one per position in the quad) instead of a five-step scan:
                    // this loop is a chain of dependent steps on one warp, and their latency is what it costs
                    uint32_t trank = ties_seen, ttotal = 0;             // tie-key elements of the tile before this quad
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t b = __ballot_sync(0xFFFFFFFFu, (tie >> c) & 1u);
                        trank += __popc(b & lt_mask); ttotal += __popc(b);
                    }
                    uint32_t keep = above;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if ((tie >> c) & 1u) { if (trank < adm) keep |= 1u << c; ++trank; }
                    ties_seen += ttotal;
                    uint32_t rank = 0, step_kept = 0;                   // among the kept elements of this step (at most 128)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t b = __ballot_sync(0xFFFFFFFFu, (keep >> c) & 1u);
                        rank += __popc(b & lt_mask); step_kept += __popc(b);
                    }
                    if (keep) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            if ((keep >> c) & 1u) {
                                stage_v[rank] = p[c]; stage_i[rank] = (uint32_t)seg.offset + (uint32_t)(qb + c);
                                ++rank;
                                p[c] = 0.0f;
                            }
                        }
                        store_quad(er, qb, valid, p);
                    }
                    __syncwarp();
                    // the step's kept entries go out together: consecutive lanes, consecutive message slots
                    for (uint32_t i = lane; i < step_kept; i += 32) {
                        if (pos + i < seg.k) { ov[pos + i] = stage_v[i]; oi[pos + i] = stage_i[i]; }
                        else atomicMin(P.status, ST_DEVICE_CHECK);
                    }
                    __syncwarp();
                    pos += step_kept;
                }
            }
        }
    }
}

// ---- restore: a segment fell back; put the sure values back so that the residual holds p ------
// (called by every CTA of the fall-back kernel before the radix select)
__device__ inline void restore_failed_segments(const FastParams& P) {
    const Layout& L = P.L;
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
        const uint32_t base = P.tile_fbase[item], cnt = P.tile_fcnt[item], zcut = st->zcut;
        if (base == 0xFFFFFFFFu || cnt == 0u) continue;                 // nothing was written, nothing was zeroed
        const uint2* flist = P.flagged + (size_t)w * L.flag_per_worker + seg.flag_begin + base;
        float* e = P.residuals + (size_t)w * L.n_total + seg.offset;
        for (uint32_t i = lane; i < cnt; i += 32) {
            const uint2 a = flist[i];
            if ((a.x & 0x7FFFFFFFu) > zcut) e[a.y] = __uint_as_float(a.x);
        }
    }
}

}  // namespace sc
