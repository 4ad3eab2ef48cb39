// Fall-back stream-compaction pack + residual writeback (Algorithm 1: q^w = C(p), e' = p - q^w) for
// segments whose sampled bracket missed; last phase of the fall-back kernel (sc_topk_fallback.cuh).
//
// The CTAs walk all (worker, segment, tile group) items of the failed segments in order, handing
// out groups of PACK_GROUP tiles through an atomic ticket so that every group's
// predecessors are already owned by running CTAs.
//   phase 1  streams the group's tiles: reads p (parked in the residual buffer), classifies every
//            element against the threshold T, keeps only the 4-bit "kept" masks per quad (shared
//            memory) and the per-warp counts;
//   scan     block scan of the counts, then ONE chained-scan look-back per group (each
//            group publishes its count, then sums its predecessors' words);
//   phase 2  re-reads only the quads that hold kept elements (they are still in L2),
//            writes values and coordinates at their ranks and zeroes them in the residual.
// kept = key > T, plus the first r coordinates with key == T.
// Grouping matters because a chained scan advances by at most 32 descriptors per L2 round
// trip: with single 16 KB tiles that caps the pass near 1 TB/s, far below HBM.
// Every wait on a predecessor is bounded; when it runs out the kernel records ST_TIMEOUT
// in the status word and carries on with a zero prefix.
#pragma once
#include "sc_common.cuh"

namespace sc {

struct PackParams {
    Layout L;
    float* residuals;
    float* out_vals;
    uint32_t* out_idx;
    const TopkState* state;
    const FastState* fstate;         // only segments whose bracket missed are served
    WorkList wl;                     // the pack groups this launch walks
    uint32_t epoch;                  // tag of this launch inside the descriptor words
    uint32_t total_items;            // groups over all workers
    uint32_t poll_limit;             // polls after which a look-back gives up
    unsigned long long* ticket;      // zeroed before the launch
    unsigned long long* desc;        // two words per group
    int* status;
};

constexpr uint32_t DESC_AGG = 1u, DESC_INC = 2u;
constexpr unsigned long long DESC_VAL_MASK = (1ull << 34) - 1ull;
constexpr uint32_t LOOKBACK_POLL_LIMIT = 1u << 21;   // default of PackParams::poll_limit

__device__ inline void desc_store(unsigned long long* p, uint32_t epoch, uint32_t st, unsigned long long v) {
    *reinterpret_cast<volatile unsigned long long*>(p) = ((unsigned long long)((epoch << 2) | st) << 34) | v;
}
__device__ inline unsigned long long desc_load(const unsigned long long* p) {
    return *reinterpret_cast<const volatile unsigned long long*>(p);
}
// status of a word for this launch: 0 = not written yet
__device__ inline uint32_t desc_status(unsigned long long w, uint32_t epoch) {
    uint32_t tag = (uint32_t)(w >> 34);
    return ((tag >> 2) == epoch) ? (tag & 3u) : 0u;
}

__device__ inline uint32_t warp_sum(uint32_t v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// Chained-scan look-back executed by warp 0.  Returns the exclusive prefixes of
// the two counters over items [first, item) of the same problem.  Each round
// inspects 32 * LB_DEPTH predecessors (LB_DEPTH consecutive words per lane), so
// the scan front moves that many groups per L2 round trip.
constexpr int LB_DEPTH = 4;

__device__ inline void lookback(const PackParams& P, uint32_t item, uint32_t first, bool dual,
                                uint32_t& ex0, uint32_t& ex1) {
    const uint32_t lane = threadIdx.x & 31u;
    unsigned long long acc0 = 0, acc1 = 0;
    long long pos = (long long)item - 1;
    uint32_t polls = 0;
    bool done = false;
    while (!done) {
        const long long mine = pos - (long long)lane * LB_DEPTH;      // nearest of this lane's words
        unsigned long long w0[LB_DEPTH], w1[LB_DEPTH];
        uint32_t st[LB_DEPTH];
        while (true) {
            bool ready = true;
#pragma unroll
            for (int d = 0; d < LB_DEPTH; ++d) {
                const long long at = mine - d;
                st[d] = DESC_INC; w0[d] = 0; w1[d] = 0;               // out of range counts as "done, zero"
                if (at >= (long long)first) {
                    w0[d] = desc_load(P.desc + 2 * at);
                    st[d] = desc_status(w0[d], P.epoch);
                    if (dual) {
                        w1[d] = desc_load(P.desc + 2 * at + 1);
                        if (desc_status(w1[d], P.epoch) != st[d]) st[d] = 0;
                    }
                    ready = ready && st[d] != 0;
                }
            }
            if (__all_sync(0xFFFFFFFFu, ready)) break;
            if (++polls > P.poll_limit) {           // give up: report and stop waiting
                if (lane == 0) atomicMin(P.status, ST_TIMEOUT);
                ex0 = 0; ex1 = 0;
                return;
            }
            __nanosleep(20);
        }
        // sum this lane's words up to and including its first inclusive one
        uint32_t s0 = 0, s1 = 0;
        bool found = false;
#pragma unroll
        for (int d = 0; d < LB_DEPTH; ++d) {
            if (!found) {
                s0 += (uint32_t)(w0[d] & DESC_VAL_MASK);
                s1 += (uint32_t)(w1[d] & DESC_VAL_MASK);
                found = st[d] == DESC_INC;
            }
        }
        const uint32_t inc_mask = __ballot_sync(0xFFFFFFFFu, found);
        const uint32_t upto = inc_mask ? (uint32_t)(__ffs((int)inc_mask) - 1) : 31u;
        acc0 += warp_sum(lane <= upto ? s0 : 0u);
        if (dual) acc1 += warp_sum(lane <= upto ? s1 : 0u);
        if (inc_mask) done = true; else pos -= 32 * LB_DEPTH;
    }
    ex0 = (uint32_t)acc0;
    ex1 = (uint32_t)acc1;
}

// Element-to-thread mapping inside a tile: thread t owns the 16 consecutive elements
// [16 t, 16 t + 16) (four float4 loads of one 64-byte run), so that the rank of a kept
// element is (kept in lower lanes, one warp scan per tile) + (kept bits below it in the
// thread's own 16-bit mask).
__device__ inline void pack_failed_segments(const PackParams& P) {
    constexpr int G = PACK_GROUP;
    constexpr int NCNT = G * WARPS;                // one count per (tile, warp)
    constexpr int EPL = NCNT / 32;                 // count entries per lane in the warp scan
    constexpr int BATCH = 4;                       // quads re-read together in phase 2
    constexpr int EPT = QUADS * 4;                 // elements per thread per tile
    static_assert(NCNT % 32 == 0 && G * QUADS <= 32 && EPT == 16, "table layout");
    __shared__ uint32_t s_dec[5];
    __shared__ uint16_t s_abits[G][THREADS];                   // kept / above-threshold bits of 16 elements
    __shared__ uint16_t s_tbits[G][THREADS];                   // tie bits
    __shared__ uint16_t s_arank[G][THREADS];                   // kept elements in lower lanes, same tile
    __shared__ uint16_t s_trank[G][THREADS];
    __shared__ uint32_t s_cnt[2][NCNT];
    __shared__ uint32_t s_grp_excl[2];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const Layout& L = P.L;

    while (true) {
        if (threadIdx.x == 0) {
            unsigned long long tk = atomicAdd(P.ticket, 1ull);
            uint32_t item = tk < (unsigned long long)P.total_items ? (uint32_t)tk : 0xFFFFFFFFu;
            s_dec[0] = item;
            if (item != 0xFFFFFFFFu) {
                uint32_t w = item / P.wl.len;
                uint32_t lg = P.wl.ids[item - w * P.wl.len];
                uint32_t s = find_by_group(L, lg);
                const SegEntry sg = L.segs[s];
                uint32_t gi = lg - sg.grp_begin;                              // group inside the segment
                uint32_t ntiles = L.segs[s + 1].tile_begin - sg.tile_begin;
                s_dec[1] = w; s_dec[2] = s; s_dec[3] = gi;
                s_dec[4] = min((uint32_t)G, ntiles - gi * G);
            }
        }
        __syncthreads();
        const uint32_t item = s_dec[0];
        if (item == 0xFFFFFFFFu) break;
        const uint32_t w = s_dec[1], s = s_dec[2], gi = s_dec[3], ntl = s_dec[4];
        if (__ldcg(&P.fstate[(size_t)w * L.nseg + s].path) != PATH_FAILED) { __syncthreads(); continue; }
        const SegEntry seg = L.segs[s];
        const size_t row = (size_t)w * L.n_total + seg.offset;
        float* e = P.residuals + row;
        const uint32_t mis = misalign_of(e);
        const long long t0 = (long long)gi * G;
        const uint32_t T = __ldcg(&P.state[(size_t)w * L.nseg + s].T), r = __ldcg(&P.state[(size_t)w * L.nseg + s].r);
        const bool dual = __ldcg(&P.state[(size_t)w * L.nseg + s].dual) != 0;

        // ---- phase 1: stream, classify, rank inside the warp, count -------------------------
        uint32_t pend = 0;                       // bit gl*QUADS+j: this thread's quad holds a candidate
#pragma unroll 2
        for (uint32_t gl = 0; gl < (uint32_t)G; ++gl) {
            uint32_t ab16 = 0, tb16 = 0;
            if (gl < ntl) {
                const long long first = (t0 + gl) * TILE - mis;          // local index of the tile's first element
                const long long mine = first + (long long)threadIdx.x * EPT;
#pragma unroll
                for (int j = 0; j < QUADS; ++j) {
                    const long long base = mine + 4 * j;
                    float p[4];
                    const uint32_t valid = load_quad(e, base, seg.n, p);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t key = key_of(p[c]);
                        const uint32_t v = (valid >> c) & 1u;
                        if (dual) {
                            ab16 |= (v & (uint32_t)(key > T)) << (4 * j + c);
                            tb16 |= (v & (uint32_t)(key == T)) << (4 * j + c);
                        } else {
                            ab16 |= (v & (uint32_t)(key >= T)) << (4 * j + c);
                        }
                    }
                }
                const uint32_t any16 = ab16 | tb16;
                if (any16) {
#pragma unroll
                    for (int j = 0; j < QUADS; ++j)
                        if ((any16 >> (4 * j)) & 0xFu) pend |= 1u << (gl * QUADS + j);
                }
                uint32_t inc = __popc(ab16);
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= (uint32_t)d) inc += t;
                }
                s_arank[gl][threadIdx.x] = (uint16_t)(inc - __popc(ab16));
                if (lane == 31u) s_cnt[0][gl * WARPS + warp] = inc;
                if (dual) {
                    uint32_t tinc = __popc(tb16);
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, tinc, d);
                        if (lane >= (uint32_t)d) tinc += t;
                    }
                    s_trank[gl][threadIdx.x] = (uint16_t)(tinc - __popc(tb16));
                    if (lane == 31u) s_cnt[1][gl * WARPS + warp] = tinc;
                }
            } else if (lane == 0) {
                s_cnt[0][gl * WARPS + warp] = 0;
                s_cnt[1][gl * WARPS + warp] = 0;
            }
            s_abits[gl][threadIdx.x] = (uint16_t)ab16;
            s_tbits[gl][threadIdx.x] = (uint16_t)tb16;
        }
        __syncthreads();

        // ---- scan of the per-(tile, warp) counts + one look-back for the group (warp 0) -------
        if (warp == 0) {
            uint32_t v0[EPL], v1[EPL], sum0 = 0, sum1 = 0;
#pragma unroll
            for (int i = 0; i < EPL; ++i) {
                v0[i] = s_cnt[0][lane * EPL + i];
                v1[i] = dual ? s_cnt[1][lane * EPL + i] : 0u;
                sum0 += v0[i]; sum1 += v1[i];
            }
            uint32_t i0 = sum0, i1 = sum1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t a = __shfl_up_sync(0xFFFFFFFFu, i0, d);
                const uint32_t b = __shfl_up_sync(0xFFFFFFFFu, i1, d);
                if (lane >= (uint32_t)d) { i0 += a; i1 += b; }
            }
            const uint32_t tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31), tot1 = __shfl_sync(0xFFFFFFFFu, i1, 31);
            uint32_t ex0 = i0 - sum0, ex1 = i1 - sum1;
#pragma unroll
            for (int i = 0; i < EPL; ++i) {
                s_cnt[0][lane * EPL + i] = ex0; ex0 += v0[i];
                s_cnt[1][lane * EPL + i] = ex1; ex1 += v1[i];
            }
            unsigned long long* my = P.desc + 2 * (size_t)item;
            uint32_t gex0 = 0, gex1 = 0;
            if (gi == 0) {
                if (lane == 0) {
                    desc_store(my, P.epoch, DESC_INC, tot0);
                    if (dual) desc_store(my + 1, P.epoch, DESC_INC, tot1);
                }
            } else {
                if (lane == 0) {
                    desc_store(my, P.epoch, DESC_AGG, tot0);
                    if (dual) desc_store(my + 1, P.epoch, DESC_AGG, tot1);
                }
                lookback(P, item, item - gi, dual, gex0, gex1);
                if (lane == 0) {
                    desc_store(my, P.epoch, DESC_INC, (unsigned long long)gex0 + tot0);
                    if (dual) desc_store(my + 1, P.epoch, DESC_INC, (unsigned long long)gex1 + tot1);
                }
            }
            if (lane == 0) { s_grp_excl[0] = gex0; s_grp_excl[1] = gex1; }
        }
        __syncthreads();

        // ---- phase 2: each thread walks its own pending quads, BATCH re-reads in flight -------
        float* ovals = P.out_vals + (size_t)w * L.K_total + seg.msg_off;
        uint32_t* oidx = P.out_idx + (size_t)w * L.K_total + seg.msg_off;
        const uint32_t gex0 = s_grp_excl[0], gex1 = s_grp_excl[1];
        const uint32_t idx0 = (uint32_t)seg.offset;
        while (pend) {
            int sl[BATCH];
            float q[BATCH][4];
            uint32_t valid[BATCH];
            long long base[BATCH];
#pragma unroll
            for (int b = 0; b < BATCH; ++b) {
                sl[b] = pend ? (__ffs((int)pend) - 1) : -1;
                if (pend) pend &= pend - 1u;
            }
#pragma unroll
            for (int b = 0; b < BATCH; ++b) {
                valid[b] = 0; base[b] = 0;
                if (sl[b] >= 0) {
                    const uint32_t gl = (uint32_t)sl[b] / QUADS, j = (uint32_t)sl[b] % QUADS;
                    base[b] = (t0 + gl) * TILE - mis + (long long)threadIdx.x * EPT + 4 * j;
                    valid[b] = load_quad(e, base[b], seg.n, q[b]);
                }
            }
#pragma unroll
            for (int b = 0; b < BATCH; ++b) {
                if (sl[b] < 0) continue;
                const uint32_t gl = (uint32_t)sl[b] / QUADS, j = (uint32_t)sl[b] % QUADS;
                const uint32_t ab16 = s_abits[gl][threadIdx.x];
                const uint32_t tb16 = dual ? s_tbits[gl][threadIdx.x] : 0u;
                const uint32_t below = (1u << (4 * j)) - 1u;
                uint32_t a_before = gex0 + s_cnt[0][gl * WARPS + warp] + s_arank[gl][threadIdx.x] + __popc(ab16 & below);
                uint32_t t_before = 0;
                if (dual)
                    t_before = gex1 + s_cnt[1][gl * WARPS + warp] + s_trank[gl][threadIdx.x] + __popc(tb16 & below);
                const uint32_t ab = (ab16 >> (4 * j)) & 0xFu, tb = (tb16 >> (4 * j)) & 0xFu;
                uint32_t kept = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t abc = (ab >> c) & 1u, tbc = (tb >> c) & 1u;
                    if (abc | tbc) {
                        uint32_t slot = 0xFFFFFFFFu;
                        if (abc) slot = a_before + (dual ? min(t_before, r) : 0u);
                        else if (t_before < r) slot = a_before + t_before;
                        if (slot != 0xFFFFFFFFu) {
                            if (slot < seg.k) {
                                ovals[slot] = q[b][c];
                                oidx[slot] = idx0 + (uint32_t)(base[b] + c);
                            } else {
                                atomicMin(P.status, ST_DEVICE_CHECK);
                            }
                            kept |= 1u << c;
                            q[b][c] = 0.0f;
                        }
                        a_before += abc;
                        t_before += tbc;
                    }
                }
                if (kept) store_quad(e, base[b], valid[b], q[b]);
            }
        }
        __syncthreads();    // shared tables are reused by the next group
    }
}

}  // namespace sc
