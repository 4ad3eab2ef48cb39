// Stream-compaction pack + residual writeback (Algorithm 1: q^w = C(p), e' = p - q^w).
//
// One persistent kernel walks all (worker, segment, tile) items in order, handing
// out tiles through an atomic ticket so that every tile's predecessors are already
// owned by running CTAs.  Inside a tile the rank of each kept element comes from
// warp ballots and population counts; across tiles from a single-pass chained scan
// (each tile publishes its count, then looks back over its predecessors' words).
// Every wait on a predecessor is bounded; when it runs out the kernel records
// ST_TIMEOUT in the status word and carries on with a zero prefix.
//
// PACK_TOPK: p is read from the residual buffer (parked there by the histogram
//            pass); kept = key > T, plus the first r coordinates with key == T.
// PACK_MASK: p = g + e is formed here; kept = membership bit of the coordinate.
#pragma once
#include "sc_common.cuh"

namespace sc {

enum { PACK_TOPK = 0, PACK_MASK = 1 };

struct PackParams {
    Layout L;
    const float* grads;
    float* residuals;
    float* out_vals;
    uint32_t* out_idx;
    const TopkState* state;          // PACK_TOPK
    const uint32_t* mask;            // PACK_MASK
    uint32_t mask_per_worker;        // 1: worker w uses mask group w, 0: all use group 0
    uint32_t epoch;                  // tag of this launch inside the tile words
    uint32_t total_items;
    uint32_t pad;
    unsigned long long* ticket;
    unsigned long long ticket_base;
    unsigned long long* desc;        // two words per item
    int* status;
};

constexpr uint32_t DESC_AGG = 1u, DESC_INC = 2u;
constexpr unsigned long long DESC_VAL_MASK = (1ull << 34) - 1ull;
constexpr uint32_t LOOKBACK_POLL_LIMIT = 1u << 21;

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
// the two counters over tiles [first, item) of the same problem.
__device__ inline void lookback(const PackParams& P, uint32_t item, uint32_t first, bool dual,
                                uint32_t& ex0, uint32_t& ex1) {
    const uint32_t lane = threadIdx.x & 31u;
    unsigned long long acc0 = 0, acc1 = 0;
    long long pos = (long long)item - 1;
    uint32_t polls = 0;
    bool done = false;
    while (!done) {
        const long long my = pos - lane;
        const bool inrange = my >= (long long)first;
        unsigned long long w0 = 0, w1 = 0;
        uint32_t st = 0;
        while (true) {
            bool ready = true;
            if (inrange) {
                w0 = desc_load(P.desc + 2 * my);
                st = desc_status(w0, P.epoch);
                ready = st != 0;
                if (dual) {
                    w1 = desc_load(P.desc + 2 * my + 1);
                    ready = ready && desc_status(w1, P.epoch) == st;
                }
            }
            if (__all_sync(0xFFFFFFFFu, ready)) break;
            if (++polls > LOOKBACK_POLL_LIMIT) {           // give up: report and stop waiting
                if (lane == 0) atomicMin(P.status, ST_TIMEOUT);
                ex0 = 0; ex1 = 0;
                return;
            }
            __nanosleep(40);
        }
        const uint32_t inc_mask = __ballot_sync(0xFFFFFFFFu, inrange && st == DESC_INC);
        const uint32_t upto = inc_mask ? (uint32_t)(__ffs((int)inc_mask) - 1) : 31u;
        const bool use = inrange && lane <= upto;
        acc0 += warp_sum(use ? (uint32_t)(w0 & DESC_VAL_MASK) : 0u);
        if (dual) acc1 += warp_sum(use ? (uint32_t)(w1 & DESC_VAL_MASK) : 0u);
        if (inc_mask) done = true; else pos -= 32;
    }
    ex0 = (uint32_t)acc0;
    ex1 = (uint32_t)acc1;
}

template <int MODE>
__global__ void __launch_bounds__(THREADS)
pack_kernel(PackParams P) {
    static_assert(QUADS * WARPS == 32, "one warp scans the per-(quad, warp) counts");
    __shared__ uint32_t s_dec[4];
    __shared__ uint32_t s_cnt[2][32];
    __shared__ uint32_t s_excl[2][32];
    __shared__ uint32_t s_tile_excl[2];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const Layout& L = P.L;

    while (true) {
        if (threadIdx.x == 0) {
            unsigned long long tk = atomicAdd(P.ticket, 1ull) - P.ticket_base;
            uint32_t item = tk < (unsigned long long)P.total_items ? (uint32_t)tk : 0xFFFFFFFFu;
            s_dec[0] = item;
            if (item != 0xFFFFFFFFu) {
                uint32_t w = item / L.tiles_per_worker;
                uint32_t lt = item - w * L.tiles_per_worker;
                uint32_t s = find_by_tile(L, lt);
                s_dec[1] = w; s_dec[2] = s; s_dec[3] = lt - L.segs[s].tile_begin;
            }
        }
        __syncthreads();
        const uint32_t item = s_dec[0];
        if (item == 0xFFFFFFFFu) break;
        const uint32_t w = s_dec[1], s = s_dec[2], t = s_dec[3];
        const SegEntry seg = L.segs[s];
        const size_t row = (size_t)w * L.n_total + seg.offset;
        float* e = P.residuals + row;
        const uint32_t mis = misalign_of(e);

        uint32_t T = 0, r = 0;
        bool dual = false;
        const uint32_t* mask = nullptr;
        if (MODE == PACK_TOPK) {
            const TopkState st = P.state[(size_t)w * L.nseg + s];
            T = st.T; r = st.r; dual = st.dual != 0;
        } else {
            mask = P.mask + (P.mask_per_worker ? (size_t)w * L.mask_words_per_group : 0) + seg.mask_word_begin;
        }

        float p[QUADS][4];
        uint32_t valid[QUADS], abits[QUADS], tbits[QUADS];
        uint32_t arank[QUADS], trank[QUADS];
#pragma unroll
        for (int j = 0; j < QUADS; ++j) {
            const long long base = (long long)t * TILE + (long long)(j * THREADS + threadIdx.x) * 4 - mis;
            valid[j] = load_quad(e, base, seg.n, p[j]);
            abits[j] = 0; tbits[j] = 0;
            if (MODE == PACK_MASK) {
                float gv[4];
                load_quad_stream(P.grads + row, base, seg.n, gv);
#pragma unroll
                for (int c = 0; c < 4; ++c) p[j][c] = gv[c] + p[j][c];
                if (valid[j] == 0xFu) {
                    const uint32_t a = (uint32_t)(base >> 5), b = (uint32_t)((base + 3) >> 5);
                    const uint32_t lo = __ldg(mask + a);
                    const uint32_t hi = (b != a) ? __ldg(mask + b) : lo;
                    abits[j] = __funnelshift_r(lo, hi, (uint32_t)(base & 31)) & 0xFu;
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if ((valid[j] >> c) & 1u) {
                            const long long i = base + c;
                            abits[j] |= ((__ldg(mask + (i >> 5)) >> (uint32_t)(i & 31)) & 1u) << c;
                        }
                }
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t key = key_of(p[j][c]);
                    const uint32_t v = (valid[j] >> c) & 1u;
                    if (dual) {
                        abits[j] |= (v & (uint32_t)(key > T)) << c;
                        tbits[j] |= (v & (uint32_t)(key == T)) << c;
                    } else {
                        abits[j] |= (v & (uint32_t)(key >= T)) << c;
                    }
                }
            }
            // rank of this thread's quad inside the warp's 128 consecutive elements
            uint32_t below = 0, wtot = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, (abits[j] >> c) & 1u);
                below += __popc(bal & lt_mask);
                wtot += __popc(bal);
            }
            arank[j] = below;
            if (lane == 0) s_cnt[0][j * WARPS + warp] = wtot;
            trank[j] = 0;
            if (dual) {
                below = 0; wtot = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, (tbits[j] >> c) & 1u);
                    below += __popc(bal & lt_mask);
                    wtot += __popc(bal);
                }
                trank[j] = below;
                if (lane == 0) s_cnt[1][j * WARPS + warp] = wtot;
            }
        }
        __syncthreads();

        if (warp == 0) {
            const uint32_t v0 = s_cnt[0][lane];
            const uint32_t v1 = dual ? s_cnt[1][lane] : 0u;
            uint32_t i0 = v0, i1 = v1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                uint32_t a = __shfl_up_sync(0xFFFFFFFFu, i0, d);
                uint32_t b = __shfl_up_sync(0xFFFFFFFFu, i1, d);
                if (lane >= (uint32_t)d) { i0 += a; i1 += b; }
            }
            s_excl[0][lane] = i0 - v0;
            s_excl[1][lane] = i1 - v1;
            const uint32_t tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31);
            const uint32_t tot1 = __shfl_sync(0xFFFFFFFFu, i1, 31);
            unsigned long long* my = P.desc + 2 * (size_t)item;
            uint32_t ex0 = 0, ex1 = 0;
            if (t == 0) {
                if (lane == 0) {
                    desc_store(my, P.epoch, DESC_INC, tot0);
                    if (dual) desc_store(my + 1, P.epoch, DESC_INC, tot1);
                }
            } else {
                if (lane == 0) {
                    desc_store(my, P.epoch, DESC_AGG, tot0);
                    if (dual) desc_store(my + 1, P.epoch, DESC_AGG, tot1);
                }
                lookback(P, item, item - t, dual, ex0, ex1);
                if (lane == 0) {
                    desc_store(my, P.epoch, DESC_INC, (unsigned long long)ex0 + tot0);
                    if (dual) desc_store(my + 1, P.epoch, DESC_INC, (unsigned long long)ex1 + tot1);
                }
            }
            if (lane == 0) { s_tile_excl[0] = ex0; s_tile_excl[1] = ex1; }
        }
        __syncthreads();

        float* ovals = P.out_vals + (size_t)w * L.K_total + seg.msg_off;
        uint32_t* oidx = P.out_idx + (size_t)w * L.K_total + seg.msg_off;
        const uint32_t tex0 = s_tile_excl[0], tex1 = s_tile_excl[1];
#pragma unroll
        for (int j = 0; j < QUADS; ++j) {
            const long long base = (long long)t * TILE + (long long)(j * THREADS + threadIdx.x) * 4 - mis;
            uint32_t a_before = tex0 + s_excl[0][j * WARPS + warp] + arank[j];
            uint32_t t_before = dual ? tex1 + s_excl[1][j * WARPS + warp] + trank[j] : 0u;
            uint32_t kept = 0;
            if (abits[j] | tbits[j]) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t ab = (abits[j] >> c) & 1u, tb = (tbits[j] >> c) & 1u;
                    if (ab | tb) {
                        uint32_t slot = 0xFFFFFFFFu;
                        if (ab) slot = a_before + (dual ? min(t_before, r) : 0u);
                        else if (t_before < r) slot = a_before + t_before;
                        if (slot != 0xFFFFFFFFu) {
                            if (slot < seg.k) {
                                ovals[slot] = p[j][c];
                                oidx[slot] = (uint32_t)(seg.offset + (uint64_t)(base + c));
                            } else {
                                atomicMin(P.status, ST_DEVICE_CHECK);
                            }
                            kept |= 1u << c;
                        }
                        a_before += ab;
                        t_before += tb;
                    }
                }
            }
            if (MODE == PACK_MASK) {
                if (valid[j]) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) if ((kept >> c) & 1u) p[j][c] = 0.0f;
                    store_quad(e, base, valid[j], p[j]);
                }
            } else if (kept) {
#pragma unroll
                for (int c = 0; c < 4; ++c) if ((kept >> c) & 1u) p[j][c] = 0.0f;
                store_quad(e, base, valid[j], p[j]);
            }
        }
        __syncthreads();    // s_dec, s_cnt, s_excl are reused by the next tile
    }
}

}  // namespace sc
