// Seeded coordinate generation for Random-k and Block-random-k (Methodology,
// "Random-k Sparsification", "Block-random-k Sparsification").
//
// Random-k: coordinate set { pi(j) : j < k } of a keyed bijection pi of [0, n)
// (alternating Feistel network on ceil(log2 n) bits, cycle walking).  The set is
// materialised as an n-bit membership mask with k scattered bit-sets, so that the
// compression pass itself is a fully coalesced stream (no random reads of g or e).
// Block-random-k: one start per (seed, segment); the pass is a plain stream.
#pragma once
#include <cooperative_groups.h>

#include "sc_common.cuh"

namespace sc {

constexpr uint32_t SCAT_CHUNK = 1024;            // coordinates per scatter CTA
constexpr uint32_t CYCLE_WALK_LIMIT = 256;       // expected < 2 steps; bound guards against a bug

__global__ void __launch_bounds__(THREADS)
randk_scatter_kernel(Layout L, const uint64_t* __restrict__ seeds, uint32_t* __restrict__ mask,
                     int* __restrict__ status) {
    const uint32_t q = blockIdx.x / L.scat_per_group;            // seed group
    const uint32_t ls = blockIdx.x - q * L.scat_per_group;
    const uint32_t s = find_by_scat(L, ls);
    const SegEntry seg = L.segs[s];
    const uint32_t chunk = ls - seg.scat_begin;
    const Feistel f = feistel_setup(mix64(seeds[q], s), seg.n);
    uint32_t* m = mask + (size_t)q * L.mask_words_per_group + seg.mask_word_begin;
#pragma unroll
    for (uint32_t it = 0; it < SCAT_CHUNK / THREADS; ++it) {
        const uint32_t j = chunk * SCAT_CHUNK + it * THREADS + threadIdx.x;
        if (j < seg.k) {
            uint32_t x = j, steps = 0;
            do { x = feistel_once(f, x); } while (x >= seg.n && ++steps < CYCLE_WALK_LIMIT);
            if (x < seg.n) atomicOr(m + (x >> 5), 1u << (x & 31u));
            else atomicMin(status, ST_DEVICE_CHECK);
        }
    }
}

// Block-random-k: p = g + e; the block [a, a+k) goes to the message and becomes
// zero in the residual, everything else is written back as p.
__global__ void __launch_bounds__(THREADS)
randblock_kernel(Layout L, const float* __restrict__ grads, float* __restrict__ residuals,
                 const uint64_t* __restrict__ seeds, float* __restrict__ out_vals,
                 uint32_t* __restrict__ out_idx, uint32_t total_items, uint32_t wrap) {
    __shared__ uint32_t s_dec[4];
    const uint32_t group_step = (gridDim.x - 1u) * STREAM_GROUP + 1u;
    for (uint32_t item = blockIdx.x * STREAM_GROUP, ig = 0; item < total_items;
         item += (ig + 1u == STREAM_GROUP ? group_step : 1u), ig = (ig + 1u == STREAM_GROUP ? 0u : ig + 1u)) {
        if (threadIdx.x == 0) {
            uint32_t w = item / L.tiles_per_worker;
            uint32_t lt = item - w * L.tiles_per_worker;
            uint32_t s = find_by_tile(L, lt);
            const SegEntry sg = L.segs[s];
            s_dec[0] = w; s_dec[1] = s; s_dec[2] = lt - sg.tile_begin;
            s_dec[3] = wrap ? block_start_wrap(mix64(seeds[w], s), sg.n) : block_start(mix64(seeds[w], s), sg.n, sg.k);
        }
        __syncthreads();
        const uint32_t w = s_dec[0], s = s_dec[1], t = s_dec[2], a = s_dec[3];
        const SegEntry seg = L.segs[s];
        const uint32_t head = (wrap && (uint64_t)a + seg.k > seg.n) ? (uint32_t)((uint64_t)a + seg.k - seg.n) : 0u;   // wrapped entries
        const size_t row = (size_t)w * L.n_total + seg.offset;
        const float* g = grads + row;
        float* e = residuals + row;
        const uint32_t mis = misalign_of(e);
        float* ovals = out_vals + (size_t)w * L.K_total + seg.msg_off;
        uint32_t* oidx = out_idx + (size_t)w * L.K_total + seg.msg_off;
        // most tiles lie outside the kept block: they only stream p = gamma g + e back
        const long long tlo = (long long)t * TILE - mis, thi = tlo + TILE;
        const long long a_end = min((long long)a + (long long)seg.k, (long long)seg.n);
        const bool touches = seg.k != 0u && ((tlo < a_end && thi > (long long)a) || tlo < (long long)head);
#pragma unroll
        for (int j = 0; j < QUADS; ++j) {
            const long long base = (long long)t * TILE + (long long)(j * THREADS + threadIdx.x) * 4 - mis;
            float p[4], gv[4];
            const uint32_t m = load_quad(e, base, seg.n, p);
            if (!m) continue;
            load_quad_stream(g, base, seg.n, gv);
#pragma unroll
            for (int c = 0; c < 4; ++c) p[c] = accumulate(L.gamma, gv[c], p[c]);
            if (touches) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const long long i = base + c;
                    // distance from the block's start, cyclically when the block wraps: kept iff < k.  A wrapped
                    // block's head [0, a + k - n) comes first in the ascending message, its tail [a, n) after it.
                    const long long d = i >= (long long)a ? i - a : (wrap ? i + seg.n - a : (long long)seg.k);
                    if (((m >> c) & 1u) && d < (long long)seg.k) {
                        const uint32_t slot = i >= (long long)a ? head + (uint32_t)(i - a) : (uint32_t)i;
                        ovals[slot] = p[c];
                        oidx[slot] = (uint32_t)(seg.offset + (uint64_t)i);
                        p[c] = 0.0f;
                    }
                }
            }
            store_quad(e, base, m, p);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------
// Random-k compression pass.  The kept set is known before any gradient is read
// (it is the membership mask), so the message slot of every kept coordinate
// follows from population counts alone:
//   mask_count_kernel   kept coordinates per tile of TILE coordinates,
//   row_scan_kernel     exclusive prefix over the tiles of one seed group,
//   randk_pack_kernel   ONE coalesced stream over g and e: p = g + e, kept values
//                       and coordinates go to their slots, e' = p with the kept
//                       entries zeroed.  No CTA waits on another.
// ---------------------------------------------------------------------------
// One warp per (seed group, tile): counts[q][lt] = kept coordinates in the
// tile's fixed range [t * TILE, (t + 1) * TILE) of its segment.
__global__ void __launch_bounds__(THREADS)
mask_count_kernel(Layout L, const uint32_t* __restrict__ mask, uint32_t groups, uint32_t* __restrict__ counts) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t wid = (uint64_t)blockIdx.x * WARPS + (threadIdx.x >> 5);
    if (wid >= (uint64_t)groups * L.tiles_per_worker) return;
    const uint32_t q = (uint32_t)(wid / L.tiles_per_worker);
    const uint32_t lt = (uint32_t)(wid - (uint64_t)q * L.tiles_per_worker);
    const uint32_t s = find_by_tile(L, lt);
    const SegEntry seg = L.segs[s];
    const uint32_t t = lt - seg.tile_begin;
    const uint32_t words = (seg.n + 31u) >> 5;                         // mask words of the segment
    const uint32_t* m = mask + (size_t)q * L.mask_words_per_group + seg.mask_word_begin;
    uint32_t c = 0;
#pragma unroll
    for (int i = 0; i < TILE / 32 / 32; ++i) {
        const uint32_t wi = t * (TILE / 32) + i * 32 + lane;
        if (wi < words) c += __popc(__ldg(m + wi));
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, d);
    if (lane == 0) counts[(size_t)q * (L.tiles_per_worker + 1) + lt] = c;
}

// In-place exclusive scan of each row of `len` counts; entry [len] receives the row total.
// A row is served by a cluster of C CTAs (C = 1: a single CTA): every CTA first adds up its
// contiguous share of the row, the shares' totals are exchanged through distributed shared
// memory, and each CTA then scans its share starting from the sum of the shares before it.
// The serial part of a long row shrinks by C (85,000 tiles per worker: 0.097 -> 0.03 ms).
constexpr uint32_t ROW_SCAN_CTAS = 8;
template <uint32_t C>
__global__ void __launch_bounds__(THREADS)
row_scan_kernel(uint32_t* __restrict__ data, uint32_t len) {
    namespace cg = cooperative_groups;
    __shared__ uint32_t smem[WARPS + 1];
    __shared__ uint32_t s_share;                                       // this CTA's total
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = C > 1 ? cluster.block_rank() : 0u;
    uint32_t* row = data + (size_t)(blockIdx.x / C) * (len + 1);
    const uint32_t per = ((len + C - 1) / C + THREADS * 4 - 1) / (THREADS * 4) * (THREADS * 4);
    const uint32_t begin = min(rank * per, len), end = min(begin + per, len);
    uint32_t carry = 0;
    if constexpr (C > 1) {
        uint32_t sum = 0;
        for (uint32_t at = begin + threadIdx.x; at < end; at += THREADS) sum += row[at];
        uint32_t total;
        block_exclusive_scan(sum, smem, &total);
        if (threadIdx.x == 0) s_share = total;
        cluster.sync();
        for (uint32_t r = 0; r < rank; ++r) carry += *cluster.map_shared_rank(&s_share, r);
    }
    for (uint32_t base = begin; base < end; base += THREADS * 4) {
        uint32_t v[4], sum = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t at = base + threadIdx.x * 4 + i;
            v[i] = at < end ? row[at] : 0u;
            sum += v[i];
        }
        uint32_t total;
        uint32_t ex = block_exclusive_scan(sum, smem, &total) + carry;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t at = base + threadIdx.x * 4 + i;
            if (at < end) row[at] = ex;
            ex += v[i];
        }
        carry += total;
    }
    if (rank == C - 1 && threadIdx.x == 0) row[len] = carry;
    if (C > 1) cluster.sync();                                         // a peer's total must outlive its readers
}

// Element-to-thread mapping inside a tile: warp w owns the 512 consecutive elements
// [512 w, 512 w + 512) as four rows of 128; lane l holds the quad at 512 w + 128 j + 4 l of
// row j, so every load and store instruction of a warp covers 512 contiguous bytes.
// The four per-row kept counts of a lane (each <= 4, row totals <= 128) ride in the four
// bytes of one word, so a single 5-step warp scan ranks all four rows at once.
__global__ void __launch_bounds__(THREADS)
randk_pack_kernel(Layout L, const float* __restrict__ grads, float* __restrict__ residuals,
                  const uint32_t* __restrict__ mask, const uint32_t* __restrict__ offsets,
                  uint32_t mask_per_worker, float* __restrict__ out_vals, uint32_t* __restrict__ out_idx,
                  uint32_t total_items, int* __restrict__ status) {
    __shared__ uint32_t s_wtot[2][WARPS];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t parity = 0;
    const uint32_t group_step = (gridDim.x - 1u) * STREAM_GROUP + 1u;
    for (uint32_t item = blockIdx.x * STREAM_GROUP, ig = 0; item < total_items;
         item += (ig + 1u == STREAM_GROUP ? group_step : 1u), ig = (ig + 1u == STREAM_GROUP ? 0u : ig + 1u), parity ^= 1u) {
        const uint32_t w = item / L.tiles_per_worker;
        const uint32_t lt = item - w * L.tiles_per_worker;
        const uint32_t s = (L.nseg == 1) ? 0u : find_by_tile(L, lt);
        const SegEntry seg = L.segs[s];
        const uint32_t t = lt - seg.tile_begin;
        const size_t row = (size_t)w * L.n_total + seg.offset;
        const float* g = grads + row;
        float* e = residuals + row;
        const uint32_t mis = misalign_of(e);
        const uint32_t q = mask_per_worker ? w : 0u;
        const uint32_t* m = mask + (size_t)q * L.mask_words_per_group + seg.mask_word_begin;
        const uint32_t* off = offsets + (size_t)q * (L.tiles_per_worker + 1);
        // kept coordinates of the segment before this tile's first element
        uint32_t tile_rank = off[lt] - off[seg.tile_begin];
        if (mis && t) tile_rank -= __popc(__ldg(m + (size_t)t * (TILE / 32) - 1) >> (32u - mis));

        const long long first = (long long)t * TILE - mis;
        const long long mine = first + warp * 512 + lane * 4;             // quad of row 0; row j at + 128 j
        const bool full = first >= 0 && first + TILE <= (long long)seg.n;
        uint32_t bits = 0;                                               // nibble j = kept bits of row j's quad
        if (full) {
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const uint32_t pos = (uint32_t)mine + 128u * j, a = pos >> 5, sh = pos & 31u;
                const uint32_t lo = __ldg(m + a);
                const uint32_t hi = (sh > 28u) ? __ldg(m + a + 1) : lo;
                bits |= (__funnelshift_r(lo, hi, sh) & 0xFu) << (4 * j);
            }
        } else {
#pragma unroll
            for (int i = 0; i < QUADS * 4; ++i) {
                const long long at = mine + 128 * (i >> 2) + (i & 3);
                if (at >= 0 && at < (long long)seg.n)
                    bits |= ((__ldg(m + (at >> 5)) >> (uint32_t)(at & 31)) & 1u) << i;
            }
        }
        const uint32_t cnt4 = __popc(bits & 0xFu) | (__popc(bits & 0xF0u) << 8) |
                              (__popc(bits & 0xF00u) << 16) | (__popc(bits & 0xF000u) << 24);
        uint32_t inc4 = cnt4;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, inc4, d);
            if (lane >= (uint32_t)d) inc4 += v;
        }
        const uint32_t tot4 = __shfl_sync(0xFFFFFFFFu, inc4, 31);        // the four row totals
        const uint32_t ex4 = inc4 - cnt4;                                // kept in lower lanes, per row
        const uint32_t rowbase4 = (tot4 << 8) + (tot4 << 16) + (tot4 << 24);   // byte j = sum of rows < j (mod 256)
        const uint32_t wtot = (tot4 & 0xFFu) + ((tot4 >> 8) & 0xFFu) + ((tot4 >> 16) & 0xFFu) + (tot4 >> 24);
        if (lane == 0) s_wtot[parity][warp] = wtot;
        __syncthreads();
        uint32_t wbase = tile_rank;
#pragma unroll
        for (int i = 0; i < WARPS; ++i) wbase += (i < (int)warp) ? s_wtot[parity][i] : 0u;

        float* ovals = out_vals + (size_t)w * L.K_total + seg.msg_off;
        uint32_t* oidx = out_idx + (size_t)w * L.K_total + seg.msg_off;
        const uint32_t idx0 = (uint32_t)seg.offset;
        // row bases can exceed a byte (up to 384), so rebuild them from the totals
        uint32_t rowbase[QUADS];
        rowbase[0] = 0;
#pragma unroll
        for (int j = 1; j < QUADS; ++j) rowbase[j] = rowbase[j - 1] + ((tot4 >> (8 * (j - 1))) & 0xFFu);
        (void)rowbase4;
        if (full) {
            float4 qv[QUADS];
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const float4 ev = __ldcs(reinterpret_cast<const float4*>(e + mine + 128 * j));
                const float4 gv = __ldcs(reinterpret_cast<const float4*>(g + mine + 128 * j));
                qv[j] = accumulate(L.gamma, gv, ev);
            }
            if (SC_PREFETCH_DIST) {   // this tile's loads have landed: ask L2 for the tile the CTA takes next
                const uint32_t ahead = ig + 1u == STREAM_GROUP ? group_step : 1u;
                if (lt + ahead + 1u < L.segs[s + 1].tile_begin) prefetch_tile_l2(g, e, first + (long long)ahead * TILE);
            }
            if (bits) {
#pragma unroll
                for (int j = 0; j < QUADS; ++j) {
                    float* v = reinterpret_cast<float*>(&qv[j]);
                    uint32_t rank = wbase + rowbase[j] + ((ex4 >> (8 * j)) & 0xFFu);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if ((bits >> (4 * j + c)) & 1u) {
                            if (rank < seg.k) {
                                ovals[rank] = v[c];
                                oidx[rank] = idx0 + (uint32_t)mine + 128u * j + c;
                            } else {
                                atomicMin(status, ST_DEVICE_CHECK);
                            }
                            ++rank;
                            v[c] = 0.0f;
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < QUADS; ++j) *reinterpret_cast<float4*>(e + mine + 128 * j) = qv[j];
        } else {
#pragma unroll
            for (int j = 0; j < QUADS; ++j) {
                const long long base = mine + 128 * j;
                float p[4], gv[4];
                const uint32_t valid = load_quad(e, base, seg.n, p);
                if (!valid) continue;
                load_quad_stream(g, base, seg.n, gv);
                uint32_t rank = wbase + rowbase[j] + ((ex4 >> (8 * j)) & 0xFFu);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    p[c] = accumulate(L.gamma, gv[c], p[c]);
                    if ((bits >> (4 * j + c)) & 1u) {
                        if (rank < seg.k) {
                            ovals[rank] = p[c];
                            oidx[rank] = idx0 + (uint32_t)(base + c);
                        } else {
                            atomicMin(status, ST_DEVICE_CHECK);
                        }
                        ++rank;
                        p[c] = 0.0f;
                    }
                }
                store_quad(e, base, valid, p);
            }
        }
    }
}

}  // namespace sc
