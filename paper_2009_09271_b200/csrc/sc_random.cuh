// Seeded coordinate generation for Random-k and Block-random-k (Methodology,
// "Random-k Sparsification", "Block-random-k Sparsification").
//
// Random-k: coordinate set { pi(j) : j < k } of a keyed bijection pi of [0, n)
// (alternating Feistel network on ceil(log2 n) bits, cycle walking).  The set is
// materialised as an n-bit membership mask with k scattered bit-sets, so that the
// compression pass itself is a fully coalesced stream (no random reads of g or e).
// Block-random-k: one start per (seed, segment); the pass is a plain stream.
#pragma once
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
                 uint32_t* __restrict__ out_idx, uint32_t total_items) {
    __shared__ uint32_t s_dec[4];
    for (uint32_t item = blockIdx.x; item < total_items; item += gridDim.x) {
        if (threadIdx.x == 0) {
            uint32_t w = item / L.tiles_per_worker;
            uint32_t lt = item - w * L.tiles_per_worker;
            uint32_t s = find_by_tile(L, lt);
            const SegEntry sg = L.segs[s];
            s_dec[0] = w; s_dec[1] = s; s_dec[2] = lt - sg.tile_begin;
            s_dec[3] = block_start(mix64(seeds[w], s), sg.n, sg.k);
        }
        __syncthreads();
        const uint32_t w = s_dec[0], s = s_dec[1], t = s_dec[2], a = s_dec[3];
        const SegEntry seg = L.segs[s];
        const size_t row = (size_t)w * L.n_total + seg.offset;
        const float* g = grads + row;
        float* e = residuals + row;
        const uint32_t mis = misalign_of(e);
        float* ovals = out_vals + (size_t)w * L.K_total + seg.msg_off;
        uint32_t* oidx = out_idx + (size_t)w * L.K_total + seg.msg_off;
#pragma unroll
        for (int j = 0; j < QUADS; ++j) {
            const long long base = (long long)t * TILE + (long long)(j * THREADS + threadIdx.x) * 4 - mis;
            float p[4], gv[4];
            const uint32_t m = load_quad(e, base, seg.n, p);
            if (!m) continue;
            load_quad_stream(g, base, seg.n, gv);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                p[c] = gv[c] + p[c];
                const long long i = base + c;
                if (((m >> c) & 1u) && i >= (long long)a && i < (long long)a + seg.k) {
                    const uint32_t slot = (uint32_t)(i - a);
                    ovals[slot] = p[c];
                    oidx[slot] = (uint32_t)(seg.offset + (uint64_t)i);
                    p[c] = 0.0f;
                }
            }
            store_quad(e, base, m, p);
        }
        __syncthreads();
    }
}

}  // namespace sc
