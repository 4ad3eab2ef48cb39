// Decompress + aggregate (Algorithm 1, aggregate line, read as the average the
// abstract describes): out[i] = (sum_{w = 0..W-1, in order} q^w[i]) / W.
//
// Every message is ascending in its coordinates, so the dense output is cut into
// tiles of ATILE coordinates and one CTA owns a tile: it finds the slice of each
// worker's message that falls into the tile (bounds computed once per call by a
// binary-search kernel), accumulates the slices in shared memory in worker order
// starting from +0.0f, divides by W and stores the tile with 128-bit writes.
// Zero fill, scatter and average are therefore one pass over `out`, and the
// result does not depend on any atomic ordering.
#pragma once
#include "sc_common.cuh"

namespace sc {

constexpr uint32_t ATILE = 4096;

// bounds[r][t] = first slot j of row r with idx[j] >= t * ATILE, t = 0..ntiles.
__global__ void __launch_bounds__(THREADS)
agg_bounds_kernel(const uint32_t* __restrict__ idx, uint32_t rows, uint32_t K, uint32_t ntiles,
                  uint32_t* __restrict__ bounds) {
    const uint64_t gid = (uint64_t)blockIdx.x * THREADS + threadIdx.x;
    const uint64_t per_row = (uint64_t)ntiles + 1;
    if (gid >= per_row * rows) return;
    const uint32_t r = (uint32_t)(gid / per_row);
    const uint32_t t = (uint32_t)(gid - (uint64_t)r * per_row);
    const uint32_t* row = idx + (size_t)r * K;
    const uint64_t target = (uint64_t)t * ATILE;
    uint32_t lo = 0, hi = K;                         // first j with row[j] >= target
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if ((uint64_t)__ldg(row + mid) < target) lo = mid + 1; else hi = mid;
    }
    bounds[gid] = lo;
}

// rows_idx: number of coordinate rows (W, or 1 when all workers share them).
__global__ void __launch_bounds__(THREADS)
agg_tiles_kernel(const float* __restrict__ vals, const uint32_t* __restrict__ idx,
                 const uint32_t* __restrict__ bounds, uint32_t W, uint32_t shared_idx, uint32_t K,
                 uint32_t n, uint32_t ntiles, float* __restrict__ out, int* __restrict__ status) {
    __shared__ __align__(16) float acc[ATILE];
    __shared__ uint32_t s_lo[64], s_hi[64];
    __shared__ uint32_t s_any;
    const float fW = (float)W;
    for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const uint32_t tile_lo = t * ATILE;
        const uint32_t tile_n = min(ATILE, n - tile_lo);
        for (uint32_t i = threadIdx.x; i < ATILE; i += THREADS) acc[i] = 0.0f;
        if (threadIdx.x == 0) s_any = 0;
        __syncthreads();
        for (uint32_t w0 = 0; w0 < W; w0 += 64) {
            const uint32_t wn = min(64u, W - w0);
            if (threadIdx.x < wn) {
                const uint32_t r = shared_idx ? 0u : (w0 + threadIdx.x);
                const uint32_t* b = bounds + (size_t)r * (ntiles + 1) + t;
                const uint32_t lo = b[0], hi = b[1];
                s_lo[threadIdx.x] = lo; s_hi[threadIdx.x] = hi;
                if (hi > lo) s_any = 1;
            }
            __syncthreads();
            if (s_any) {
                for (uint32_t ww = 0; ww < wn; ++ww) {
                    const uint32_t w = w0 + ww;
                    const uint32_t lo = s_lo[ww], hi = s_hi[ww];
                    const float* v = vals + (size_t)w * K;
                    const uint32_t* ix = idx + (shared_idx ? 0 : (size_t)w * K);
                    for (uint32_t j = lo + threadIdx.x; j < hi; j += THREADS) {
                        const uint32_t loc = ix[j] - tile_lo;
                        if (loc < tile_n) acc[loc] = acc[loc] + v[j];
                        else atomicMin(status, ST_DEVICE_CHECK);
                    }
                    __syncthreads();
                }
            }
            __syncthreads();
        }
        float* o = out + tile_lo;
        if (tile_n == ATILE) {
            for (uint32_t i = threadIdx.x; i < ATILE / 4; i += THREADS) {
                float4 a = reinterpret_cast<const float4*>(acc)[i];
                a.x = a.x / fW; a.y = a.y / fW; a.z = a.z / fW; a.w = a.w / fW;
                __stcs(reinterpret_cast<float4*>(o) + i, a);
            }
        } else {
            for (uint32_t i = threadIdx.x; i < tile_n; i += THREADS) o[i] = acc[i] / fW;
        }
        __syncthreads();
    }
}

}  // namespace sc
