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

constexpr uint32_t ATILE = 4096;          // default tile of the dense output
constexpr uint32_t ATILE_BIG = 8192;      // used when the messages are sparse enough to stage a whole tile at once

// bounds[r][t] = first slot j of row r with idx[j] >= t * tile, t = 0..ntiles.
__global__ void __launch_bounds__(THREADS)
agg_bounds_kernel(const uint32_t* __restrict__ idx, uint32_t rows, uint32_t K, uint32_t ntiles, uint32_t tile,
                  uint32_t* __restrict__ bounds) {
    const uint64_t gid = (uint64_t)blockIdx.x * THREADS + threadIdx.x;
    const uint64_t per_row = (uint64_t)ntiles + 1;
    if (gid >= per_row * rows) return;
    const uint32_t r = (uint32_t)(gid / per_row);
    const uint32_t t = (uint32_t)(gid - (uint64_t)r * per_row);
    const uint32_t* row = idx + (size_t)r * K;
    const uint64_t target = (uint64_t)t * tile;
    uint32_t lo = 0, hi = K;                         // first j with row[j] >= target
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if ((uint64_t)__ldg(row + mid) < target) lo = mid + 1; else hi = mid;
    }
    bounds[gid] = lo;
}

// The same bounds when the messages come straight from the one-pass top-k of ONE segment that covers the
// whole row and lies on the aggregate's tile grid: the per-tile message offsets that step has just left ARE
// the bounds (kept coordinates before tile t = first slot with a coordinate >= t * tile), so a row is a copy
// instead of a binary search per tile.  A row whose segment was redone by the fall-back is searched as above.
__global__ void __launch_bounds__(THREADS)
agg_bounds_from_offsets_kernel(const uint32_t* __restrict__ idx, uint32_t rows, uint32_t K, uint32_t ntiles, uint32_t tile,
                               uint32_t* __restrict__ bounds, const uint32_t* __restrict__ offsets, uint32_t off_stride,
                               const FastState* __restrict__ state) {
    const uint64_t gid = (uint64_t)blockIdx.x * THREADS + threadIdx.x;
    const uint64_t per_row = (uint64_t)ntiles + 1;
    if (gid >= per_row * rows) return;
    const uint32_t r = (uint32_t)(gid / per_row);
    const uint32_t t = (uint32_t)(gid - (uint64_t)r * per_row);
    if (state[r].path == PATH_FAST) {
        bounds[gid] = t < ntiles ? offsets[(size_t)r * off_stride + (size_t)t * (tile / 4096u)] : K;
        return;
    }
    const uint32_t* row = idx + (size_t)r * K;
    const uint64_t target = (uint64_t)t * tile;
    uint32_t lo = 0, hi = K;
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if ((uint64_t)__ldg(row + mid) < target) lo = mid + 1; else hi = mid;
    }
    bounds[gid] = lo;
}

constexpr uint32_t AGG_STAGE = 1536;     // message entries staged in shared memory per round

// One CTA per tile of ATILE coordinates.  The slices of all W messages that fall into the
// tile are first fetched together into shared memory (one wave of independent loads), then
// applied to the accumulator worker by worker, so the per-coordinate sum runs in worker
// order without one global-memory round trip per worker.  With shared coordinates every
// slot j carries W values, summed in registers in worker order.
template <uint32_t AT>
__global__ void __launch_bounds__(THREADS)
agg_tiles_kernel(const float* __restrict__ vals, const uint32_t* __restrict__ idx,
                 const uint32_t* __restrict__ bounds, uint32_t W, uint32_t shared_idx, uint32_t K,
                 uint32_t n, uint32_t ntiles, float* __restrict__ out, int* __restrict__ status) {
    __shared__ __align__(16) float acc[AT];
    __shared__ uint32_t st_loc[AGG_STAGE];
    __shared__ float st_val[AGG_STAGE];
    __shared__ uint32_t s_lo[64], s_off[65];
    const float fW = (float)W;
    // Dividing by a power of two equals multiplying by its (exact) reciprocal, bit for bit, and an
    // IEEE division costs about ten instructions: take the product when W allows it.
    const bool pow2 = (W & (W - 1u)) == 0u;
    const float rW = 1.0f / fW;
    for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const uint32_t tile_lo = t * AT;
        const uint32_t tile_n = min(AT, n - tile_lo);
        for (uint32_t i = threadIdx.x; i < AT / 4; i += THREADS)
            reinterpret_cast<float4*>(acc)[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (shared_idx) {
            const uint32_t lo = bounds[t], hi = bounds[t + 1];
            __syncthreads();
            for (uint32_t j = lo + threadIdx.x; j < hi; j += THREADS) {
                const uint32_t loc = idx[j] - tile_lo;
                float sum = 0.0f;
#pragma unroll 8
                for (uint32_t w = 0; w < W; ++w) sum = sum + vals[(size_t)w * K + j];
                if (loc < tile_n) acc[loc] = sum;
                else atomicMin(status, ST_DEVICE_CHECK);
            }
            __syncthreads();
        } else {
            for (uint32_t w0 = 0; w0 < W; w0 += 64) {
                const uint32_t wn = min(64u, W - w0);
                __syncthreads();
                if (threadIdx.x < wn) {
                    const uint32_t* b = bounds + (size_t)(w0 + threadIdx.x) * (ntiles + 1) + t;
                    const uint32_t lo = b[0], hi = b[1];
                    s_lo[threadIdx.x] = lo;
                    s_off[threadIdx.x + 1] = hi - lo;
                }
                __syncthreads();
                if (threadIdx.x == 0) {
                    uint32_t run = 0;
                    s_off[0] = 0;
                    for (uint32_t i = 0; i < wn; ++i) { run += s_off[i + 1]; s_off[i + 1] = run; }
                }
                __syncthreads();
                const uint32_t total = s_off[wn];
                for (uint32_t cs = 0; cs < total; cs += AGG_STAGE) {
                    const uint32_t ce = min(total, cs + AGG_STAGE);
                    for (uint32_t q = cs + threadIdx.x; q < ce; q += THREADS) {
                        uint32_t lo = 0, hi = wn;               // last i with s_off[i] <= q
                        while (hi - lo > 1) {
                            const uint32_t mid = (lo + hi) >> 1;
                            if (s_off[mid] <= q) lo = mid; else hi = mid;
                        }
                        const size_t j = (size_t)(w0 + lo) * K + s_lo[lo] + (q - s_off[lo]);
                        uint32_t loc = idx[j] - tile_lo;
                        float v = vals[j];
                        if (loc >= tile_n) { atomicMin(status, ST_DEVICE_CHECK); loc = 0xFFFFFFFFu; v = 0.0f; }   // never applied
                        st_loc[q - cs] = loc;
                        st_val[q - cs] = v;
                    }
                    __syncthreads();
                    for (uint32_t i = 0; i < wn; ++i) {
                        const uint32_t a = max(s_off[i], cs), b = min(s_off[i + 1], ce);
                        if (a < b) {                             // uniform over the CTA
                            for (uint32_t q = a + threadIdx.x; q < b; q += THREADS) {
                                const uint32_t loc = st_loc[q - cs];
                                if (loc < AT) acc[loc] = acc[loc] + st_val[q - cs];
                            }
                            __syncthreads();
                        }
                    }
                }
            }
            __syncthreads();
        }
        float* o = out + tile_lo;
        if (tile_n == AT) {
            for (uint32_t i = threadIdx.x; i < AT / 4; i += THREADS) {
                float4 a = reinterpret_cast<const float4*>(acc)[i];
                if (pow2) { a.x *= rW; a.y *= rW; a.z *= rW; a.w *= rW; }
                else { a.x = a.x / fW; a.y = a.y / fW; a.z = a.z / fW; a.w = a.w / fW; }
                __stcs(reinterpret_cast<float4*>(o) + i, a);
            }
        } else {
            for (uint32_t i = threadIdx.x; i < tile_n; i += THREADS) o[i] = pow2 ? acc[i] * rW : acc[i] / fW;
        }
        __syncthreads();
    }
}

// The part of one worker's slice that the register rounds of the two kernels below do not cover (dense
// stretches of a message: ties admitted from the lowest coordinate up, a block of the block scheme).  Eight
// rounds of 32 entries are requested together, so that the loop costs one memory latency per 256 entries
// instead of one per 32; the entries of one worker have distinct coordinates, so their order does not matter.
__device__ inline void add_rest_of_slice(const uint32_t* __restrict__ idx_row, const float* __restrict__ val_row, uint32_t from,
                                         uint32_t to, uint32_t base, uint32_t cnt_here, float* acc, uint32_t lane) {
    constexpr int U = 8;
    for (uint32_t j0 = from + lane; j0 < to; j0 += 32u * U) {
        uint32_t ix[U];
        float vv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t j = j0 + 32u * u;
            ix[u] = 0xFFFFFFFFu; vv[u] = 0.0f;
            if (j < to) { ix[u] = __ldg(idx_row + j); vv[u] = __ldg(val_row + j); }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t loc = ix[u] - base;
            if (loc < cnt_here) acc[loc] = acc[loc] + vv[u];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Sparse messages with different coordinates per worker (top-k at the usual densities): one WARP
// owns 1024 coordinates.  It reads, for eight workers at a time, the workers' slices of the
// enclosing 4096-coordinate tile (a few dozen entries each, all loads of the batch in flight
// together), keeps the entries that fall into its own quarter and adds them in worker order.
// No shared staging area, no CTA-wide barrier: the warps of a CTA never wait for each other.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t AWARP = 1024;                 // coordinates per warp

constexpr uint32_t AWARP_BATCH = 8;              // workers whose slices are fetched together
constexpr uint32_t AWARP_MAX_SLICE = 64;         // entries of one worker in one 4096-tile served by the fast loop

template <uint32_t AW>
__global__ void __launch_bounds__(THREADS)
agg_warp_kernel(const float* __restrict__ vals, const uint32_t* __restrict__ idx,
                const uint32_t* __restrict__ bounds /* at ATILE granularity */, uint32_t W, uint32_t K, uint32_t n,
                uint32_t ntiles, float* __restrict__ out, int* __restrict__ status) {
    extern __shared__ __align__(16) float acc_dyn[];                   // WARPS x AW floats
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    float* acc = acc_dyn + warp * AW;
    const float fW = (float)W;
    const bool pow2 = (W & (W - 1u)) == 0u;
    const float rW = 1.0f / fW;
    const uint32_t nq = (n + AW - 1) / AW;                             // warp-owned parts of a tile
    const uint32_t warps_total = gridDim.x * WARPS;
    for (uint32_t q = blockIdx.x * WARPS + warp; q < nq; q += warps_total) {
        const uint32_t t = q / (ATILE / AW);                             // enclosing tile of the bounds table
        const uint32_t base = q * AW;
        const uint32_t cnt_here = min(AW, n - base);
#pragma unroll
        for (int i = 0; i < (int)(AW / 128); ++i)
            reinterpret_cast<float4*>(acc)[i * 32 + lane] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        __syncwarp();
        for (uint32_t w0 = 0; w0 < W; w0 += AWARP_BATCH) {
            uint32_t lo[AWARP_BATCH], hi[AWARP_BATCH];
            uint32_t ix[AWARP_BATCH][2];
            float vv[AWARP_BATCH][2];
#pragma unroll
            for (uint32_t u = 0; u < AWARP_BATCH; ++u) {
                lo[u] = 0; hi[u] = 0;
                if (w0 + u < W) {
                    const uint32_t* b = bounds + (size_t)(w0 + u) * (ntiles + 1) + t;
                    lo[u] = __ldg(b); hi[u] = __ldg(b + 1);
                }
            }
#pragma unroll
            for (uint32_t u = 0; u < AWARP_BATCH; ++u) {
                const size_t row = (size_t)(w0 + u) * K;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t j = lo[u] + 32u * h + lane;
                    ix[u][h] = 0xFFFFFFFFu; vv[u][h] = 0.0f;
                    if (j < hi[u]) { ix[u][h] = __ldg(idx + row + j); vv[u][h] = __ldg(vals + row + j); }
                }
            }
#pragma unroll
            for (uint32_t u = 0; u < AWARP_BATCH; ++u) {                 // worker order
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t loc = ix[u][h] - base;
                    if (loc < cnt_here) acc[loc] = acc[loc] + vv[u][h];
                }
                if (hi[u] - lo[u] > AWARP_MAX_SLICE)                      // a long slice: finish it before the next worker
                    add_rest_of_slice(idx + (size_t)(w0 + u) * K, vals + (size_t)(w0 + u) * K, lo[u] + AWARP_MAX_SLICE, hi[u],
                                      base, cnt_here, acc, lane);
                __syncwarp();
            }
        }
        float* o = out + base;
        if (cnt_here == AW) {
#pragma unroll
            for (int i = 0; i < (int)(AW / 128); ++i) {
                float4 a = reinterpret_cast<const float4*>(acc)[i * 32 + lane];
                if (pow2) { a.x *= rW; a.y *= rW; a.z *= rW; a.w *= rW; }
                else { a.x = a.x / fW; a.y = a.y / fW; a.z = a.z / fW; a.w = a.w / fW; }
                __stcs(reinterpret_cast<float4*>(o) + i * 32 + lane, a);
            }
        } else {
            for (uint32_t i = lane; i < cnt_here; i += 32) o[i] = pow2 ? acc[i] * rW : acc[i] / fW;
        }
        __syncwarp();
    }
    (void)status;
}

// ---------------------------------------------------------------------------------------------
// The same ownership for denser messages (slices of about 50 to 800 entries per worker and
// 4096-tile).  Reading the whole tile slice in each of its four warps would quadruple the
// traffic from L2, so each warp first narrows the tile's slice to its own 1024 coordinates: lane
// u of the lower half searches the first entry >= base for worker u of the batch, lane u of the
// upper half the first entry >= base + 1024 (binary search inside the tile slice, all workers of
// the batch at once).  Then H rounds of 32 entries per worker are fetched for B workers together
// and added in worker order; what exceeds 32 H entries is finished before the next worker.
// ---------------------------------------------------------------------------------------------
template <int H, int B, uint32_t AW>
__global__ void __launch_bounds__(THREADS)
agg_warp_fine_kernel(const float* __restrict__ vals, const uint32_t* __restrict__ idx,
                     const uint32_t* __restrict__ bounds /* at ATILE granularity */, uint32_t W, uint32_t K, uint32_t n,
                     uint32_t ntiles, float* __restrict__ out, int* __restrict__ status) {
    static_assert(B <= 16, "a batch lies inside one group of 16 workers");
    extern __shared__ __align__(16) float acc_dyn[];                   // WARPS x AW floats
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    float* acc = acc_dyn + warp * AW;
    const float fW = (float)W;
    const bool pow2 = (W & (W - 1u)) == 0u;
    const float rW = 1.0f / fW;
    const uint32_t nq = (n + AW - 1) / AW;
    const uint32_t warps_total = gridDim.x * WARPS;
    for (uint32_t q = blockIdx.x * WARPS + warp; q < nq; q += warps_total) {
        const uint32_t t = q / (ATILE / AW);
        const uint32_t base = q * AW;
        const uint32_t cnt_here = min(AW, n - base);
#pragma unroll
        for (int i = 0; i < (int)(AW / 128); ++i)
            reinterpret_cast<float4*>(acc)[i * 32 + lane] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        __syncwarp();
        for (uint32_t g0 = 0; g0 < W; g0 += 16) {
        // boundaries of this quarter inside the tile slices of workers g0 .. g0+15: lane u the first
        // entry, lane 16+u the end; an 8-way search (7 probes in flight per step) keeps the chain of
        // dependent loads to three or four for slices of several hundred entries
        uint32_t found = 0;
        {
            const uint32_t u = lane & 15u, upper = lane >> 4;
            if (g0 + u < W) {
                const uint32_t* b = bounds + (size_t)(g0 + u) * (ntiles + 1) + t;
                uint32_t a = __ldg(b), e = __ldg(b + 1);
                const uint32_t target = base + (upper ? AW : 0u);
                const uint32_t* row = idx + (size_t)(g0 + u) * K;
                const uint32_t qi = q % (ATILE / AW);
                if (!upper && qi == 0) e = a;                             // the tile's own first coordinate
                else if (upper && qi == ATILE / AW - 1) a = e;         // the tile's end
                while (a < e) {
                    const uint32_t len = e - a;
                    uint32_t c = 0;
#pragma unroll
                    for (uint32_t i = 1; i < 8; ++i) c += (__ldg(row + a + ((len * i) >> 3)) < target) ? 1u : 0u;
                    const uint32_t na = c ? a + ((len * c) >> 3) + 1u : a;
                    const uint32_t ne = c < 7 ? a + ((len * (c + 1u)) >> 3) : e;
                    a = na; e = ne;
                }
                found = a;
            }
        }
        const uint32_t gend = min(W, g0 + 16u);
        for (uint32_t w0 = g0; w0 < gend; w0 += B) {
            uint32_t lo[B], hi[B];
#pragma unroll
            for (int u = 0; u < B; ++u) {
                const uint32_t gu = w0 - g0 + u;                               // position in the group of 16
                const uint32_t l = __shfl_sync(0xFFFFFFFFu, found, gu & 15u);
                const uint32_t h = __shfl_sync(0xFFFFFFFFu, found, 16u + (gu & 15u));
                lo[u] = gu < 16u ? l : 0u;
                hi[u] = gu < 16u ? h : 0u;
            }
            uint32_t ix[B][H];
            float vv[B][H];
#pragma unroll
            for (int u = 0; u < B; ++u) {
                const size_t row = (size_t)(w0 + u) * K;
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    const uint32_t j = lo[u] + 32u * h + lane;
                    ix[u][h] = 0xFFFFFFFFu; vv[u][h] = 0.0f;
                    if (j < hi[u]) { ix[u][h] = __ldg(idx + row + j); vv[u][h] = __ldg(vals + row + j); }
                }
            }
#pragma unroll
            for (int u = 0; u < B; ++u) {                                    // worker order
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    const uint32_t loc = ix[u][h] - base;
                    if (loc < cnt_here) acc[loc] = acc[loc] + vv[u][h];
                }
                if (hi[u] - lo[u] > 32u * H)                                 // a long slice: finish it before the next worker
                    add_rest_of_slice(idx + (size_t)(w0 + u) * K, vals + (size_t)(w0 + u) * K, lo[u] + 32u * H, hi[u],
                                      base, cnt_here, acc, lane);
                __syncwarp();
            }
        }
        }
        float* o = out + base;
        if (cnt_here == AW) {
#pragma unroll
            for (int i = 0; i < (int)(AW / 128); ++i) {
                float4 a = reinterpret_cast<const float4*>(acc)[i * 32 + lane];
                if (pow2) { a.x *= rW; a.y *= rW; a.z *= rW; a.w *= rW; }
                else { a.x = a.x / fW; a.y = a.y / fW; a.z = a.z / fW; a.w = a.w / fW; }
                __stcs(reinterpret_cast<float4*>(o) + i * 32 + lane, a);
            }
        } else {
            for (uint32_t i = lane; i < cnt_here; i += 32) o[i] = pow2 ? acc[i] * rW : acc[i] / fW;
        }
        __syncwarp();
    }
    (void)status;
}

// ---------------------------------------------------------------------------------------------
// Aggregate fused with the model update (Algorithm 1, update line: x <- x - q, q read as the
// average): only coordinates that some worker sent are read and written, the dense q is never
// materialised.  x - (+0.0) == x bit for bit, so skipping coordinates whose sum is zero gives
// exactly what the dense formulation gives.
// ---------------------------------------------------------------------------------------------
template <uint32_t AT>
__global__ void __launch_bounds__(THREADS)
agg_apply_tiles_kernel(const float* __restrict__ vals, const uint32_t* __restrict__ idx,
                       const uint32_t* __restrict__ bounds, uint32_t W, uint32_t K, uint32_t n, uint32_t ntiles,
                       float* __restrict__ x, int* __restrict__ status) {
    __shared__ __align__(16) float acc[AT];
    __shared__ uint32_t st_loc[AGG_STAGE];
    __shared__ float st_val[AGG_STAGE];
    __shared__ uint32_t s_lo[64], s_off[65];
    const float fW = (float)W;
    const bool pow2 = (W & (W - 1u)) == 0u;
    const float rW = 1.0f / fW;
    for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const uint32_t tile_lo = t * AT;
        const uint32_t tile_n = min(AT, n - tile_lo);
        bool zeroed = false;
        for (uint32_t w0 = 0; w0 < W; w0 += 64) {
            const uint32_t wn = min(64u, W - w0);
            __syncthreads();
            if (threadIdx.x < wn) {
                const uint32_t* b = bounds + (size_t)(w0 + threadIdx.x) * (ntiles + 1) + t;
                const uint32_t lo = b[0], hi = b[1];
                s_lo[threadIdx.x] = lo;
                s_off[threadIdx.x + 1] = hi - lo;
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t run = 0;
                s_off[0] = 0;
                for (uint32_t i = 0; i < wn; ++i) { run += s_off[i + 1]; s_off[i + 1] = run; }
            }
            __syncthreads();
            const uint32_t total = s_off[wn];
            if (total && !zeroed) {                              // uniform: the tile is touched, start from +0.0
                for (uint32_t i = threadIdx.x; i < AT / 4; i += THREADS)
                    reinterpret_cast<float4*>(acc)[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                zeroed = true;
                __syncthreads();
            }
            for (uint32_t cs = 0; cs < total; cs += AGG_STAGE) {
                const uint32_t ce = min(total, cs + AGG_STAGE);
                for (uint32_t q = cs + threadIdx.x; q < ce; q += THREADS) {
                    uint32_t lo = 0, hi = wn;
                    while (hi - lo > 1) {
                        const uint32_t mid = (lo + hi) >> 1;
                        if (s_off[mid] <= q) lo = mid; else hi = mid;
                    }
                    const size_t j = (size_t)(w0 + lo) * K + s_lo[lo] + (q - s_off[lo]);
                    uint32_t loc = idx[j] - tile_lo;
                    float v = vals[j];
                    if (loc >= tile_n) { atomicMin(status, ST_DEVICE_CHECK); loc = 0xFFFFFFFFu; v = 0.0f; }   // never applied
                    st_loc[q - cs] = loc;
                    st_val[q - cs] = v;
                }
                __syncthreads();
                for (uint32_t i = 0; i < wn; ++i) {
                    const uint32_t a = max(s_off[i], cs), b = min(s_off[i + 1], ce);
                    if (a < b) {                                 // uniform over the CTA
                        for (uint32_t q = a + threadIdx.x; q < b; q += THREADS) {
                            const uint32_t loc = st_loc[q - cs];
                            if (loc < AT) acc[loc] = acc[loc] + st_val[q - cs];
                        }
                        __syncthreads();
                    }
                }
            }
        }
        if (zeroed) {
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < tile_n; i += THREADS) {
                const float a = acc[i];
                if (a != 0.0f) {                                   // also true for NaN
                    // two roundings, as in "average, then subtract": never contracted into one fused multiply-add
                    const float q = pow2 ? __fmul_rn(a, rW) : __fdiv_rn(a, fW);
                    x[tile_lo + i] = __fsub_rn(x[tile_lo + i], q);
                }
            }
        }
        __syncthreads();
    }
}

// All workers kept the same coordinates: one thread per message slot.
__global__ void __launch_bounds__(THREADS)
agg_apply_shared_kernel(const float* __restrict__ vals, const uint32_t* __restrict__ idx, uint32_t W, uint32_t K,
                        uint32_t n, float* __restrict__ x, int* __restrict__ status) {
    const float fW = (float)W;
    const bool pow2 = (W & (W - 1u)) == 0u;
    const float rW = 1.0f / fW;
    for (uint32_t j = blockIdx.x * THREADS + threadIdx.x; j < K; j += gridDim.x * THREADS) {
        const uint32_t i = idx[j];
        float sum = 0.0f;
        for (uint32_t w = 0; w < W; ++w) sum = sum + vals[(size_t)w * K + j];
        if (i >= n) { atomicMin(status, ST_DEVICE_CHECK); continue; }
        if (sum != 0.0f) x[i] = __fsub_rn(x[i], pow2 ? __fmul_rn(sum, rW) : __fdiv_rn(sum, fW));   // never one fused multiply-add
    }
}

}  // namespace sc
