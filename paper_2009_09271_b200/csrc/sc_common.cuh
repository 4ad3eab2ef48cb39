// Shared device-side definitions for the sparsified-SGD compressor kernels (sm_100a).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace sc {

constexpr int THREADS = 256;            // threads per CTA in every tile kernel
constexpr int QUADS = 4;                // float4 per thread per tile
constexpr int TILE = THREADS * QUADS * 4;   // 4096 elements = 16 KB per operand per tile
constexpr int WARPS = THREADS / 32;
constexpr int PACK_GROUP = 8;           // tiles handled per chained-scan step of the pack kernel

constexpr uint32_t HIST0_BINS = 2048;   // key bits 30..20
constexpr uint32_t HIST1_BINS = 1024;   // key bits 19..10
constexpr uint32_t HIST2_BINS = 1024;   // key bits  9..0
constexpr uint32_t HIST_WORDS = HIST0_BINS + HIST1_BINS + HIST2_BINS;

// device status codes (mirrors the public header)
constexpr int ST_TIMEOUT = -5;
constexpr int ST_DEVICE_CHECK = -7;

// One tensor of the gradient as the kernels see it.
struct SegEntry {
    uint64_t offset;          // first element inside a worker row
    uint64_t mask_word_begin; // first 32-bit word of this segment's membership mask
    uint32_t n, k;
    uint32_t msg_off;         // K_s: first message slot of the segment
    uint32_t tile_begin;      // first tile of the segment inside a worker
    uint32_t scat_begin;      // first scatter chunk of the segment inside a seed group
    uint32_t grp_begin;       // first pack group (PACK_GROUP tiles) of the segment inside a worker
    uint32_t fast;            // 1: large segment, top-k goes through the sampled-bracket path
    uint32_t sample_m;        // sample size of that path (multiple of 8)
    uint32_t cand_cap;        // capacity of ONE region of the segment's candidate list
    uint32_t fast_index;      // index among the fast segments of a worker
    uint64_t cand_begin;      // first candidate slot of the segment inside a worker
    uint64_t flag_begin;      // first flagged-list slot of the segment inside a worker
    uint32_t flag_cap;        // capacity of ONE region of the segment's flagged list
    uint32_t region_per_tile; // 1: one list region per tile (few tiles), 0: one per CTA of the main pass
    uint64_t sample_begin;    // first sample key of the segment inside a worker
    uint32_t ext_begin;       // the regions are followed by a pool handed out on demand: its first slot ...
    uint32_t ext_cap;         // ... and its size (a tile or CTA whose region is full continues there)
    uint32_t ext_chunk;       // slots a CTA takes from the pool at a time (0: exactly what the tile needs)
    uint32_t cov_cap;         // candidates that find their tile's slice full go, one by one, to an overflow list ...
    uint64_t cov_begin;       // ... of this size, at this slot of the worker's candidate array
};

struct Layout {
    const SegEntry* segs;     // device array, nseg + 1 entries (last = sentinel with the totals)
    const uint32_t* fast_list; // device array: segment index of the i-th fast segment
    uint32_t nseg;
    uint32_t tiles_per_worker;
    uint32_t groups_per_worker;
    uint32_t scat_per_group;
    uint32_t K_total;         // message entries per worker
    uint64_t n_total;         // elements per worker row
    uint64_t mask_words_per_group;
    uint64_t cand_per_worker; // candidate slots per worker (all fast segments)
    uint64_t flag_per_worker; // flagged-list slots per worker
    uint64_t sample_per_worker; // sample keys per worker
    uint32_t fast_per_worker; // fast segments per worker
    float gamma;              // step size of the accumulate line, p = gamma g + e (1: the plain add)
};

// The tiles (or pack groups) one launch of a radix-select kernel walks: indices inside a worker row,
// the same list for every worker.  The launch returns at once when *gate == 0.
struct WorkList {
    const uint32_t* ids;
    const uint32_t* gate;
    uint32_t len;
    uint32_t pad;
};

// Per (worker, segment) result of the radix select.
struct TopkState {
    uint32_t prefix;   // key bits fixed so far
    uint32_t need;     // how many elements of the current bucket are still to be taken
    uint32_t active;   // 1 while the threshold is not final
    uint32_t T;        // threshold key: every key > T is kept
    uint32_t r;        // number of elements with key == T that are kept (lowest coordinates first)
    uint32_t dual;     // 1 if only some of the ties are kept (r < number of ties)
    uint32_t pad0, pad1;
};

// Top-k of a large segment: state of the sampled-bracket path.
enum { PATH_SLOW = 0,     // small segment: multi-pass radix select
       PATH_FAST = 1,     // bracket holds: single streaming pass + sparse emit
       PATH_FAILED = 2,   // bracket missed or a list overflowed: radix select on the parked p
       PATH_TINY = 3 };   // short segment: one CTA, everything in shared memory
constexpr uint32_t TIE_NONE = 0xFFFFFFFFu;
enum { FAIL_NONE = 0, FAIL_OVERFLOW = 1, FAIL_BRACKET = 2, FAIL_SHORT_LIST = 3 };
struct FastState {
    uint32_t path;
    uint32_t lo, hi;       // bracket: key > hi is surely kept, key < lo surely dropped
    uint32_t shift;        // candidate histogram bin = (key - lo) >> shift
    uint32_t sure_total;   // elements with key > hi
    uint32_t cand_total;   // candidate slots reserved (may exceed the capacity)
    uint32_t lo2, hi2;     // key range of the candidate-histogram bin that holds the threshold
    uint32_t need2;        // 1-based rank of the threshold inside that bin (0: no candidate is kept)
    uint32_t cnt2;         // candidates copied into the short list
    uint32_t T, icut;      // kept <=> key > T, or key == T and coordinate < icut
    uint32_t overflow;     // a list region was full during the main pass
    uint32_t tie_key;      // TIE_NONE, or lo - 1: a key value so frequent in the sample that its elements are
                           // counted per tile instead of being listed (massive ties around the threshold)
    uint32_t tie_total;    // elements with key == tie_key
    uint32_t need_ties;    // how many of them are kept, lowest coordinates first (then T == tie_key)
    uint32_t zcut;         // the streaming pass zeroes flagged elements with key > zcut at once (the sample's estimate of
                           // the threshold; the emit step corrects the few it got wrong)
    uint32_t pad1;
    uint32_t ext_used;     // slots handed out from the flagged list's extension pool
    uint32_t fail;         // FAIL_*: why the one-pass path gave up
    uint32_t expect2;      // entries the short list must hold (from the candidate histogram)
    uint32_t cov_used;     // entries appended to the candidate overflow list (may exceed its capacity)
    uint32_t pad[2];
};

constexpr uint32_t FAST_MIN_N = 1u << 16;
// The top-k streaming pass hands out tiles in groups of MAIN_GROUP consecutive tiles: CTA b takes groups
// b, b + grid, b + 2 grid, ...  Consecutive tiles mostly belong to the same segment, so the per-segment
// bookkeeping of a CTA is flushed once per group instead of once per tile when segments are short.
#ifndef SC_MAIN_GROUP
#define SC_MAIN_GROUP 8
#endif
constexpr uint32_t MAIN_GROUP = SC_MAIN_GROUP;
#ifndef SC_STREAM_GROUP
#define SC_STREAM_GROUP 4
#endif
constexpr uint32_t STREAM_GROUP = SC_STREAM_GROUP;        // the same for the random-k and block-random-k streams
constexpr uint32_t SAMPLE_MIN = 1u << 12, SAMPLE_MAX = 1u << 20;
constexpr uint32_t CAND_BINS = 2048;
constexpr uint32_t LIST2_CAP = 4096;

// ---------------------------------------------------------------------------
// integer hashing (the generator specification; integer-only, so host, device
// and any other implementation agree bit for bit)
// ---------------------------------------------------------------------------
__host__ __device__ inline uint64_t mix64(uint64_t a, uint64_t b) {
    uint64_t z = a + (b + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__host__ __device__ inline uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0x6A09E667u;
    x ^= x >> 15; x *= 0xBB67AE85u;
    x ^= x >> 16;
    return x;
}

constexpr uint64_t SALT_BLOCK = 0x626C6F636Bull;
constexpr uint64_t SALT_RANDK = 0x72616E646B00ull;
constexpr int FEISTEL_ROUNDS = 6;

// Algorithm 1, accumulate line: p = gamma g + e as ONE fused multiply-add (a single rounding);
// fmaf(1, g, e) is the plain fp32 add, bit for bit.
__device__ inline float accumulate(float gamma, float g, float e) { return fmaf(gamma, g, e); }
__device__ inline float4 accumulate(float gamma, const float4& g, const float4& e) {
    return make_float4(fmaf(gamma, g.x, e.x), fmaf(gamma, g.y, e.y), fmaf(gamma, g.z, e.z), fmaf(gamma, g.w, e.w));
}

// Wrap-around variant of the block scheme: the start is uniform on [0, n) and the block is
// {(a + j) mod n : j < k}, which keeps every coordinate with the same probability k / n.
__device__ inline uint32_t block_start_wrap(uint64_t seed_s, uint32_t n) {
    uint64_t h = mix64(seed_s, SALT_BLOCK);
    return (uint32_t)__umul64hi(h, (uint64_t)n);
}

__device__ inline uint32_t block_start(uint64_t seed_s, uint32_t n, uint32_t k) {
    uint64_t h = mix64(seed_s, SALT_BLOCK);
    return (uint32_t)__umul64hi(h, (uint64_t)(n - k) + 1ull);
}

struct Feistel {
    uint32_t keys[FEISTEL_ROUNDS];
    uint32_t left, right, mask_l, mask_r;
};

__device__ inline Feistel feistel_setup(uint64_t seed_s, uint32_t n) {
    Feistel f;
    uint32_t b = (n <= 1u) ? 0u : 32u - (uint32_t)__clz((int)(n - 1u));
    if (b < 2u) b = 2u;
    f.left = b >> 1;
    f.right = b - f.left;
    f.mask_l = (1u << f.left) - 1u;
    f.mask_r = (f.right >= 32u) ? 0xFFFFFFFFu : ((1u << f.right) - 1u);
#pragma unroll
    for (int r = 0; r < FEISTEL_ROUNDS; ++r) f.keys[r] = (uint32_t)(mix64(seed_s, SALT_RANDK + (uint64_t)r) >> 32);
    return f;
}

__device__ inline uint32_t feistel_once(const Feistel& f, uint32_t x) {
    uint32_t L = (x >> f.right) & f.mask_l;
    uint32_t R = x & f.mask_r;
#pragma unroll
    for (int r = 0; r < FEISTEL_ROUNDS; ++r) {
        if ((r & 1) == 0) L ^= mix32(R ^ f.keys[r]) & f.mask_l;
        else              R ^= mix32(L ^ f.keys[r]) & f.mask_r;
    }
    return (L << f.right) | R;
}

// ---------------------------------------------------------------------------
// tile addressing
// ---------------------------------------------------------------------------
// Finds the segment that owns local tile `lt` (thread-uniform, a few cached loads).
__device__ inline uint32_t find_by_tile(const Layout& L, uint32_t lt) {
    uint32_t lo = 0, hi = L.nseg;
    while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (L.segs[mid].tile_begin <= lt) lo = mid; else hi = mid;
    }
    return lo;
}
__device__ inline uint32_t find_by_group(const Layout& L, uint32_t lg) {
    uint32_t lo = 0, hi = L.nseg;
    while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (L.segs[mid].grp_begin <= lg) lo = mid; else hi = mid;
    }
    return lo;
}
__device__ inline uint32_t find_by_scat(const Layout& L, uint32_t ls) {
    uint32_t lo = 0, hi = L.nseg;
    while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (L.segs[mid].scat_begin <= ls) lo = mid; else hi = mid;
    }
    return lo;
}

// A quad is four consecutive elements starting at segment-local element `base`
// (which may be negative or reach past n for the ragged first/last quad).  The
// address seg + base is 16-byte aligned by construction (base pointers are, and
// tiles start on the 128-byte grid).
__device__ inline uint32_t load_quad(const float* seg, long long base, uint32_t n, float v[4]) {
    if (base >= 0 && base + 3 < (long long)n) {
        float4 q = *reinterpret_cast<const float4*>(seg + base);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        return 0xFu;
    }
    uint32_t m = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        long long i = base + c;
        if (i >= 0 && i < (long long)n) { v[c] = seg[i]; m |= 1u << c; } else v[c] = 0.0f;
    }
    return m;
}
__device__ inline uint32_t load_quad_stream(const float* seg, long long base, uint32_t n, float v[4]) {
    if (base >= 0 && base + 3 < (long long)n) {
        float4 q = __ldcs(reinterpret_cast<const float4*>(seg + base));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        return 0xFu;
    }
    uint32_t m = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        long long i = base + c;
        if (i >= 0 && i < (long long)n) { v[c] = __ldcs(seg + i); m |= 1u << c; } else v[c] = 0.0f;
    }
    return m;
}
__device__ inline void store_quad(float* seg, long long base, uint32_t valid, const float v[4]) {
    if (valid == 0xFu) {
        *reinterpret_cast<float4*>(seg + base) = make_float4(v[0], v[1], v[2], v[3]);
        return;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c)
        if ((valid >> c) & 1u) seg[base + c] = v[c];
}

__device__ inline uint32_t key_of(float p) { return __float_as_uint(p) & 0x7FFFFFFFu; }

// Tiles are laid on the 128-byte grid of the row, so that a warp's 512-byte access covers four
// whole cache lines: elements of the segment before its first 128-byte boundary (0..31).
// A persistent kernel knows which tile it takes next.  While a CTA works on a tile (ranking, list and
// message writes) it has no loads in flight, so once the tile's loads have landed each thread asks L2 for
// one 128-byte line of the next tile (g by the lower half of the CTA, e by the upper half) and the next
// round of loads finds its data in L2.  The request must come AFTER the current loads: issued before them
// it made the random-k and block-random-k streams 15-25 % slower, after them it gains 12 % in the top-k
// pass and 1.3 % in the random-k pass (the block-random-k stream already runs at the copy rate).
#ifndef SC_PREFETCH_DIST
#define SC_PREFETCH_DIST 1
#endif
__device__ inline void prefetch_tile_l2(const float* g, const float* e, long long first_next) {
    const float* src = (threadIdx.x < 128u ? g : e) + first_next + (threadIdx.x & 127u) * 32u;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(src));
}

__device__ inline uint32_t misalign_of(const void* p) { return (uint32_t)((reinterpret_cast<uintptr_t>(p) >> 2) & 31u); }

// block-wide exclusive scan of one value per thread (THREADS threads); returns
// the exclusive prefix, *total receives the block sum.  smem: WARPS + 1 words.
__device__ inline uint32_t block_exclusive_scan(uint32_t v, uint32_t* smem, uint32_t* total) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= (uint32_t)d) inc += t;
    }
    if (lane == 31u) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = (lane < (uint32_t)WARPS) ? smem[lane] : 0u;
        uint32_t winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t t = __shfl_up_sync(0xFFFFFFFFu, winc, d);
            if (lane >= (uint32_t)d) winc += t;
        }
        if (lane < (uint32_t)WARPS) smem[lane] = winc - w;
        if (lane == (uint32_t)WARPS - 1u) smem[WARPS] = winc;
    }
    __syncthreads();
    uint32_t res = smem[warp] + inc - v;
    *total = smem[WARPS];
    __syncthreads();
    return res;
}

}  // namespace sc
