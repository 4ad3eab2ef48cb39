// Host side of the C ABI declared in include/sparsecomm.h: argument checks, scratch
// ownership, the device-side segment table and the launch sequences.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/sparsecomm.h"
#include "sc_aggregate.cuh"
#include "sc_common.cuh"
#include "sc_random.cuh"
#include "sc_topk_fallback.cuh"
#include "sc_topk_tiny.cuh"

using namespace sc;

struct sc_ctx {
    int device = 0;
    int sm_count = 0;
    size_t max_n = 0;
    int max_W = 0, max_seg = 0;
    size_t max_tiles_per_worker = 0;
    size_t max_mask_words = 0;      // per seed group
    size_t max_atiles = 0;
    size_t scratch_bytes = 0;

    SegEntry* d_segs = nullptr;
    uint32_t* d_fast_list = nullptr;
    uint32_t* d_tiny_list = nullptr;      // [max_segments]: short segments, the <= TINY_SMALL_MAX ones first
    uint32_t tiny_small = 0, tiny_large = 0, tiny_large_max_n = 0;
    int occ_tiny_small = 1;
    uint32_t* d_lists = nullptr;     // tiles of the large segments | their pack groups (each max_tiles long)
    uint32_t n_fast_tiles = 0, n_fast_groups = 0;
    uint32_t* d_hist = nullptr;      // radix histograms of the fall-back (cleared by the fall-back kernel itself)
    TopkState* d_state = nullptr;
    unsigned long long* d_desc = nullptr;
    unsigned long long* d_ticket = nullptr;
    uint32_t* d_mask = nullptr;
    uint32_t* d_bounds = nullptr;
    uint32_t* d_offsets = nullptr;   // per seed group / worker: exclusive kept-count prefix over tiles
    // sampled-bracket top-k path.  Everything that must start at zero in a top-k call lies in one block
    // (one memset): counters and the barrier word, then the per-problem states, then the candidate histograms.
    unsigned char* d_zero = nullptr;
    size_t zero_bytes = 0;
    FastState* d_fstate = nullptr;   // inside d_zero
    uint32_t* d_sample = nullptr;
    uint2* d_cand = nullptr;
    uint2* d_list2 = nullptr;
    uint32_t* d_tile_sure = nullptr;
    uint32_t* d_tile_csum = nullptr;
    uint32_t* d_tile_cbase = nullptr;
    uint32_t* d_tile_ccnt = nullptr;
    uint32_t* d_tile_fbase = nullptr;
    uint32_t* d_tile_fcnt = nullptr;
    uint32_t* d_tile_tie = nullptr;
    size_t max_main_grid = 0;            // CTAs of the top-k pass in the build chosen for the current table
    size_t main_grid_v[2] = {0, 0};      // [0]: three CTAs per SM, [1]: the two-CTA build
    int main_wide = 0;                   // 1: the current table uses the two-CTA build
    uint2* d_flagged = nullptr;      // grown on demand: its size depends on k
    size_t flagged_slots = 0;
    size_t max_fast_per_worker = 0, max_cand_per_worker = 0;
    uint32_t last_topk_problems = 0; // (worker, segment) pairs of the most recent top-k call
    uint32_t max_sample_m = 0, fast_big = 0, fast_huge = 0;   // of the fast list: the first fast_huge are long segments, the first fast_big have large samples
    float gamma = 1.0f;                  // step size of the accumulate line (sc_set_gamma)
    int occ_main = 1, occ_main_wide = 1, occ_emit_v[4] = {1, 1, 1, 1}, occ_fallback = 1, occ_filter = 1;
    uint32_t lookback_poll_limit = LOOKBACK_POLL_LIMIT, barrier_poll_limit = BARRIER_POLL_LIMIT;
    uint64_t* d_seeds = nullptr;
    int* d_status = nullptr;

    std::vector<sc_segment> cached_segs;
    size_t cached_n = 0;
    bool layout_valid = false;
    Layout layout{};

    uint32_t epoch = 0;
    uint64_t launches = 0;

    int occ_pack_mask = 1, occ_block = 1, occ_agg = 1, occ_agg_big = 1, occ_agg_warp = 1;
    int occ_agg_fine[5] = {1, 1, 1, 1, 1};

    // optional per-kernel timing (sc_profile)
    bool prof_on = false;
    struct ProfRec { int kind; cudaEvent_t a, b; };
    std::vector<ProfRec> prof_recs;
    std::vector<cudaEvent_t> prof_free;

    // host-buffer entry point
    float* d_stage_grads = nullptr;
    float* d_stage_vals = nullptr;
    uint32_t* d_stage_idx = nullptr;
    float* d_stage_out = nullptr;
    size_t stage_grads_elems = 0, stage_msg_elems = 0, stage_out_elems = 0;
    cudaStream_t copy_stream = nullptr;
    cudaStream_t aux_stream = nullptr;   // short top-k segments run here, beside the large ones
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaEvent_t ev_start = nullptr;
    std::vector<cudaEvent_t> ev_worker;
};

// Top-k of segments below FAST_MIN_N elements runs with the segment in shared memory: one CTA per (worker,
// segment) up to TINY_SMALL_MAX elements (the many very short tensors of a network keep several CTAs per SM),
// a cluster of TINY_CTAS CTAs beyond.
constexpr uint32_t TINY_SMALL_MAX = 4096;        // elements: 16 KB of shared memory

// Emit variants by the average number of flagged entries per tile: 8 or 16 lanes per tile for sparse slices
// (4 or 2 tiles per warp side by side), the whole warp with 4 or 8 entries per lane for longer ones.
constexpr double EMIT_MAX_8 = 12.0, EMIT_MAX_16 = 80.0, EMIT_MAX_32 = 200.0;

namespace {

#define SC_CUDA(call)                                   \
    do {                                                \
        cudaError_t err__ = (call);                     \
        if (err__ != cudaSuccess) return SC_ERR_CUDA;   \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
int dev_alloc(sc_ctx* c, T** p, size_t count) {
    size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
    if (cudaMalloc(reinterpret_cast<void**>(p), bytes) != cudaSuccess) { *p = nullptr; return SC_ERR_WORKSPACE; }
    c->scratch_bytes += bytes;
    return SC_OK;
}

class DeviceGuard {
  public:
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev_); if (prev_ != dev) { cudaSetDevice(dev); set_ = true; } }
    ~DeviceGuard() { if (set_) cudaSetDevice(prev_); }
  private:
    int prev_ = 0;
    bool set_ = false;
};

enum { KIND_SCATTER = 0, KIND_MASK_COUNT, KIND_ROW_SCAN, KIND_RANDK_PACK, KIND_RANDBLOCK, KIND_AGG_BOUNDS, KIND_AGG_TILES,
       KIND_AGG_WARP, KIND_AGG_FINE, KIND_AGG_APPLY, KIND_TINY, KIND_BRACKET, KIND_MAIN, KIND_FILTER, KIND_FINISH, KIND_RESOLVE_SMALL, KIND_EMIT,
       KIND_FALLBACK, KIND_COUNT };
const char* const kKindNames[KIND_COUNT] = {"randk_scatter", "mask_count", "row_scan", "randk_pack", "randblock", "agg_bounds",
                                            "agg_tiles", "agg_warp", "agg_fine", "agg_apply", "topk_tiny", "topk_bracket",
                                            "topk_main", "topk_filter", "topk_finish", "topk_resolve_small", "topk_emit", "topk_fallback"};

// Counts a kernel launch and, when profiling is on, brackets it with two events.
class Launch {
  public:
    Launch(sc_ctx* c, int kind, cudaStream_t st) : c_(c), st_(st) {
        ++c->launches;
        if (!c->prof_on) return;
        rec_.kind = kind;
        rec_.a = take(); rec_.b = take();
        if (rec_.a && rec_.b) { cudaEventRecord(rec_.a, st_); on_ = true; }
    }
    ~Launch() {
        if (!on_) return;
        cudaEventRecord(rec_.b, st_);
        c_->prof_recs.push_back(rec_);
    }
  private:
    cudaEvent_t take() {
        if (!c_->prof_free.empty()) { cudaEvent_t e = c_->prof_free.back(); c_->prof_free.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        return e;
    }
    sc_ctx* c_;
    cudaStream_t st_;
    sc_ctx::ProfRec rec_{};
    bool on_ = false;
};

// Validates the segment table and (re)builds the device copy when it changed.
int prepare_layout(sc_ctx* c, size_t n, const sc_segment* segs, int nseg, cudaStream_t stream) {
    if (c->layout_valid && c->cached_n == n && (int)c->cached_segs.size() == nseg &&
        std::memcmp(c->cached_segs.data(), segs, sizeof(sc_segment) * nseg) == 0)
        return SC_OK;
    // From here on the cached table no longer describes the scratch: a failure below must not let a later
    // call with the old table take the early-out above.  Nothing of the context changes before the new
    // table has been validated.
    c->layout_valid = false;
    int main_wide = 0;
    size_t max_main_grid = 0;
    std::vector<SegEntry> h(nseg + 1);
    std::vector<uint32_t> fast_list, lists[2], tiny_a, tiny_b;
    uint32_t tiny_max_n = 0;
    uint64_t tiles = 0, scat = 0, maskw = 0, msg = 0, end_prev = 0, groups = 0, cand = 0, flag = 0, smp = 0;
    uint32_t fast_count = 0, max_m = 0;
    // Which build of the top-k streaming pass serves this table: the two-CTA build when every large segment is
    // long (more tiles than the three-CTA build has CTAs) and the lists are sparse (at most 3 % flagged).
    {
        uint64_t big_n = 0, big_k = 0;
        bool all_long = true;
        for (int s = 0; s < nseg; ++s) {
            if (segs[s].n < FAST_MIN_N) continue;
            big_n += segs[s].n; big_k += segs[s].k;
            if ((segs[s].n + 31 + TILE - 1) / TILE <= c->main_grid_v[0]) all_long = false;
        }
        main_wide = (big_n > 0 && all_long && 1.05 * (double)big_k <= 0.03 * (double)big_n) ? 1 : 0;
        max_main_grid = c->main_grid_v[main_wide];
    }
    for (int s = 0; s < nseg; ++s) {
        const sc_segment& g = segs[s];
        if (g.offset < end_prev || g.offset > n || g.n > n - g.offset) return SC_ERR_INVALID;
        if (g.k > g.n) return SC_ERR_RANGE;
        end_prev = g.offset + g.n;
        SegEntry e{};
        e.offset = g.offset; e.n = (uint32_t)g.n; e.k = (uint32_t)g.k;
        e.msg_off = (uint32_t)msg; e.tile_begin = (uint32_t)tiles; e.scat_begin = (uint32_t)scat;
        e.mask_word_begin = maskw; e.grp_begin = (uint32_t)groups;
        const uint64_t seg_tiles = (g.n + 31 + TILE - 1) / TILE;   // a tile grid shifted by up to 31 elements
        if (g.n >= FAST_MIN_N) {
            // Sample size.  A larger sample narrows the bracket (candidates ~ 12 sqrt(q (1 - q) / m) n) but costs
            // time itself (one scattered 32-byte read per 8 keys): the two balance at m ~ (n sqrt(q))^(2/3), scaled
            // so that 350 M elements at 10 % kept get 2^20 keys (measured optimum there: 2^18 at 0.1 %, 2^19 at
            // 1 %, 2^20 at 10 %).  The second term keeps the candidates within a fraction of the list capacity.
            const double q = (double)g.k / (double)g.n;
            const double balance = 1048576.0 * std::pow(((double)g.n / 350e6) * std::sqrt(std::max(q, 1e-9) / 0.1), 2.0 / 3.0);
            const double capacity = 230400.0 * q * (1.0 - q);
            uint64_t m = (uint64_t)std::max(balance, capacity);
            m = std::min<uint64_t>(std::min<uint64_t>(m, g.n / 16), SAMPLE_MAX);
            m = std::max<uint64_t>(m, SAMPLE_MIN) & ~7ull;
            // Segments of few tiles whose bracket leaves few candidates are resolved by one CTA each
            // (topk_resolve_small_kernel); the others go through the filter and finish kernels (see below).
            const double candidates = 12.0 * std::sqrt(q * (1.0 - q) / (double)m) * (double)g.n;
            const bool small = seg_tiles <= SMALL_MAX_TILES && candidates <= 16384.0;
            e.fast = small ? 2u : 1u;
            e.sample_m = (uint32_t)m; e.fast_index = fast_count++;
            e.sample_begin = smp; smp += m;
            fast_list.push_back((uint32_t)s);
            // The main pass appends to private regions of the segment's flagged and candidate lists:
            // one region per tile when the segment has no more tiles than the pass has CTAs, else one
            // per CTA (which sees at most ceil(tiles / CTAs) tiles of the segment).  A region holds its
            // tiles' share of (k + slack) resp. slack entries plus a little room per tile.
            const bool per_tile = seg_tiles <= max_main_grid;
            const uint64_t slack = per_tile ? g.n / 16 + 1024 : g.n / 32 + 16384;
            const uint64_t regions = per_tile ? seg_tiles : max_main_grid;
            // (a CTA takes groups of MAIN_GROUP consecutive tiles, every regions-th group: the segment overlaps at
            // most seg_tiles / MAIN_GROUP + 2 groups)
            uint64_t tiles_per_region = 1;                             // (the pass may take smaller groups when the call has few tiles)
            for (uint64_t gsz = 1; !per_tile && gsz <= MAIN_GROUP; gsz *= 2)
                tiles_per_region = std::max(tiles_per_region, gsz * ((seg_tiles / gsz + 2 + regions - 1) / regions));
            const uint64_t cand_region = tiles_per_region * ((slack + seg_tiles - 1) / seg_tiles + 16);
            const uint64_t flag_region = tiles_per_region * ((g.k + slack + seg_tiles - 1) / seg_tiles + 16);
            // Behind the regions lies a pool from which a full region continues (elements above the bracket
            // may crowd in a part of the segment: the dense tensors of a flat vector that is mostly zero rows).
            // Its size covers any distribution of k flagged elements over the tiles; a CTA takes it in chunks.
            const uint64_t chunk = per_tile ? 0 : std::min<uint64_t>(8192, std::max<uint64_t>(1024, 8 * ((g.k + slack) / seg_tiles)));
            const uint64_t pool = g.k + g.n / 64 + 4096 + regions * chunk;
            if (flag_region * regions + pool > 0xFFFFFFF0ull) return SC_ERR_RANGE;
            e.region_per_tile = per_tile ? 1u : 0u;
            e.cand_cap = (uint32_t)cand_region;
            e.flag_cap = (uint32_t)flag_region;
            e.ext_begin = (uint32_t)(flag_region * regions);
            e.ext_cap = (uint32_t)pool;
            e.ext_chunk = (uint32_t)chunk;
            e.cand_begin = cand;
            e.flag_begin = flag;
            e.cov_begin = cand + cand_region * regions;
            e.cov_cap = (uint32_t)(slack / 2 + 4096);
            cand += cand_region * regions + e.cov_cap;
            flag += flag_region * regions + pool;
            max_m = std::max(max_m, e.sample_m);
        } else {                                                       // short: served in shared memory
            (g.n <= TINY_SMALL_MAX ? tiny_a : tiny_b).push_back((uint32_t)s);
            tiny_max_n = std::max<uint32_t>(tiny_max_n, g.n <= TINY_SMALL_MAX ? 0u : (uint32_t)g.n);
        }
        h[s] = e;
        // the fall-back walks the tiles (and pack groups) of the large segments only
        for (uint64_t t = 0; e.fast && t < seg_tiles; ++t) lists[0].push_back((uint32_t)(tiles + t));
        for (uint64_t t = 0; e.fast && t < (seg_tiles + PACK_GROUP - 1) / PACK_GROUP; ++t) lists[1].push_back((uint32_t)(groups + t));
        tiles += seg_tiles;
        groups += (seg_tiles + PACK_GROUP - 1) / PACK_GROUP;
        scat += (g.k + SCAT_CHUNK - 1) / SCAT_CHUNK;
        maskw += (g.n + 31) / 32;
        msg += g.k;
    }
    // The fast list starts with the segments whose sample is large enough for a cluster of CTAs to pay
    // (the bracket kernel takes them eight CTAs at a time, the rest one CTA each); the position in the
    // list is the segment's fast index, and the sample keys are stored in list order.
    // Before them come the segments that the filter and finish kernels serve (they take the cluster form of the
    // bracket kernel whatever their sample); the others are resolved by one CTA each.
    // A table that needs the filter and finish kernels anyway lets a handful of small segments ride along with
    // them instead of paying for a launch of their own.
    {
        uint32_t n_large = 0, n_small = 0;
        for (uint32_t a : fast_list) (h[a].fast == 1u ? n_large : n_small) += 1u;
        if (n_large && n_small < 8u)
            for (uint32_t a : fast_list) h[a].fast = 1u;
    }
    auto rank_of = [&](uint32_t a) { return h[a].fast == 1u ? 2 : h[a].sample_m >= BRACKET_BIG_SAMPLE ? 1 : 0; };
    std::stable_sort(fast_list.begin(), fast_list.end(), [&](uint32_t a, uint32_t b) { return rank_of(a) > rank_of(b); });
    uint32_t big_count = 0, huge_count = 0;
    smp = 0;
    for (size_t i = 0; i < fast_list.size(); ++i) {
        SegEntry& e = h[fast_list[i]];
        e.fast_index = (uint32_t)i;
        e.sample_begin = smp; smp += e.sample_m;
        if (rank_of(fast_list[i]) >= 1) ++big_count;               // the cluster form of the bracket kernel serves these
        if (rank_of(fast_list[i]) == 2) ++huge_count;
    }
    if (tiles > c->max_tiles_per_worker || maskw > c->max_mask_words || tiles > 0xFFFFFFFFull) return SC_ERR_RANGE;
    if (fast_count > c->max_fast_per_worker) return SC_ERR_RANGE;
    const size_t smp_slots = ((size_t)c->max_W * smp + 1) / 2 + 1;  // sample keys are 4 bytes, list entries 8; +1 to align
    if ((size_t)c->max_W * (flag + cand) + smp_slots > c->flagged_slots) {   // the lists follow k: grow them (synchronous, rare)
        SC_CUDA(cudaStreamSynchronize(stream));
        cudaFree(c->d_flagged); c->d_flagged = nullptr; c->d_cand = nullptr; c->d_sample = nullptr;
        c->scratch_bytes -= c->flagged_slots * sizeof(uint2);
        c->flagged_slots = 0;
        const size_t want = (size_t)c->max_W * (flag + cand) + smp_slots;
        if (cudaMalloc(reinterpret_cast<void**>(&c->d_flagged), want * sizeof(uint2)) != cudaSuccess) return SC_ERR_WORKSPACE;
        c->flagged_slots = want;
        c->scratch_bytes += want * sizeof(uint2);
    }
    c->d_cand = c->d_flagged + (size_t)c->max_W * flag;         // candidate lists live behind the flagged lists
    c->d_sample = reinterpret_cast<uint32_t*>(c->d_flagged + (((size_t)c->max_W * (flag + cand) + 1) & ~(size_t)1));   // then the sample keys, 16-byte aligned
    SegEntry sentinel{};
    sentinel.offset = n; sentinel.msg_off = (uint32_t)msg; sentinel.tile_begin = (uint32_t)tiles;
    sentinel.scat_begin = (uint32_t)scat; sentinel.mask_word_begin = maskw; sentinel.grp_begin = (uint32_t)groups;
    h[nseg] = sentinel;
    SC_CUDA(cudaMemcpyAsync(c->d_segs, h.data(), sizeof(SegEntry) * (nseg + 1), cudaMemcpyHostToDevice, stream));
    for (int i = 0; i < 2; ++i)
        if (!lists[i].empty())
            SC_CUDA(cudaMemcpyAsync(c->d_lists + (size_t)i * c->max_tiles_per_worker, lists[i].data(),
                                    sizeof(uint32_t) * lists[i].size(), cudaMemcpyHostToDevice, stream));
    c->n_fast_tiles = (uint32_t)lists[0].size(); c->n_fast_groups = (uint32_t)lists[1].size();
    c->tiny_small = (uint32_t)tiny_a.size(); c->tiny_large = (uint32_t)tiny_b.size(); c->tiny_large_max_n = tiny_max_n;
    tiny_a.insert(tiny_a.end(), tiny_b.begin(), tiny_b.end());
    if (!tiny_a.empty())
        SC_CUDA(cudaMemcpyAsync(c->d_tiny_list, tiny_a.data(), sizeof(uint32_t) * tiny_a.size(), cudaMemcpyHostToDevice, stream));
    if (!fast_list.empty())
        SC_CUDA(cudaMemcpyAsync(c->d_fast_list, fast_list.data(), sizeof(uint32_t) * fast_list.size(),
                                cudaMemcpyHostToDevice, stream));
    Layout L{};
    L.segs = c->d_segs; L.fast_list = c->d_fast_list; L.nseg = (uint32_t)nseg; L.tiles_per_worker = (uint32_t)tiles; L.groups_per_worker = (uint32_t)groups;
    L.scat_per_group = (uint32_t)scat; L.K_total = (uint32_t)msg; L.n_total = n; L.mask_words_per_group = maskw;
    L.cand_per_worker = cand; L.flag_per_worker = flag; L.sample_per_worker = smp; L.fast_per_worker = fast_count;
    c->layout = L;
    c->main_wide = main_wide; c->max_main_grid = max_main_grid;
    c->fast_big = big_count; c->fast_huge = huge_count; c->max_sample_m = max_m;
    c->cached_segs.assign(segs, segs + nseg);
    c->cached_n = n;
    c->layout_valid = true;
    return SC_OK;
}

int check_batch_args(const sc_ctx* c, int scheme, int W, const void* grads, const void* residuals, size_t n,
                     const sc_segment* segs, int nseg, const uint64_t* seeds, const void* out_vals,
                     const void* out_idx) {
    if (!c || !segs || !seeds) return SC_ERR_INVALID;
    if (scheme != SC_TOPK && scheme != SC_RANDK && scheme != SC_RANDBLOCK && scheme != SC_RANDBLOCK_WRAP) return SC_ERR_INVALID;
    if (W < 1 || W > c->max_W || nseg < 1 || nseg > c->max_seg) return SC_ERR_RANGE;
    if (n >= (1ull << 32) || n > c->max_n) return SC_ERR_RANGE;
    uint64_t K = 0;
    for (int s = 0; s < nseg; ++s) {
        if (segs[s].k > segs[s].n) return SC_ERR_RANGE;
        K += segs[s].k;
    }
    if (n > 0 && (!grads || !residuals)) return SC_ERR_INVALID;
    if (K > 0 && (!out_vals || !out_idx)) return SC_ERR_INVALID;
    if (!aligned16(grads) || !aligned16(residuals)) return SC_ERR_INVALID;
    return SC_OK;
}

inline uint32_t persistent_grid(const sc_ctx* c, int occ, uint64_t items) {
    uint64_t cap = (uint64_t)c->sm_count * (uint64_t)std::max(occ, 1);
    return (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(items, cap));
}

// Compression of rows [0, W) of the given base pointers.  `mask_ready` tells the
// random-k path that the membership mask of seed group 0 is already built (used
// when one shared-seed step is issued worker by worker).
// Exclusive scan of `rows` rows of `len` counts: clusters of ROW_SCAN_CTAS CTAs for long rows.
int launch_row_scan(uint32_t* data, uint32_t rows, uint32_t len, cudaStream_t stream) {
    if (rows == 0) return SC_OK;
    if (len < 8192u) {
        row_scan_kernel<1><<<rows, THREADS, 0, stream>>>(data, len);
        return SC_OK;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(rows * ROW_SCAN_CTAS); cfg.blockDim = dim3(THREADS); cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = ROW_SCAN_CTAS; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    SC_CUDA(cudaLaunchKernelEx(&cfg, row_scan_kernel<ROW_SCAN_CTAS>, data, len));
    return SC_OK;
}

// Top-k of the short segments of the table: one CTA per (worker, segment) up to TINY_SMALL_MAX elements, a
// cluster of TINY_CTAS CTAs for the longer ones.
int launch_short_segments(sc_ctx* c, TinyParams tp, int W, cudaStream_t stream) {
    Launch l(c, KIND_TINY, stream);
    if (c->tiny_small) {
        tp.list = c->d_tiny_list; tp.count = c->tiny_small;
        const uint32_t grid = persistent_grid(c, c->occ_tiny_small, (uint64_t)W * c->tiny_small);
        topk_tiny_kernel<1><<<grid, THREADS, TINY_SMALL_MAX * sizeof(float), stream>>>(tp);
    }
    if (c->tiny_large) {
        tp.list = c->d_tiny_list + c->tiny_small; tp.count = c->tiny_large;
        const uint32_t per = (((c->tiny_large_max_n + TINY_CTAS - 1) / TINY_CTAS) + 3u) & ~3u;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((uint32_t)W * c->tiny_large * TINY_CTAS); cfg.blockDim = dim3(THREADS);
        cfg.dynamicSmemBytes = (size_t)per * sizeof(float); cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = TINY_CTAS; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr; cfg.numAttrs = 1;
        SC_CUDA(cudaLaunchKernelEx(&cfg, topk_tiny_kernel<TINY_CTAS>, tp));
    }
    return SC_OK;
}

int compress_rows(sc_ctx* c, int scheme, int W, const float* grads, float* residuals, size_t n,
                  const uint64_t* h_seeds, bool shared_seeds, bool mask_ready,
                  float* out_vals, uint32_t* out_idx, cudaStream_t stream) {
    Layout L = c->layout;
    L.gamma = c->gamma;
    int rc_scan = SC_OK;
    if (n == 0 || L.tiles_per_worker == 0) return SC_OK;
    const uint64_t items64 = (uint64_t)W * L.tiles_per_worker;
    if (items64 > 0xFFFFFFF0ull) return SC_ERR_RANGE;
    const uint32_t items = (uint32_t)items64;
    const uint32_t P = (uint32_t)W * L.nseg;

    if (scheme == SC_TOPK) {
        // one memset for everything that starts at zero: counters, barrier word, problem states, candidate histograms
        const uint32_t PF = (uint32_t)W * L.fast_per_worker;           // fast (worker, segment) pairs
        const size_t state_bytes = ((size_t)P * sizeof(FastState) + 15) & ~(size_t)15;
        uint32_t* counters = reinterpret_cast<uint32_t*>(c->d_zero);
        unsigned int* barrier = reinterpret_cast<unsigned int*>(c->d_zero + 16);
        FastState* fstate = reinterpret_cast<FastState*>(c->d_zero + 64);
        uint32_t* cand_hist = reinterpret_cast<uint32_t*>(c->d_zero + 64 + state_bytes);
        SC_CUDA(cudaMemsetAsync(c->d_zero, 0, 64 + state_bytes + (size_t)PF * CAND_BINS * sizeof(uint32_t), stream));
        c->d_fstate = fstate;
        c->last_topk_problems = P;
        bool forked = false;
        if (c->tiny_small || c->tiny_large) {                          // short segments: one CTA each, in shared memory
            TinyParams tp{};
            tp.L = L; tp.grads = grads; tp.residuals = residuals; tp.out_vals = out_vals; tp.out_idx = out_idx;
            tp.state = fstate; tp.W = (uint32_t)W; tp.status = c->d_status;
            // They touch other segments than the one-pass path below (which is mostly waiting for memory in its
            // small kernels): when the table has both kinds, the short ones run beside it on a stream of their own.
            cudaStream_t main_stream = stream;
            if (L.fast_per_worker && c->aux_stream) {
                SC_CUDA(cudaEventRecord(c->ev_fork, main_stream));
                SC_CUDA(cudaStreamWaitEvent(c->aux_stream, c->ev_fork, 0));
                stream = c->aux_stream;
                forked = true;
            }
            if ((rc_scan = launch_short_segments(c, tp, W, stream)) != SC_OK) return rc_scan;
            if (forked) SC_CUDA(cudaEventRecord(c->ev_join, stream));
            stream = main_stream;
        }
        if (L.fast_per_worker) {
            FastParams fp{};
            fp.L = L; fp.grads = grads; fp.residuals = residuals; fp.out_vals = out_vals; fp.out_idx = out_idx;
            fp.state = fstate; fp.sample = c->d_sample; fp.cand_hist = cand_hist;
            fp.list2 = c->d_list2; fp.cand = c->d_cand; fp.tile_sure = c->d_tile_sure; fp.tile_csum = c->d_tile_csum; fp.tile_cbase = c->d_tile_cbase;
            fp.tile_ccnt = c->d_tile_ccnt; fp.tile_fbase = c->d_tile_fbase; fp.tile_fcnt = c->d_tile_fcnt; fp.tile_tie = c->d_tile_tie;
            fp.flagged = c->d_flagged; fp.offsets = c->d_offsets;
            fp.counters = counters; fp.status = c->d_status; fp.total_items = items;
            { Launch l(c, KIND_BRACKET, stream);
              const uint32_t big = c->fast_big, small = L.fast_per_worker - big;
              if (big) {                                               // clusters of BRACKET_CTAS CTAs, one per problem
                  cudaLaunchConfig_t cfg = {};
                  cfg.gridDim = dim3(big * (uint32_t)W * BRACKET_CTAS); cfg.blockDim = dim3(THREADS); cfg.stream = stream;
                  cudaLaunchAttribute attr;
                  attr.id = cudaLaunchAttributeClusterDimension;
                  attr.val.clusterDim.x = BRACKET_CTAS; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
                  cfg.attrs = &attr; cfg.numAttrs = 1;
                  SC_CUDA(cudaLaunchKernelEx(&cfg, topk_bracket_kernel<BRACKET_CTAS>, fp, 0u, big));
              }
              if (small) topk_bracket_kernel<1><<<small * (uint32_t)W, THREADS, 0, stream>>>(fp, big, small); }
            { Launch l(c, KIND_MAIN, stream);
              // groups of 8 consecutive tiles, fewer when that would leave CTAs without work
              const uint64_t cap = (uint64_t)c->sm_count * (uint64_t)std::max(c->main_wide ? c->occ_main_wide : c->occ_main, 1);
              uint32_t group = MAIN_GROUP;
              while (group > 1u && (items + group - 1) / group < 2 * cap) group /= 2;
              fp.main_group = group;
              const uint64_t groups_of_tiles = (items + group - 1) / group;
              if (c->main_wide) topk_main_kernel<1><<<persistent_grid(c, c->occ_main_wide, groups_of_tiles), THREADS, 0, stream>>>(fp);
              else topk_main_kernel<3><<<persistent_grid(c, c->occ_main, groups_of_tiles), THREADS, 0, stream>>>(fp); }
            const uint32_t huge = c->fast_huge, rest = L.fast_per_worker - huge;
            if (huge) {
            { Launch l(c, KIND_FILTER, stream);
              const uint64_t batches = (items + FILTER_TILES_PER_CTA - 1) / FILTER_TILES_PER_CTA;
              const uint32_t grid = persistent_grid(c, c->occ_filter, batches);
              const uint32_t per_cta = (uint32_t)((batches + grid - 1) / grid) * FILTER_TILES_PER_CTA;
              topk_filter_kernel<<<grid, THREADS, 0, stream>>>(fp, per_cta); }
            { Launch l(c, KIND_FINISH, stream);                        // one cluster per long (worker, segment)
              cudaLaunchConfig_t cfg = {};
              cfg.gridDim = dim3(huge * (uint32_t)W * FINISH_CTAS); cfg.blockDim = dim3(THREADS); cfg.stream = stream;
              cudaLaunchAttribute attr;
              attr.id = cudaLaunchAttributeClusterDimension;
              attr.val.clusterDim.x = FINISH_CTAS; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
              cfg.attrs = &attr; cfg.numAttrs = 1;
              SC_CUDA(cudaLaunchKernelEx(&cfg, topk_finish_kernel<FINISH_CTAS>, fp, 0u, huge)); }
            }
            if (rest) {                                                // segments of few tiles: one CTA each does all of it
                Launch l(c, KIND_RESOLVE_SMALL, stream);
                topk_resolve_small_kernel<<<rest * (uint32_t)W, THREADS, 0, stream>>>(fp, huge, rest);
            }
            { Launch l(c, KIND_EMIT, stream);
              // flagged entries per tile, on average (the list holds the kept elements and a few per cent more)
              const double per_tile = 1.05 * (double)L.K_total * TILE / (double)std::max<size_t>(L.n_total, 1);
              const int v = per_tile <= EMIT_MAX_8 ? 0 : per_tile <= EMIT_MAX_16 ? 1 : per_tile <= EMIT_MAX_32 ? 2 : 3;
              const uint32_t tiles_per_warp = v == 0 ? 4u : v == 1 ? 2u : 1u;
              const uint64_t warps = (items + tiles_per_warp - 1) / tiles_per_warp;
              const uint32_t blocks = persistent_grid(c, c->occ_emit_v[v], (warps + WARPS - 1) / WARPS);
              if (v == 0) topk_emit_kernel<8, 4><<<blocks, THREADS, 0, stream>>>(fp);
              else if (v == 1) topk_emit_kernel<16, 4><<<blocks, THREADS, 0, stream>>>(fp);
              else if (v == 2) topk_emit_kernel<32, 4><<<blocks, THREADS, 0, stream>>>(fp);
              else topk_emit_kernel<32, 8><<<blocks, THREADS, 0, stream>>>(fp); }
            // The fall-back: one cooperative launch, which returns at once unless some segment's bracket missed.
            FallbackParams fb{};
            fb.F = fp;
            fb.K.L = L; fb.K.residuals = residuals; fb.K.out_vals = out_vals; fb.K.out_idx = out_idx;
            fb.K.state = c->d_state; fb.K.fstate = fstate;
            fb.K.wl = WorkList{c->d_lists + c->max_tiles_per_worker, counters, c->n_fast_groups, 0u};
            if (++c->epoch >= (1u << 28)) {        // tags wrapped: forget every old word
                SC_CUDA(cudaMemsetAsync(c->d_desc, 0, (size_t)c->max_W * c->max_tiles_per_worker * 2 * sizeof(unsigned long long), stream));
                c->epoch = 1;
            }
            fb.K.epoch = c->epoch; fb.K.total_items = (uint32_t)W * c->n_fast_groups; fb.K.poll_limit = c->lookback_poll_limit;
            fb.K.ticket = c->d_ticket; fb.K.desc = c->d_desc; fb.K.status = c->d_status;
            fb.hist = c->d_hist; fb.rstate = c->d_state;
            fb.tiles = WorkList{c->d_lists, counters, c->n_fast_tiles, 0u};
            fb.W = (uint32_t)W; fb.poll_limit = c->barrier_poll_limit; fb.barrier = barrier;
            { Launch l(c, KIND_FALLBACK, stream);
              void* args[] = {&fb};
              const uint32_t grid = (uint32_t)c->sm_count * (uint32_t)std::max(c->occ_fallback, 1);
              SC_CUDA(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(topk_fallback_kernel), dim3(grid), dim3(THREADS), args, 0, stream)); }
        }
        if (forked) SC_CUDA(cudaStreamWaitEvent(stream, c->ev_join, 0));
        SC_CUDA(cudaGetLastError());
        return SC_OK;
    }
    SC_CUDA(cudaMemcpyAsync(c->d_seeds, h_seeds, sizeof(uint64_t) * W, cudaMemcpyHostToDevice, stream));

    if (scheme == SC_RANDBLOCK || scheme == SC_RANDBLOCK_WRAP) {
        { Launch l(c, KIND_RANDBLOCK, stream);
          randblock_kernel<<<persistent_grid(c, c->occ_block, (items + STREAM_GROUP - 1) / STREAM_GROUP), THREADS, 0, stream>>>(
              L, grads, residuals, c->d_seeds, out_vals, out_idx, items, scheme == SC_RANDBLOCK_WRAP ? 1u : 0u); }
        SC_CUDA(cudaGetLastError());
        return SC_OK;
    }

    if (scheme == SC_RANDK) {
        const uint32_t groups = shared_seeds ? 1u : (uint32_t)W;
        if (!mask_ready) {
            SC_CUDA(cudaMemsetAsync(c->d_mask, 0, (size_t)groups * L.mask_words_per_group * sizeof(uint32_t), stream));
            const uint64_t blocks = (uint64_t)groups * L.scat_per_group;
            if (blocks > 0x7FFFFFFFull) return SC_ERR_RANGE;
            if (blocks > 0) {
                Launch l(c, KIND_SCATTER, stream);
                randk_scatter_kernel<<<(uint32_t)blocks, THREADS, 0, stream>>>(L, c->d_seeds, c->d_mask, c->d_status);
            }
            const uint64_t warps = (uint64_t)groups * L.tiles_per_worker;
            { Launch l(c, KIND_MASK_COUNT, stream);
              mask_count_kernel<<<(uint32_t)((warps + WARPS - 1) / WARPS), THREADS, 0, stream>>>(
                  L, c->d_mask, groups, c->d_offsets); }
            { Launch l(c, KIND_ROW_SCAN, stream);
              if ((rc_scan = launch_row_scan(c->d_offsets, groups, L.tiles_per_worker, stream)) != SC_OK) return rc_scan; }
        }
        { Launch l(c, KIND_RANDK_PACK, stream);
          randk_pack_kernel<<<persistent_grid(c, c->occ_pack_mask, (items + STREAM_GROUP - 1) / STREAM_GROUP), THREADS, 0, stream>>>(
              L, grads, residuals, c->d_mask, c->d_offsets, shared_seeds ? 0u : 1u, out_vals, out_idx, items,
              c->d_status); }
        SC_CUDA(cudaGetLastError());
        return SC_OK;
    }

    return SC_ERR_INVALID;
}

// Tile of the dense output: the larger one halves the per-tile overhead, but only pays while all
// slices of a tile fit the shared-memory staging area in one round.
// Largest expected slice of one worker per 1024 coordinates served with 2, 4 and 6 rounds of 32 entries held
// in registers (a longer slice is still correct: its remainder is read in a loop of its own).
#ifndef AGG_FINE_Q0
#define AGG_FINE_Q0 43.0
#endif
#ifndef AGG_FINE_Q1
#define AGG_FINE_Q1 120.0
#endif
#ifndef AGG_FINE_Q2
#define AGG_FINE_Q2 200.0
#endif

// Coordinates owned by one warp of agg_warp_kernel (a part of a 4096-tile).
#ifndef SC_AGG_WARP_PART
#define SC_AGG_WARP_PART 2048
#endif
constexpr uint32_t AGG_WARP_PART = SC_AGG_WARP_PART;

inline uint32_t aggregate_tile(int W, size_t k, size_t n) {
    const double per_big_tile = (double)ATILE_BIG * (double)W * (double)k / (double)std::max<size_t>(n, 1);
    return per_big_tile <= 0.9 * AGG_STAGE ? ATILE_BIG : ATILE;
}

// `from_topk`: the messages are those the top-k call on this stream has just written for a table of one segment
// that covers the row on the aggregate's tile grid; its per-tile offsets then serve as the bounds.
int aggregate_rows(sc_ctx* c, int W, const float* vals, const uint32_t* idx, bool shared_idx, size_t k, size_t n,
                   float* out, cudaStream_t stream, bool from_topk = false) {
    if (n == 0) return SC_OK;
    // sparse messages with private coordinates: warp-owned quarter tiles (slices of ~k/n*4096 entries)
    const double slice = (double)k * ATILE / (double)std::max<size_t>(n, 1);       // entries of one worker per 4096-tile
    const bool by_warp = !shared_idx && slice >= 8.0 && slice <= 0.75 * AWARP_MAX_SLICE;
    // denser private coordinates: the same ownership with boundaries per warp-owned part; a part is half a tile
    // while H rounds of 32 entries per worker cover its expected slice, a quarter beyond
    const double half = slice / 2.0, quarter = slice / 4.0;
    const int fine = (shared_idx || by_warp || slice < 8.0) ? -1
                     : half <= AGG_FINE_Q0 ? 0 : half <= AGG_FINE_Q1 ? 1 : half <= 150.0 ? 2
                     : quarter <= AGG_FINE_Q1 ? 3 : quarter <= AGG_FINE_Q2 ? 4 : -1;
    const uint32_t tile = (by_warp || fine >= 0) ? ATILE : aggregate_tile(shared_idx ? 1 : W, k, n);
    const uint32_t ntiles = (uint32_t)((n + tile - 1) / tile);
    const uint32_t rows = shared_idx ? 1u : (uint32_t)W;
    const uint64_t threads = (uint64_t)rows * (ntiles + 1ull);
    { Launch l(c, KIND_AGG_BOUNDS, stream);
      if (from_topk && !shared_idx)
          agg_bounds_from_offsets_kernel<<<(uint32_t)((threads + THREADS - 1) / THREADS), THREADS, 0, stream>>>(
              idx, rows, (uint32_t)k, ntiles, tile, c->d_bounds, c->d_offsets, c->layout.tiles_per_worker + 1u, c->d_fstate);
      else
          agg_bounds_kernel<<<(uint32_t)((threads + THREADS - 1) / THREADS), THREADS, 0, stream>>>(
              idx, rows, (uint32_t)k, ntiles, tile, c->d_bounds); }
    { Launch l(c, by_warp ? KIND_AGG_WARP : fine >= 0 ? KIND_AGG_FINE : KIND_AGG_TILES, stream);
      if (by_warp) {
          const uint64_t nparts = (n + AGG_WARP_PART - 1) / AGG_WARP_PART;
          agg_warp_kernel<AGG_WARP_PART><<<persistent_grid(c, c->occ_agg_warp, (nparts + WARPS - 1) / WARPS), THREADS,
                                           WARPS * AGG_WARP_PART * sizeof(float), stream>>>(
              vals, idx, c->d_bounds, (uint32_t)W, (uint32_t)k, (uint32_t)n, ntiles, out, c->d_status);
      } else if (fine >= 0) {
          const uint32_t part = fine <= 2 ? 2048u : 1024u;
          const uint64_t nparts = (n + part - 1) / part;
          const uint32_t grid = persistent_grid(c, c->occ_agg_fine[fine], (nparts + WARPS - 1) / WARPS);
          const size_t smem = WARPS * part * sizeof(float);
#define SC_FINE_LAUNCH(H, B, AW) agg_warp_fine_kernel<H, B, AW><<<grid, THREADS, smem, stream>>>( \
              vals, idx, c->d_bounds, (uint32_t)W, (uint32_t)k, (uint32_t)n, ntiles, out, c->d_status)
          switch (fine) {
              case 0: SC_FINE_LAUNCH(2, 8, 2048); break;
              case 1: SC_FINE_LAUNCH(4, 4, 2048); break;
              case 2: SC_FINE_LAUNCH(6, 3, 2048); break;
              case 3: SC_FINE_LAUNCH(4, 4, 1024); break;
              default: SC_FINE_LAUNCH(6, 3, 1024); break;
          }
#undef SC_FINE_LAUNCH
      } else {
          const uint32_t grid = persistent_grid(c, tile == ATILE_BIG ? c->occ_agg_big : c->occ_agg, ntiles);
          if (tile == ATILE_BIG)
              agg_tiles_kernel<ATILE_BIG><<<grid, THREADS, 0, stream>>>(
                  vals, idx, c->d_bounds, (uint32_t)W, shared_idx ? 1u : 0u, (uint32_t)k, (uint32_t)n, ntiles, out, c->d_status);
          else
              agg_tiles_kernel<ATILE><<<grid, THREADS, 0, stream>>>(
                  vals, idx, c->d_bounds, (uint32_t)W, shared_idx ? 1u : 0u, (uint32_t)k, (uint32_t)n, ntiles, out, c->d_status);
      } }
    SC_CUDA(cudaGetLastError());
    return SC_OK;
}

// x <- x - average of the W messages, at the coordinates that were sent only.
int apply_rows(sc_ctx* c, int W, const float* vals, const uint32_t* idx, bool shared_idx, size_t k, size_t n, float* x,
               cudaStream_t st) {
    if (n == 0 || k == 0) return SC_OK;
    if (shared_idx) {
        Launch l(c, KIND_AGG_APPLY, st);
        const uint64_t blocks = (k + THREADS - 1) / THREADS;
        agg_apply_shared_kernel<<<persistent_grid(c, 8, blocks), THREADS, 0, st>>>(
            vals, idx, (uint32_t)W, (uint32_t)k, (uint32_t)n, x, c->d_status);
    } else {
        const uint32_t ntiles = (uint32_t)((n + ATILE - 1) / ATILE);
        const uint64_t threads = (uint64_t)W * (ntiles + 1ull);
        { Launch l(c, KIND_AGG_BOUNDS, st);
          agg_bounds_kernel<<<(uint32_t)((threads + THREADS - 1) / THREADS), THREADS, 0, st>>>(
              idx, (uint32_t)W, (uint32_t)k, ntiles, ATILE, c->d_bounds); }
        { Launch l(c, KIND_AGG_APPLY, st);
          agg_apply_tiles_kernel<ATILE><<<persistent_grid(c, c->occ_agg, ntiles), THREADS, 0, st>>>(
              vals, idx, c->d_bounds, (uint32_t)W, (uint32_t)k, (uint32_t)n, ntiles, x, c->d_status); }
    }
    SC_CUDA(cudaGetLastError());
    return SC_OK;
}

int check_aggregate_args(const sc_ctx* c, int W, const void* vals, const void* idx, size_t k, size_t n, const void* out) {
    if (!c) return SC_ERR_INVALID;
    if (W < 1 || W > c->max_W) return SC_ERR_RANGE;
    if (n >= (1ull << 32) || n > c->max_n || k > n) return SC_ERR_RANGE;
    if (n > 0 && !out) return SC_ERR_INVALID;
    if (k > 0 && (!vals || !idx)) return SC_ERR_INVALID;
    if (!aligned16(out)) return SC_ERR_INVALID;
    return SC_OK;
}

bool all_equal(const uint64_t* s, int W) {
    for (int w = 1; w < W; ++w) if (s[w] != s[0]) return false;
    return true;
}

}  // namespace

extern "C" {

const char* sc_strerror(int code) {
    switch (code) {
        case SC_OK: return "ok";
        case SC_ERR_INVALID: return "invalid argument";
        case SC_ERR_RANGE: return "size out of range";
        case SC_ERR_WORKSPACE: return "scratch allocation failed";
        case SC_ERR_CUDA: return "CUDA runtime error";
        case SC_ERR_TIMEOUT: return "bounded device wait timed out";
        case SC_ERR_UNSUPPORTED: return "unsupported";
        case SC_ERR_DEVICE_CHECK: return "device-side range check failed";
        default: return "unknown status";
    }
}

int sc_create(sc_ctx** out, size_t max_n, int max_W, int max_segments) {
    if (!out) return SC_ERR_INVALID;
    *out = nullptr;
    if (max_W < 1 || max_segments < 1 || max_n >= (1ull << 32)) return SC_ERR_RANGE;
    sc_ctx* c = new (std::nothrow) sc_ctx();
    if (!c) return SC_ERR_WORKSPACE;
    if (cudaGetDevice(&c->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) {
        delete c;
        return SC_ERR_CUDA;
    }
    c->max_n = max_n; c->max_W = max_W; c->max_seg = max_segments;
    c->max_tiles_per_worker = (max_n + 31 + TILE - 1) / TILE + (size_t)max_segments + 1;
    c->max_mask_words = (max_n + 31) / 32 + (size_t)max_segments;
    c->max_atiles = (max_n + ATILE - 1) / ATILE;
    const size_t P = (size_t)max_W * max_segments;
    c->max_fast_per_worker = std::min<size_t>((size_t)max_segments, std::max<size_t>(1, max_n >> 16));
    c->max_cand_per_worker = max_n / 32 + c->max_fast_per_worker * 16384;
    const size_t items_max = (size_t)max_W * c->max_tiles_per_worker;
    const size_t fastP = (size_t)max_W * c->max_fast_per_worker;
    c->zero_bytes = 64 + ((P * sizeof(FastState) + 15) & ~(size_t)15) + fastP * CAND_BINS * sizeof(uint32_t);
    int rc = SC_OK;
    if ((rc = dev_alloc(c, &c->d_segs, (size_t)max_segments + 1)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_fast_list, (size_t)max_segments)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tiny_list, (size_t)max_segments)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_lists, 2 * c->max_tiles_per_worker)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_hist, P * HIST_WORDS)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_state, P)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_desc, (size_t)max_W * c->max_tiles_per_worker * 2)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_ticket, 1)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_mask, (size_t)max_W * c->max_mask_words)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_bounds, (size_t)max_W * (c->max_atiles + 1))) == SC_OK &&
        (rc = dev_alloc(c, &c->d_offsets, (size_t)max_W * (c->max_tiles_per_worker + 1))) == SC_OK &&
        (rc = dev_alloc(c, &c->d_zero, c->zero_bytes)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_list2, fastP * LIST2_CAP)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_sure, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_csum, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_cbase, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_ccnt, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_fbase, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_fcnt, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_tile_tie, items_max)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_seeds, (size_t)max_W)) == SC_OK &&
        (rc = dev_alloc(c, &c->d_status, 1)) == SC_OK) {
        bool ok = cudaMemset(c->d_desc, 0, (size_t)max_W * c->max_tiles_per_worker * 2 * sizeof(unsigned long long)) == cudaSuccess &&
                  cudaMemset(c->d_ticket, 0, sizeof(unsigned long long)) == cudaSuccess &&
                  cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess &&
                  cudaMemset(c->d_state, 0, P * sizeof(TopkState)) == cudaSuccess;
        if (!ok) rc = SC_ERR_CUDA;
    }
    if (rc == SC_OK) {
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_main, topk_main_kernel<3>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_main_wide, topk_main_kernel<1>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_tiny_small, topk_tiny_kernel<1>, THREADS, TINY_SMALL_MAX * sizeof(float));
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_fallback, topk_fallback_kernel, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_filter, topk_filter_kernel, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_emit_v[0], topk_emit_kernel<8, 4>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_emit_v[1], topk_emit_kernel<16, 4>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_emit_v[2], topk_emit_kernel<32, 4>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_emit_v[3], topk_emit_kernel<32, 8>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_pack_mask, randk_pack_kernel, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_block, randblock_kernel, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_agg, agg_tiles_kernel<ATILE>, THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_agg_big, agg_tiles_kernel<ATILE_BIG>, THREADS, 0);
        cudaFuncSetAttribute(agg_warp_kernel<AGG_WARP_PART>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(WARPS * AGG_WARP_PART * sizeof(float)));
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_agg_warp, agg_warp_kernel<AGG_WARP_PART>, THREADS,
                                                      WARPS * AGG_WARP_PART * sizeof(float));
        {
#define SC_FINE_SETUP(I, H, B, AW)                                                                                         \
    cudaFuncSetAttribute(agg_warp_fine_kernel<H, B, AW>, cudaFuncAttributeMaxDynamicSharedMemorySize,                      \
                         (int)(WARPS * AW * sizeof(float)));                                                               \
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_agg_fine[I], agg_warp_fine_kernel<H, B, AW>, THREADS,           \
                                                  WARPS * AW * sizeof(float))
            SC_FINE_SETUP(0, 2, 8, 2048); SC_FINE_SETUP(1, 4, 4, 2048); SC_FINE_SETUP(2, 6, 3, 2048);
            SC_FINE_SETUP(3, 4, 4, 1024); SC_FINE_SETUP(4, 6, 3, 1024);
#undef SC_FINE_SETUP
        }
        if (cudaGetLastError() != cudaSuccess) rc = SC_ERR_CUDA;
        c->main_grid_v[0] = (size_t)c->sm_count * (size_t)std::max(c->occ_main, 1);
        c->main_grid_v[1] = (size_t)c->sm_count * (size_t)std::max(c->occ_main_wide, 1);
        c->max_main_grid = c->main_grid_v[0];
    }
    if (rc == SC_OK && (cudaStreamCreateWithFlags(&c->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess))
        rc = SC_ERR_CUDA;
    if (rc != SC_OK) { sc_destroy(c); return rc; }
    *out = c;
    return SC_OK;
}

void sc_destroy(sc_ctx* c) {
    if (!c) return;
    DeviceGuard guard(c->device);
    cudaFree(c->d_segs); cudaFree(c->d_fast_list); cudaFree(c->d_tiny_list); cudaFree(c->d_lists); cudaFree(c->d_hist); cudaFree(c->d_state); cudaFree(c->d_desc);
    cudaFree(c->d_ticket); cudaFree(c->d_mask); cudaFree(c->d_bounds); cudaFree(c->d_offsets); cudaFree(c->d_zero);
    cudaFree(c->d_list2); cudaFree(c->d_tile_sure); cudaFree(c->d_tile_csum); cudaFree(c->d_tile_cbase);
    cudaFree(c->d_tile_ccnt); cudaFree(c->d_tile_fbase); cudaFree(c->d_tile_fcnt); cudaFree(c->d_tile_tie);
    cudaFree(c->d_flagged); cudaFree(c->d_seeds); cudaFree(c->d_status);
    cudaFree(c->d_stage_grads); cudaFree(c->d_stage_vals); cudaFree(c->d_stage_idx); cudaFree(c->d_stage_out);
    for (cudaEvent_t e : c->ev_worker) cudaEventDestroy(e);
    for (auto& r : c->prof_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (cudaEvent_t e : c->prof_free) cudaEventDestroy(e);
    if (c->ev_start) cudaEventDestroy(c->ev_start);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->aux_stream) cudaStreamDestroy(c->aux_stream);
    delete c;
}

int sc_set_gamma(sc_ctx* c, float gamma) {
    if (!c) return SC_ERR_INVALID;
    c->gamma = gamma;
    return SC_OK;
}

int sc_sync_status(sc_ctx* c, void* stream) {
    if (!c) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SC_CUDA(cudaStreamSynchronize(st));
    int h = 0;
    SC_CUDA(cudaMemcpyAsync(&h, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    SC_CUDA(cudaStreamSynchronize(st));
    if (h != 0) {
        SC_CUDA(cudaMemsetAsync(c->d_status, 0, sizeof(int), st));
        SC_CUDA(cudaStreamSynchronize(st));
    }
    return h;
}

int sc_profile(sc_ctx* c, int enable) {
    if (!c) return SC_ERR_INVALID;
    for (auto& r : c->prof_recs) { c->prof_free.push_back(r.a); c->prof_free.push_back(r.b); }
    c->prof_recs.clear();
    c->prof_on = enable != 0;
    return SC_OK;
}

int sc_profile_kinds(void) { return KIND_COUNT; }

const char* sc_profile_name(int kind) { return (kind >= 0 && kind < KIND_COUNT) ? kKindNames[kind] : "?"; }

int sc_profile_read(sc_ctx* c, double* ms, uint64_t* launches) {
    if (!c || !ms || !launches) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    for (int k = 0; k < KIND_COUNT; ++k) { ms[k] = 0.0; launches[k] = 0; }
    for (auto& r : c->prof_recs) {
        SC_CUDA(cudaEventSynchronize(r.b));
        float t = 0.f;
        SC_CUDA(cudaEventElapsedTime(&t, r.a, r.b));
        ms[r.kind] += t;
        launches[r.kind] += 1;
    }
    return SC_OK;
}

int sc_topk_path_counts(sc_ctx* c, void* stream, uint32_t* h_counts) {
    if (!c || !h_counts) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<FastState> h(c->last_topk_problems);
    h_counts[0] = h_counts[1] = h_counts[2] = 0;
    if (h.empty() || !c->d_fstate) return SC_OK;
    SC_CUDA(cudaMemcpyAsync(h.data(), c->d_fstate, h.size() * sizeof(FastState), cudaMemcpyDeviceToHost, st));
    SC_CUDA(cudaStreamSynchronize(st));
    for (const FastState& f : h) {
        if (f.path < 3) ++h_counts[f.path];
        else if (f.path == PATH_TINY) ++h_counts[0];                   // a short segment: radix select in shared memory
    }
    return SC_OK;
}

int sc_topk_path_detail(sc_ctx* c, void* stream, uint32_t* h_counts) {
    if (!c || !h_counts) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<FastState> h(c->last_topk_problems);
    for (int i = 0; i < 8; ++i) h_counts[i] = 0;
    if (h.empty() || !c->d_fstate) return SC_OK;
    SC_CUDA(cudaMemcpyAsync(h.data(), c->d_fstate, h.size() * sizeof(FastState), cudaMemcpyDeviceToHost, st));
    SC_CUDA(cudaStreamSynchronize(st));
    for (const FastState& f : h) {
        if (f.path == PATH_TINY) ++h_counts[0];
        else if (f.path == PATH_FAST) ++h_counts[1];
        else if (f.path == PATH_FAILED) ++h_counts[2];
        if (f.path == PATH_FAST || f.path == PATH_FAILED) {
            if (f.tie_key != TIE_NONE) ++h_counts[3];
            if (f.path == PATH_FAST && f.need_ties) ++h_counts[4];
            if (f.path == PATH_FAILED && f.fail >= FAIL_OVERFLOW && f.fail <= FAIL_SHORT_LIST) ++h_counts[4 + f.fail];
        }
    }
    return SC_OK;
}

int sc_debug_set_poll_limits(sc_ctx* c, uint32_t lookback_polls, uint32_t barrier_polls) {
    if (!c) return SC_ERR_INVALID;
    c->lookback_poll_limit = lookback_polls ? lookback_polls : LOOKBACK_POLL_LIMIT;
    c->barrier_poll_limit = barrier_polls ? barrier_polls : BARRIER_POLL_LIMIT;
    return SC_OK;
}

int sc_debug_wait_probe(sc_ctx* c, int which, void* stream) {
    if (!c || (which != 0 && which != 1)) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PackParams k{};
    if (++c->epoch >= (1u << 28)) {
        SC_CUDA(cudaMemsetAsync(c->d_desc, 0, (size_t)c->max_W * c->max_tiles_per_worker * 2 * sizeof(unsigned long long), st));
        c->epoch = 1;
    }
    k.epoch = c->epoch; k.poll_limit = c->lookback_poll_limit; k.desc = c->d_desc; k.status = c->d_status;
    unsigned int* barrier = reinterpret_cast<unsigned int*>(c->d_zero + 16);
    SC_CUDA(cudaMemsetAsync(barrier, 0, sizeof(unsigned int), st));
    ++c->launches;
    wait_probe_kernel<<<which == 0 ? 2 : 1, THREADS, 0, st>>>(k, barrier, which == 0 ? c->barrier_poll_limit : 0u, which);
    SC_CUDA(cudaGetLastError());
    return SC_OK;
}

size_t sc_scratch_bytes(const sc_ctx* c) { return c ? c->scratch_bytes : 0; }
uint64_t sc_launch_count(const sc_ctx* c) { return c ? c->launches : 0; }

int sc_compress_batch(sc_ctx* c, int scheme, int W, const float* grads, float* residuals, size_t n,
                      const sc_segment* segs, int nseg, const uint64_t* h_seeds,
                      float* out_vals, uint32_t* out_idx, void* stream) {
    int rc = check_batch_args(c, scheme, W, grads, residuals, n, segs, nseg, h_seeds, out_vals, out_idx);
    if (rc != SC_OK) return rc;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = prepare_layout(c, n, segs, nseg, st)) != SC_OK) return rc;
    return compress_rows(c, scheme, W, grads, residuals, n, h_seeds, all_equal(h_seeds, W), false, out_vals, out_idx, st);
}

int sc_compress(sc_ctx* c, int scheme, const float* grad, float* residual, size_t n, size_t k,
                uint64_t seed, float* out_vals, uint32_t* out_idx, void* stream) {
    sc_segment seg{0, n, k};
    return sc_compress_batch(c, scheme, 1, grad, residual, n, &seg, 1, &seed, out_vals, out_idx, stream);
}

int sc_aggregate(sc_ctx* c, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                 float* out, void* stream) {
    int rc = check_aggregate_args(c, W, vals, idx, k, n, out);
    if (rc != SC_OK) return rc;
    DeviceGuard guard(c->device);
    return aggregate_rows(c, W, vals, idx, false, k, n, out, static_cast<cudaStream_t>(stream));
}

int sc_aggregate_shared(sc_ctx* c, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                        float* out, void* stream) {
    int rc = check_aggregate_args(c, W, vals, idx, k, n, out);
    if (rc != SC_OK) return rc;
    DeviceGuard guard(c->device);
    return aggregate_rows(c, W, vals, idx, true, k, n, out, static_cast<cudaStream_t>(stream));
}

int sc_aggregate_apply(sc_ctx* c, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                       float* x, void* stream) {
    int rc = check_aggregate_args(c, W, vals, idx, k, n, x);
    if (rc != SC_OK) return rc;
    DeviceGuard guard(c->device);
    return apply_rows(c, W, vals, idx, false, k, n, x, static_cast<cudaStream_t>(stream));
}

int sc_aggregate_apply_shared(sc_ctx* c, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                              float* x, void* stream) {
    int rc = check_aggregate_args(c, W, vals, idx, k, n, x);
    if (rc != SC_OK) return rc;
    DeviceGuard guard(c->device);
    return apply_rows(c, W, vals, idx, true, k, n, x, static_cast<cudaStream_t>(stream));
}

int sc_step(sc_ctx* c, int scheme, int W, const float* grads, float* residuals, size_t n,
            const sc_segment* segs, int nseg, const uint64_t* h_seeds,
            float* out_vals, uint32_t* out_idx, float* out, void* stream) {
    int rc = check_batch_args(c, scheme, W, grads, residuals, n, segs, nseg, h_seeds, out_vals, out_idx);
    if (rc != SC_OK) return rc;
    if ((n > 0 && !out) || !aligned16(out)) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = prepare_layout(c, n, segs, nseg, st)) != SC_OK) return rc;
    const bool shared = all_equal(h_seeds, W);
    if ((rc = compress_rows(c, scheme, W, grads, residuals, n, h_seeds, shared, false, out_vals, out_idx, st)) != SC_OK)
        return rc;
    // top-k of one large segment that is the whole row, rows on the 128-byte grid: the tiles of the two steps coincide
    const bool one_segment = scheme == SC_TOPK && nseg == 1 && segs[0].offset == 0 && segs[0].n == n &&
                             c->layout.fast_per_worker == 1 && n % 32 == 0 &&
                             (reinterpret_cast<uintptr_t>(residuals) & 127u) == 0;
    return aggregate_rows(c, W, out_vals, out_idx, shared && scheme != SC_TOPK, c->layout.K_total, n, out, st, one_segment);
}

int sc_step_apply(sc_ctx* c, int scheme, int W, const float* grads, float* residuals, size_t n,
                  const sc_segment* segs, int nseg, const uint64_t* h_seeds,
                  float* out_vals, uint32_t* out_idx, float* x, void* stream) {
    int rc = check_batch_args(c, scheme, W, grads, residuals, n, segs, nseg, h_seeds, out_vals, out_idx);
    if (rc != SC_OK) return rc;
    if ((n > 0 && !x) || !aligned16(x)) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = prepare_layout(c, n, segs, nseg, st)) != SC_OK) return rc;
    const bool shared = all_equal(h_seeds, W);
    if ((rc = compress_rows(c, scheme, W, grads, residuals, n, h_seeds, shared, false, out_vals, out_idx, st)) != SC_OK)
        return rc;
    return apply_rows(c, W, out_vals, out_idx, shared && scheme != SC_TOPK, c->layout.K_total, n, x, st);
}

int sc_step_host(sc_ctx* c, int scheme, int W, const float* h_grads, float* residuals, size_t n,
                 const sc_segment* segs, int nseg, const uint64_t* h_seeds, float* h_out, void* stream) {
    // message pointers are internal here; pass non-null placeholders to the checker
    int rc = check_batch_args(c, scheme, W, h_grads, residuals, n, segs, nseg, h_seeds, c, c);
    if (rc != SC_OK) return rc;
    if (n > 0 && !h_out) return SC_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = prepare_layout(c, n, segs, nseg, st)) != SC_OK) return rc;
    const size_t K = c->layout.K_total;
    // staging, grown on demand (first call, or a larger problem)
    if (c->stage_grads_elems < (size_t)W * n) {
        SC_CUDA(cudaStreamSynchronize(st));
        cudaFree(c->d_stage_grads); c->d_stage_grads = nullptr; c->stage_grads_elems = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&c->d_stage_grads), std::max<size_t>((size_t)W * n, 4) * sizeof(float)) != cudaSuccess)
            return SC_ERR_WORKSPACE;
        c->stage_grads_elems = (size_t)W * n;
    }
    if (c->stage_msg_elems < (size_t)W * K) {
        SC_CUDA(cudaStreamSynchronize(st));
        cudaFree(c->d_stage_vals); cudaFree(c->d_stage_idx); c->d_stage_vals = nullptr; c->d_stage_idx = nullptr;
        c->stage_msg_elems = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&c->d_stage_vals), std::max<size_t>((size_t)W * K, 4) * sizeof(float)) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&c->d_stage_idx), std::max<size_t>((size_t)W * K, 4) * sizeof(uint32_t)) != cudaSuccess)
            return SC_ERR_WORKSPACE;
        c->stage_msg_elems = (size_t)W * K;
    }
    if (c->stage_out_elems < n) {
        SC_CUDA(cudaStreamSynchronize(st));
        cudaFree(c->d_stage_out); c->d_stage_out = nullptr; c->stage_out_elems = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&c->d_stage_out), std::max<size_t>(n, 4) * sizeof(float)) != cudaSuccess)
            return SC_ERR_WORKSPACE;
        c->stage_out_elems = n;
    }
    if (!c->copy_stream) SC_CUDA(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
    if (!c->ev_start) SC_CUDA(cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming));
    while ((int)c->ev_worker.size() < W) {
        cudaEvent_t e;
        SC_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        c->ev_worker.push_back(e);
    }
    // copies of worker w+1.. overlap the compression of worker w
    SC_CUDA(cudaEventRecord(c->ev_start, st));
    SC_CUDA(cudaStreamWaitEvent(c->copy_stream, c->ev_start, 0));
    for (int w = 0; w < W; ++w) {
        SC_CUDA(cudaMemcpyAsync(c->d_stage_grads + (size_t)w * n, h_grads + (size_t)w * n, n * sizeof(float),
                                cudaMemcpyHostToDevice, c->copy_stream));
        SC_CUDA(cudaEventRecord(c->ev_worker[w], c->copy_stream));
    }
    const bool shared = all_equal(h_seeds, W);
    for (int w = 0; w < W; ++w) {
        SC_CUDA(cudaStreamWaitEvent(st, c->ev_worker[w], 0));
        rc = compress_rows(c, scheme, 1, c->d_stage_grads + (size_t)w * n, residuals + (size_t)w * n, n,
                           h_seeds + w, shared, shared && w > 0,
                           c->d_stage_vals + (size_t)w * K, c->d_stage_idx + (size_t)w * K, st);
        if (rc != SC_OK) return rc;
    }
    rc = aggregate_rows(c, W, c->d_stage_vals, c->d_stage_idx, shared && scheme != SC_TOPK, K, n, c->d_stage_out, st);
    if (rc != SC_OK) return rc;
    SC_CUDA(cudaMemcpyAsync(h_out, c->d_stage_out, n * sizeof(float), cudaMemcpyDeviceToHost, st));
    SC_CUDA(cudaStreamSynchronize(st));
    return SC_OK;
}

// ---------------------------------------------------------------------------------------------
// sc_aggregate_static: the aggregate without a context, for callers that must not allocate.
// Its scratch (the per-tile message bounds and a status word) lives in the fixed array below,
// which every GPU that loads this library holds until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticMaxN = (size_t)1 << 24;                 // coordinates of the dense output
constexpr int kStaticMaxW = 64;                                   // workers
constexpr size_t kStaticTiles = kStaticMaxN / ATILE;
constexpr size_t kStaticBoundsWords = (size_t)kStaticMaxW * (kStaticTiles + 1);
constexpr size_t kStaticBytes = kStaticBoundsWords * sizeof(uint32_t) + 256;   // bounds, then the status word

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct StaticDevice { unsigned char* base = nullptr; int sm_count = 0; };
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mutex;

// Looks up, once per device and with that device current, where the array lives on it.
int static_scratch_for_current_device(StaticDevice* out) {
    int dev = -1;
    SC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice& d = g_static_dev[dev];
    if (!d.base) {
        void* ptr = nullptr;
        SC_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        int sms = 0;
        SC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (!ptr || sms <= 0) return SC_ERR_CUDA;
        d.sm_count = sms;
        d.base = static_cast<unsigned char*>(ptr);
    }
    *out = d;
    return SC_OK;
}

}  // namespace

int sc_aggregate_static(int W, const float* vals, const uint32_t* idx, size_t k, size_t n, float* out, void* stream) {
    if (W < 1 || W > kStaticMaxW || n > kStaticMaxN || k > n) return SC_ERR_RANGE;
    if ((n > 0 && !out) || (k > 0 && (!vals || !idx)) || !aligned16(out)) return SC_ERR_INVALID;
    if (n == 0) return SC_OK;
    StaticDevice d;
    int rc = static_scratch_for_current_device(&d);
    if (rc != SC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t* bounds = reinterpret_cast<uint32_t*>(d.base);
    int* status = reinterpret_cast<int*>(d.base + kStaticBoundsWords * sizeof(uint32_t));
    // the array keeps whatever the previous call left: the bounds in use are rewritten below,
    // the status word has to start at zero
    SC_CUDA(cudaMemsetAsync(status, 0, sizeof(int), st));
    const uint32_t ntiles = (uint32_t)((n + ATILE - 1) / ATILE);
    const uint64_t threads = (uint64_t)W * (ntiles + 1ull);
    agg_bounds_kernel<<<(uint32_t)((threads + THREADS - 1) / THREADS), THREADS, 0, st>>>(
        idx, (uint32_t)W, (uint32_t)k, ntiles, ATILE, bounds);
    const uint32_t grid = std::max(1u, std::min<uint32_t>(ntiles, (uint32_t)d.sm_count * 4u));
    agg_tiles_kernel<ATILE><<<grid, THREADS, 0, st>>>(vals, idx, bounds, (uint32_t)W, 0u, (uint32_t)k, (uint32_t)n, ntiles,
                                                      out, status);
    SC_CUDA(cudaGetLastError());
    return SC_OK;
}

}  // extern "C"
