/*
 * sparsecomm.h -- C ABI of the sparsified-SGD gradient compressor for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-step hot path of "Sparsified SGD with
 * error-feedback" (Algorithm 1 of "Sparse Communication for Training Deep
 * Networks"): for every worker w
 *     p   = g + e            accumulate the residual   (Algorithm 1, accumulate line; gamma folded into g)
 *     q^w = C(p)             keep k coordinates        (Methodology: Top-k, Random-k, Block-random-k)
 *     e'  = p - q^w          kept coordinates become 0 (Methodology prose on error feedback)
 * and, after the exchange,
 *     q   = (sum_w q^w) / W  dense average             (Algorithm 1, aggregate line; abstract: "average")
 *
 * Conventions
 *  - All data pointers are DEVICE pointers owned by the caller unless a name
 *    starts with h_ (then it is a HOST pointer).  The library never frees them.
 *  - fp32 IEEE-754 round-to-nearest, denormals kept; coordinates are uint32.
 *  - Every call is asynchronous on `stream` (a cudaStream_t passed as void*; NULL
 *    is the legacy default stream) and returns a status code, never throws.
 *    Argument errors are detected on the host before any launch and leave every
 *    buffer untouched.  Problems seen on the device (a bounded wait that ran out,
 *    a coordinate outside its range) set a sticky status word read by
 *    sc_sync_status().
 *  - A context owns scratch memory and is bound to the device that was current
 *    in sc_create().  Use one context per stream; calls on one context must not
 *    overlap on the GPU.
 *  - grad/residual/out must not alias; base pointers must be 16-byte aligned.
 *  - Messages: coordinates ascending and distinct, vals[j] = p[idx[j]].  With a
 *    segment table (layer-wise scope, Methodology "scope of sparsification")
 *    segment s owns message slots [K_s, K_s + k_s), K_s = sum of earlier k, and
 *    its coordinates are global (segment offset added).  Segment s of a call
 *    draws its coordinates from the seed mix64(seed, s).
 */
#ifndef SPARSECOMM_H
#define SPARSECOMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sc_ctx sc_ctx;

/* Compressor C(.) -- Methodology, "compressor or sparsification scheme". */
enum { SC_TOPK = 0,       /* k largest |p|, ties to the lowest coordinate            */
       SC_RANDK = 1,      /* k distinct coordinates from a seeded bijection of [0,n)  */
       SC_RANDBLOCK = 2,  /* one seeded start a in [0,n-k], coordinates a..a+k-1      */
       SC_RANDBLOCK_WRAP = 3 /* start a in [0,n), coordinates (a+j) mod n: a variant of the
                               block scheme (Methodology, Block-random-k) in which every
                               coordinate is kept with the same probability k/n; the
                               message is still ascending (wrapped head first)          */ };

enum { SC_OK = 0,
       SC_ERR_INVALID = -1,      /* null pointer, misaligned base pointer, unknown scheme, bad table */
       SC_ERR_RANGE = -2,        /* k > n, n >= 2^32, W < 1, sizes beyond what the context was made for */
       SC_ERR_WORKSPACE = -3,    /* scratch allocation failed */
       SC_ERR_CUDA = -4,         /* a CUDA runtime call failed */
       SC_ERR_TIMEOUT = -5,      /* a bounded device-side wait gave up (reported by sc_sync_status) */
       SC_ERR_UNSUPPORTED = -6,
       SC_ERR_DEVICE_CHECK = -7  /* a device-side range check failed (e.g. unsorted message) */ };

/* One tensor of the gradient: elements [offset, offset+n) keep k coordinates. */
typedef struct { uint64_t offset, n, k; } sc_segment;

/* Allocates the context and all scratch for problems up to max_n elements per
 * worker, max_W workers and max_segments segments (cudaMalloc; synchronous). */
int sc_create(sc_ctx** out, size_t max_n, int max_W, int max_segments);
void sc_destroy(sc_ctx* ctx);
const char* sc_strerror(int code);

/* Step size of the accumulate line of Algorithm 1, p = gamma * g + e.  The default, 1, is the plain
 * fp32 add (the caller has folded gamma into g).  Any other value makes every later compress call of
 * this context evaluate the line as ONE fused multiply-add per element (a single rounding), so the
 * caller can pass the raw gradient.  Host-side state, no device work; always returns SC_OK for a
 * valid context. */
int sc_set_gamma(sc_ctx* ctx, float gamma);

/* Synchronises `stream`, then returns (and clears) the sticky device status. */
int sc_sync_status(sc_ctx* ctx, void* stream);

/* Bytes of device scratch the context holds; kernels launched so far. */
size_t sc_scratch_bytes(const sc_ctx* ctx);
uint64_t sc_launch_count(const sc_ctx* ctx);

/* Instrumentation (no counterpart in the paper).  sc_profile(ctx, 1) makes every
 * later kernel launch of this context be bracketed by two CUDA events on the
 * launching stream and forgets earlier records; sc_profile(ctx, 0) stops it.
 * sc_profile_read waits for the recorded launches and fills, for each of
 * sc_profile_kinds() kernel kinds (named by sc_profile_name), the summed device
 * time in milliseconds and the number of launches (HOST arrays of that length). */
int sc_profile(sc_ctx* ctx, int enable);
int sc_profile_kinds(void);
const char* sc_profile_name(int kind);
int sc_profile_read(sc_ctx* ctx, double* h_ms, uint64_t* h_launches);

/* Instrumentation (no counterpart in the paper).  Top-k of a segment of 65,536 or
 * more elements first tries a one-pass path whose work depends on a sampled
 * bracket of the threshold; if the exact counts show the bracket missed, it redoes
 * the selection with a multi-pass radix select.  Both give the same bits.  After
 * synchronising `stream` this fills h_counts[3] for the most recent top-k call:
 * (worker, segment) pairs served by [0] the radix select in shared memory because the
 * segment is short, [1] the one-pass path, [2] the radix select after a missed bracket. */
int sc_topk_path_counts(sc_ctx* ctx, void* stream, uint32_t* h_counts);

/* Instrumentation (no counterpart in the paper).  More about the most recent top-k call, after
 * synchronising `stream`: h_counts[8] (HOST) = (worker, segment) pairs [0] served in shared memory
 * (short segments), [1] served by the one-pass path, [2] redone by the radix select; of the large
 * segments: [3] those for which the sample showed one massive key value (a "tie key": exact zeros of a
 * sparse tensor, a constant tensor) whose elements are counted instead of listed, [4] those whose
 * threshold turned out to BE that key (tie-key elements admitted by coordinate order); reasons for
 * [2]: [5] a list overflowed, [6] the exact counts disproved the bracket, [7] too many candidates share
 * the threshold's histogram bin. */
int sc_topk_path_detail(sc_ctx* ctx, void* stream, uint32_t* h_counts);

/* Instrumentation for tests of the bounded device-side waits (no counterpart in the paper).  The
 * fall-back radix select is one kernel whose CTAs meet at grid-wide barriers and whose pack phase looks
 * back at its predecessors' counts; both waits give up after a number of polls, record
 * SC_ERR_TIMEOUT in the status word and let the kernel return.  sc_debug_set_poll_limits changes the
 * two limits for later calls of this context (0 restores the default).  sc_debug_wait_probe launches a
 * small kernel that runs one of the waits where what it waits for never arrives: which = 0, a barrier
 * that expects one CTA more than the launch has; which = 1, a look-back at a count nobody publishes.
 * The kernel returns when the limit is reached (set a small one first); sc_sync_status then reports
 * SC_ERR_TIMEOUT. */
int sc_debug_set_poll_limits(sc_ctx* ctx, uint32_t lookback_polls, uint32_t barrier_polls);
int sc_debug_wait_probe(sc_ctx* ctx, int which, void* stream);

/* Algorithm 1, accumulate + compress + residual lines, one worker, global scope.
 * grad[n] read-only; residual[n] in/out (reads e, writes e'); out_vals[k],
 * out_idx[k] written.  k == 0 is allowed (residual <- gamma g + e, see sc_set_gamma). */
int sc_compress(sc_ctx* ctx, int scheme, const float* grad, float* residual, size_t n, size_t k,
                uint64_t seed, float* out_vals, uint32_t* out_idx, void* stream);

/* Same for W workers and a segment table in one call.  grads and residuals are
 * W rows of n elements (row w at +w*n); segs is a HOST array of nseg segments,
 * ascending and non-overlapping inside [0,n); elements outside every segment
 * are left alone.  h_seeds is a HOST array of W seeds; equal seeds give equal
 * coordinates (workers sharing their seed state, Methodology).  Messages: row w of out_vals /
 * out_idx has K = sum k_s entries (row w at +w*K). */
int sc_compress_batch(sc_ctx* ctx, int scheme, int W, const float* grads, float* residuals, size_t n,
                      const sc_segment* segs, int nseg, const uint64_t* h_seeds,
                      float* out_vals, uint32_t* out_idx, void* stream);

/* Algorithm 1, aggregate line, read as an average: out[i] = (sum over w = 0..W-1,
 * in that order, starting from +0.0, of q^w[i]) / (float)W; untouched i give
 * +0.0.  vals and idx are W rows of k entries, each row ascending and distinct,
 * all coordinates < n.  out[n] is fully overwritten. */
int sc_aggregate(sc_ctx* ctx, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                 float* out, void* stream);

/* The same when all workers kept the same coordinates (the paper's allReduce
 * case): vals is W rows of k, idx is ONE row of k. */
int sc_aggregate_shared(sc_ctx* ctx, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                        float* out, void* stream);

/* Algorithm 1, aggregate line fused with the model-update line (x <- x - q, q read as the
 * average as above): x[i] <- x[i] - (sum over w = 0..W-1, in order, from +0.0, of q^w[i]) / W
 * for every coordinate some worker sent; all other x[i] are left untouched.  The result is
 * bit-identical to computing the dense average with sc_aggregate and subtracting it, but the
 * dense vector is never written or read.  Same message conventions as sc_aggregate; x[n] is
 * updated in place.  The _shared form takes ONE row of coordinates for all workers. */
int sc_aggregate_apply(sc_ctx* ctx, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                       float* x, void* stream);
int sc_aggregate_apply_shared(sc_ctx* ctx, int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                              float* x, void* stream);

/* The paper has no counterpart for this entry point: it is sc_aggregate for callers that
 * are not allowed to allocate device memory.  Every other entry point needs an sc_ctx, and
 * sc_create calls cudaMalloc.  That rules the library out for code that runs after a
 * framework has handed all free device memory to its own pool (a later cudaMalloc fails),
 * and for code inside a latency-critical section, since cudaMalloc may synchronise the
 * whole device.  sc_aggregate_static needs no context and calls no cudaMalloc, cudaFree or
 * any other allocating routine: its scratch (the per-tile message bounds, about 1 MB) is a
 * fixed __device__ array inside the library, present on every GPU that loads the library
 * until the process exits.
 *   - Same arguments and result as sc_aggregate, same bits, for W <= 64 and
 *     n <= 16,777,216.  Anything larger returns SC_ERR_RANGE before touching a buffer.
 *   - The first call on a device looks up the array's address on that device (the device
 *     must be current) and remembers it; make that first call before any stream capture.
 *   - All calls on one GPU share the one array, which keeps the previous call's contents
 *     (what has to start at zero is cleared on `stream` by the call itself).  Two calls
 *     whose kernels can overlap on the GPU (different streams, no ordering) race on it.
 *   - A message that breaks the ascending-coordinate rule is skipped silently here: there
 *     is no context whose status word could report it. */
int sc_aggregate_static(int W, const float* vals, const uint32_t* idx, size_t k, size_t n,
                        float* out, void* stream);

/* One whole step: sc_compress_batch followed by the aggregate over the W
 * messages it produced (the shared-coordinate form when all seeds are equal and
 * the scheme is not top-k).  out[n] receives the dense average. */
int sc_step(sc_ctx* ctx, int scheme, int W, const float* grads, float* residuals, size_t n,
            const sc_segment* segs, int nseg, const uint64_t* h_seeds,
            float* out_vals, uint32_t* out_idx, float* out, void* stream);

/* One whole step of Algorithm 1 without the dense average: sc_compress_batch followed by the
 * model-update line applied at the sent coordinates only, x[i] <- x[i] - (sum over w, in order, from
 * +0.0, of q^w[i]) / W (the same bits as sc_step followed by x - out, see sc_aggregate_apply).  x[n] is
 * updated in place; no dense vector of n elements is written or read besides g, e and the touched x. */
int sc_step_apply(sc_ctx* ctx, int scheme, int W, const float* grads, float* residuals, size_t n,
                  const sc_segment* segs, int nseg, const uint64_t* h_seeds,
                  float* out_vals, uint32_t* out_idx, float* x, void* stream);

/* One whole step with the step's inputs and result in HOST memory: h_grads
 * (W rows of n, ideally pinned) is copied to device staging owned by the
 * context, worker by worker, overlapped with the compression of the previous
 * worker; the dense average is copied back to h_out[n].  residuals stay on the
 * device (they are the only state carried between steps).  The first call
 * allocates the staging (cudaMalloc).  Returns after the result is in h_out. */
int sc_step_host(sc_ctx* ctx, int scheme, int W, const float* h_grads, float* residuals, size_t n,
                 const sc_segment* segs, int nseg, const uint64_t* h_seeds, float* h_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPARSECOMM_H */
