/*
 * libfda - Federated Dynamic Averaging (FDA) monitoring and synchronisation on one GPU.
 *
 * The K workers of FDA are K rows of one K x d float32 tensor that lives in the memory of
 * a single device.  Each round the caller runs
 *
 *   fda_local_state      -> S^(k) = (||u^(k)||^2, <xi,u^(k)>, sk(u^(k))),  u^(k) = w^(k) - w_t0
 *   fda_combine_estimate -> S-bar = mean_k S^(k), H(S-bar), trigger = (H > Theta)
 *   fda_average_models   -> w^(k) := w-bar = mean_k w^(k)  (and w_t0 := w-bar) if triggered
 *
 * which are the monitoring and synchronisation steps of Algorithm 1 of the FDA paper (Section 3)
 * with the two AllReduce steps replaced by reductions over rows in device memory.
 *
 * Conventions
 *   - plain C ABI; every function returns an fda_status and never throws or aborts;
 *   - unless a parameter says "host", pointers are DEVICE pointers to memory owned by the
 *     caller; the library never frees or reallocates caller memory;
 *   - the context owns its own device scratch (list schedule, per-block partial sums);
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream); calls
 *     enqueue work and return, unless stated otherwise;
 *   - arguments are validated on the host before anything is launched; an invalid call
 *     launches nothing and leaves its outputs untouched;
 *   - one context serves one stream at a time (calls on the same context must not overlap
 *     on the device, because they share the context's scratch).
 *
 * State layout (float32, state_len = 2 + l*m per worker, row-major):
 *   [0]              ||u^(k)||^2                                   (Section 3, local state)
 *   [1]              <xi, u^(k)>                                   (Theorem 2, LinearFDA)
 *   [2 + i*m + c]    cell c of row i of the AMS sketch sk(u^(k))   (Theorem 1, SketchFDA)
 */
#ifndef FDA_H_
#define FDA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fda_ctx fda_ctx; /* opaque, library-owned */

typedef enum {
    FDA_OK = 0,
    FDA_ERR_INVALID_ARG = 1, /* NULL pointer, size out of range, bad flag               */
    FDA_ERR_UNSUPPORTED = 2, /* valid request the kernels cannot serve (sketch too big) */
    FDA_ERR_CUDA = 3,        /* a CUDA runtime call failed; see fda_last_error          */
    FDA_ERR_NOMEM = 4        /* host or device allocation failed                        */
} fda_status;

/* Which parts of the local state fda_local_state computes; parts not asked for are
 * written as 0. */
enum { FDA_STATE_NORM = 1, FDA_STATE_LINEAR = 2, FDA_STATE_SKETCH = 4 };
/* Estimator used by fda_combine_estimate. */
enum { FDA_VARIANT_LINEAR = 0, FDA_VARIANT_SKETCH = 1 };
/* fda_average_models flags. */
enum {
    FDA_AVG_BROADCAST = 1,     /* also overwrite every w^(k) with w-bar (in-place sync) */
    FDA_AVG_UNCONDITIONAL = 2  /* ignore the trigger flag of the estimate               */
};

#define FDA_MAX_ROWS 16 /* largest supported number of sketch rows l */

/* Result of fda_combine_estimate. */
typedef struct {
    float mean_sq_norm;        /* (1/K) sum_k ||u^(k)||^2                              */
    float est_sq_norm_of_mean; /* the estimate of ||u-bar||^2 that H subtracts         */
    float H;                   /* variance over-estimate                               */
    float theta;               /* the threshold it was compared with                   */
    int32_t trigger;           /* 1 if H > theta (strictly), else 0                    */
    int32_t l;                 /* number of valid entries of row_sq_norm               */
    float row_sq_norm[FDA_MAX_ROWS]; /* ||row i of the averaged sketch||^2             */
} fda_estimate;

/*
 * Create a context on CUDA device `device` for sketches of l rows x m columns.
 *   hash_coeffs  HOST pointer to 6*l uint64 values, per row {a, b, c3, c2, c1, c0}, each in
 *                [0, 2^61-2], a != 0 and c3 != 0.  They define the AMS hash family
 *                (Section 3.1 cites the sketch but prints no family; this is the classical
 *                2-wise bucket / 4-wise sign construction over p = 2^61-1):
 *                  bucket_i(j) = ((a*j + b) mod p) mod m
 *                  sign_i(j)   = +1 if ((((c3*j + c2)*j + c1)*j + c0) mod p) is even, else -1
 *                May be NULL when l == 0 (a context without sketch: state_len = 2).
 *   d_max, K_max largest model dimension / worker count later calls will use; they size
 *                the context's scratch.
 * Device memory the context takes (fda_context_info reports the figures):
 *   - per-block partial sums: (SM count) * l*m * 128 bytes plus 64 * (SM count) * max(K_max, 32) bytes;
 *   - the list schedule of the sketch kernel, when the sketch allows one (tiles of at least 6*m
 *     indices fit the shared memory): about 2.4 * l bytes per index of d_max (2.4 GB for
 *     d_max = 2 * 10^8 and l = 5), built here in about 4 ms per million indices; it is dropped,
 *     and sketch requests are then served by the slower plain-load kernels, when it would take
 *     more than a third of the free device memory (see fda_create_limited for another cap);
 *   - lazily, by the first call that needs them: a 16-bit hash table of 2*l bytes per index
 *     (sketch requests on a context without a schedule), d_max floats (fda_mean_state with
 *     more than 2*l workers, or without a schedule), K_max*d_max floats of staging
 *     (fda_round_host).
 * Blocking: allocates, builds the schedule, synchronises the device.
 * Errors: INVALID_ARG (out == NULL, l < 0 or > FDA_MAX_ROWS, m < 1 or > 32768 with l > 0,
 * d_max < 1 or >= 2^31, K_max < 1, coefficient out of range), UNSUPPORTED (l*m too large
 * for the shared-memory bins), NOMEM, CUDA.
 */
fda_status fda_create(fda_ctx **out, int device, int l, int m, const uint64_t *hash_coeffs,
                      int64_t d_max, int K_max);

/*
 * fda_create with a cap on the list schedule (the paper has no counterpart): the schedule is
 * kept only if it takes at most `schedule_limit_bytes` (and a third of the free device memory);
 * 0 means no cap of the caller's (fda_create), a negative value builds no schedule at all.
 * Other arguments and errors as fda_create.
 */
fda_status fda_create_limited(fda_ctx **out, int device, int l, int m, const uint64_t *hash_coeffs,
                              int64_t d_max, int K_max, int64_t schedule_limit_bytes);

/*
 * What the context holds (the paper has no counterpart).  info (host, 8 values):
 *   [0] device bytes the context owns now   [1] of which: the list schedule (0: none)
 *   [2] 1 when sketch requests run on the list kernel, 0 when on the plain-load kernels
 *   [3] indices per tile of the schedule    [4] bytes of a schedule that was built and dropped
 *       for lack of memory (0: none)        [5] bytes of the lazily built 16-bit hash table
 *   [6] microseconds fda_create spent on the schedule   [7] other lazily allocated bytes.
 * Errors: INVALID_ARG (NULL).
 */
fda_status fda_context_info(const fda_ctx *ctx, int64_t *info);

/* Free the context and its scratch.  Blocking (synchronises the device). NULL is a no-op. */
fda_status fda_destroy(fda_ctx *ctx);

/* Floats per worker state: 2 + l*m. 0 if ctx == NULL. */
size_t fda_state_len(const fda_ctx *ctx);

/* HOST string describing the last error on this context (empty if none). */
const char *fda_last_error(const fda_ctx *ctx);

/*
 * Local states of all K workers in one pass over w (Section 3: local drift, local state;
 * Section 3.1: sk(.); Section 3.2: <xi,u>).
 *   w           K rows of d floats, row k at w + k*row_stride (row_stride >= d, elements)
 *   w_t0        d floats, model after the last synchronisation
 *   xi          d floats (unit vector of LinearFDA) or NULL; used only with FDA_STATE_LINEAR
 *   flags       OR of FDA_STATE_*; FDA_STATE_SKETCH needs l > 0
 *   states      out, K x state_len floats
 * Any alignment of w, w_t0, xi is accepted; 16-byte aligned pointers with row_stride a
 * multiple of 4 take the vector path.  Errors: INVALID_ARG (NULL, K < 1 or > K_max, d < 1
 * or > d_max, row_stride < d, unknown flag, SKETCH without a sketch), UNSUPPORTED (more worker
 * groups than the context's partial-sum scratch holds: K above 4 x the SM count with a list
 * schedule, above 32 x the SM count without; nothing is launched), CUDA.
 * Stream order: the call's work starts after what `stream` held before it and is complete before
 * anything enqueued on `stream` after it.  Part of it may run on a second stream that the context
 * owns (forked from and joined to `stream` with events; also legal while `stream` is being
 * captured into a graph), which is why a context serves one stream at a time.
 */
fda_status fda_local_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                           const float *w_t0, const float *xi, uint32_t flags, float *states,
                           void *stream);

/*
 * Averaged state S-bar in one pass, without the K per-worker states: mean_state (one row of
 * state_len floats) = ( (1/K) sum_k ||u^(k)||^2, (1/K) sum_k <xi,u^(k)>, sk(u-bar) ) with
 * u-bar = (1/K) sum_k u^(k).  By the linearity of the sketch (Section 3.1, property (a); the
 * "(lin.)" step in the proof of Theorem 1) sk(u-bar) equals the average of the K worker
 * sketches that Algorithm 1 forms when it averages the states, so fda_combine_estimate(ctx, mean_state, K = 1, ...)
 * yields the same H and trigger as the per-worker route, with l instead of K*l bin updates
 * per index.  Arguments and errors as fda_local_state; mean_state is state_len floats.  On a
 * context with a list schedule the cells come from the list kernel: in one pass over the K rows
 * for K <= 2*l, else from the vector of averaged drifts that a first pass leaves in device
 * memory; that vector (d_max floats) is allocated by the first call that needs it (NOMEM if that
 * fails), and so is the 16-bit hash table on a context without a schedule.
 */
fda_status fda_mean_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                          const float *w_t0, const float *xi, uint32_t flags, float *mean_state,
                          void *stream);

/*
 * Average the K states and evaluate the variance over-estimate (Algorithm 1: the state average and
 * the variance test).
 *   FDA_VARIANT_SKETCH: H = S-bar[0] - median_i ||row_i(S-bar sketch)||^2 / (1 + epsilon)
 *                       (Theorem 1; the median of an even number of rows is the mean of
 *                       the two middle values);
 *   FDA_VARIANT_LINEAR: H = S-bar[0] - S-bar[1]^2                            (Theorem 2).
 *   trigger = (H > theta).  Accumulation is in fp64, results are rounded to fp32.
 *   states      K x state_len floats (as written by fda_local_state)
 *   est_dev     out, DEVICE fda_estimate
 *   est_host    out, HOST fda_estimate or NULL.  If not NULL the call copies the result
 *               and synchronises `stream` before returning.
 * Errors: INVALID_ARG (NULL, K < 1 or > K_max, bad variant, SKETCH variant with l == 0,
 * epsilon <= -1 or not finite, theta not finite), CUDA.
 */
fda_status fda_combine_estimate(fda_ctx *ctx, const float *states, int K, int variant,
                                float epsilon, float theta, fda_estimate *est_dev,
                                fda_estimate *est_host, void *stream);

/*
 * Synchronise: w-bar[j] = (1/K) sum_k w^(k)[j] (fp32, summed in the order k = 0..K-1), then
 * w_t0 := w-bar and, with FDA_AVG_BROADCAST, every w^(k) := w-bar in place (Section 3: the
 * workers synchronise with an AllReduce of their models; the synchronisation step of Algorithm 1).
 *   est_dev     DEVICE fda_estimate whose `trigger` gates the whole operation on the
 *               device (nothing is read or written when it is 0); NULL or
 *               FDA_AVG_UNCONDITIONAL averages always.
 * Errors: INVALID_ARG (NULL w or w_t0, K < 1, d < 1, row_stride < d, unknown flag), CUDA.
 */
fda_status fda_average_models(fda_ctx *ctx, float *w, int64_t row_stride, int K, int64_t d,
                              float *w_t0, const fda_estimate *est_dev, uint32_t flags,
                              void *stream);

/*
 * fda_average_models that also refreshes the LinearFDA direction (Section 3.2, the heuristic
 * choice of xi; Table 1): xi_out := (w-bar_new - w_t0_old) / ||w-bar_new - w_t0_old||, the
 * normalised step of the global model between the last two synchronisations, computed in the
 * same pass that averages (w_t0 is read before it is overwritten).  xi_out is d floats and is
 * left untouched when the gate does not fire; it becomes all zero when the step is exactly
 * zero.  xi_out must not alias w or w_t0.  Errors as fda_average_models, plus INVALID_ARG for
 * a NULL xi_out.
 */
fda_status fda_average_models_xi(fda_ctx *ctx, float *w, int64_t row_stride, int K, int64_t d,
                                 float *w_t0, float *xi_out, const fda_estimate *est_dev,
                                 uint32_t flags, void *stream);

/*
 * One whole round on HOST buffers: copies w, w_t0 and xi to device staging owned by the
 * context (allocated on first use for K_max x d_max), runs fda_local_state,
 * fda_combine_estimate and fda_average_models (FDA_AVG_BROADCAST, gated by the trigger) and
 * copies back the states, the estimate and - only if the round triggered - the averaged
 * model into w_t0_host (and into every row of w_host when `avg_flags` has
 * FDA_AVG_BROADCAST).  Blocking.  Pinned host buffers make the copies asynchronous to the
 * host but the call still waits for completion.
 *   states_host  out, K x state_len floats, may be NULL
 *   est_host     out, required
 * Errors: as the three calls above, plus NOMEM for the staging buffers.
 */
fda_status fda_round_host(fda_ctx *ctx, float *w_host, int64_t row_stride, int K, int64_t d,
                          float *w_t0_host, const float *xi_host, uint32_t state_flags,
                          int variant, float epsilon, float theta, uint32_t avg_flags,
                          float *states_host, fda_estimate *est_host, void *stream);

/*
 * Hash dump for parity checks: for indices j0 .. j0+n-1 and every row i < l writes
 * buckets[i*n + t] = bucket_i(j0+t) and signs[i*n + t] = sign_i(j0+t) (+1 / -1), evaluated
 * directly from the coefficients (not read from the context's table).
 * Errors: INVALID_ARG (NULL, l == 0, j0 < 0, n < 1, j0 + n > 2^31), CUDA.
 */
fda_status fda_debug_hash(fda_ctx *ctx, int64_t j0, int64_t n, uint16_t *buckets,
                          int8_t *signs, void *stream);

/*
 * Read-only bandwidth probe (the paper has no counterpart): streams src[0..n) once with the
 * access pattern of the bandwidth-bound kernels and writes the sum of its elements to
 * *sum_out (device, one float; fp32 per thread, fp64 across threads, fixed order).  Timing
 * this call gives the rate a kernel that only reads reaches on the device, which is the
 * yardstick quoted beside the local-state and averaging kernels.  src need not be aligned.
 * Uses the context's partial-sum scratch: not concurrent with other calls on the context.
 * Errors: INVALID_ARG (NULL, n < 1), CUDA.
 */
fda_status fda_debug_read_probe(fda_ctx *ctx, const float *src, int64_t n, float *sum_out,
                                void *stream);

/*
 * Copy of one record of the list schedule that k_local_state_gather walks (the paper has no
 * counterpart; Section 3.1 only fixes what the sketch sums).  The record of a tile lists the
 * tile's indices cell by cell for every sketch row.  Layout (byte offsets):
 *   [0] u32 items  [4] u32 bytes of the record  [8] u32 entry chunks  [12] u32 0
 *   [16] items x { u16 steps, u16 cell block, u32 first chunk }, most steps first
 *   cells_offset = 16 + 8*items rounded up to 64: cell blocks of 32 u16, the cell index
 *       row*m + bucket of the list a lane walks (bit 15 set when the cell has several lists,
 *       l*m when the lane has none)
 *   entries_offset = cells_offset + 64*items rounded up to 256: chunks of 256 bytes,
 *       chunk[lane][4] u16 entries for steps 4c .. 4c+3 of an item; entry = row of the drift
 *       tile (bits 0..12) | sign << 15, where index r of the tile is stored in row
 *       r ^ ((r >> 3) & 3) and rows tile_indices + r, r < 8, are padding (zeros).
 * In every step the eight lanes 8q .. 8q+7 of an item address rows in eight different 16-byte
 * bank groups (row mod 8), so that the shared-memory load of the step is conflict free.
 * record_host: host buffer of `capacity` bytes, receives min(capacity, record_bytes) bytes.
 * info (host, 8 values): tile_indices, lanes per item (32), longest list (64), record_bytes,
 * tiles in the schedule, padding rows (8), lanes per pass (8), bytes of the whole schedule.
 * Synchronises the device.
 * Errors: INVALID_ARG (NULL, tile out of range), UNSUPPORTED (the context has no schedule:
 * no sketch, lists too short for it, or not enough free memory at fda_create), CUDA.
 */
fda_status fda_debug_schedule(const fda_ctx *ctx, int64_t tile, void *record_host, size_t capacity,
                              int64_t *info);

/*
 * Name of the kernel that served the context's last fda_local_state or fda_mean_state call (the
 * paper has no counterpart): "k_local_state_gather" (sketch pass over per-cell index lists: every sketch request
 * on a context that holds a list schedule), "k_local_state_linear" (no sketch requested),
 * "k_local_state_fast" / "k_local_state" (sketch requests without a schedule: aligned rows with 5
 * or 7 sketch rows / everything else); for fda_mean_state "k_mean_state_gather" (one pass on
 * the list kernel), "k_mean_model + k_mean_state_gather" (averaged drifts, then the list
 * kernel on them), "k_mean_model + k_sketch_vector" (no schedule) or "k_mean_model" (no sketch
 * requested); "" before the first call.  The string is static;
 * ctx == NULL gives "".  Tests and the benchmark use it to say which kernel a number belongs to.
 */
const char *fda_debug_last_kernel(const fda_ctx *ctx);

/*
 * Number of kernels the context's last fda_local_state call launched (the paper has no
 * counterpart): 2 (the pass and the kernel that adds up its per-block partial sums), or 4 when the
 * sketch pass over index lists also ran its two tail launches on the context's second stream (worker
 * groups that do not divide the SMs, long vectors).  0 before the first call or for ctx == NULL.
 * The benchmark uses it to count the launches of a step.
 */
int fda_debug_last_launches(const fda_ctx *ctx);

/*
 * Local state without a context and without any allocation.  (The paper has no counterpart
 * to this call; it exists for the way some programs have to use the library.)
 *
 * Every other entry point works on an fda_ctx, and creating one calls cudaMalloc.  Some
 * callers cannot do that: a monitoring hook that runs inside a training step while the
 * framework's caching allocator owns all free device memory (a cudaMalloc there fails, or
 * stalls the whole device while it is served), and embedders whose device-memory budget is
 * fixed when the library is loaded.  For them this call computes, for each of the K rows of
 * w, states[k][0] = ||w^(k) - w_t0||^2 and states[k][1] = <xi, w^(k) - w_t0> (the LinearFDA
 * local state, Section 3.2 of the FDA paper), using as scratch a fixed array that is part of
 * the library image: 1 MiB of device memory on every GPU that loads the library, held until
 * the process exits.
 *   device      CUDA device that owns the pointers
 *   w, w_t0, xi as in fda_local_state (any alignment; xi may be NULL)
 *   flags       FDA_STATE_NORM and/or FDA_STATE_LINEAR; slots not asked for are written as 0
 *   states      out, K x 2 floats (not K x state_len)
 * Limits: K <= FDA_NOALLOC_MAX_WORKERS, otherwise FDA_ERR_UNSUPPORTED and nothing is
 * launched.  Neither this call nor anything it uses calls cudaMalloc, cudaFree or an
 * allocating library routine.  The first call on a device looks up the device address of the
 * scratch array (cudaGetSymbolAddress); make that first call before starting any stream
 * capture, and make it at start-up: with CUDA's lazy module loading the library's kernels and
 * the scratch array itself are placed in device memory when they are first touched, i.e. by
 * that first call, which therefore still needs a little free device memory - later calls need
 * none.  All calls on a device share the one scratch array: two calls whose kernels
 * overlap on the GPU (different streams, or different host threads) race on it and give
 * wrong sums, so serialise them.  Nothing in the array has to be cleared between calls:
 * every slot a call reads is first written by that call.
 * Errors: INVALID_ARG (NULL w, w_t0 or states, K < 1, d < 1, row_stride < d, unknown flag,
 * FDA_STATE_SKETCH, device out of range), UNSUPPORTED (K too large), CUDA.
 */
#define FDA_NOALLOC_MAX_WORKERS 64
fda_status fda_local_state_linear_noalloc(int device, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FDA_H_ */
