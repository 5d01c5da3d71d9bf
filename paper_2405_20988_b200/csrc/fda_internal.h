// Internal declarations shared by the translation units of libfda (not installed).
#ifndef FDA_INTERNAL_H_
#define FDA_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>
#include <string>

#include "../../include/fda.h"

// Hash-table entry: bits 0..14 bucket, bit 15 set when the sign is -1.
#define FDA_TAB_SIGN_BIT 0x8000u

// Geometry of the sorted-list sketch kernel (fda_local_state_gather.cu) and of its schedule
// (fda_sched.cu).  A tile is nbox boxes of kGatherBox indices; entries address rows of the
// transposed drift tile: bits 0..12 row, bit 15 set when the sign is -1.
constexpr int kGatherWorkers = 8;      // workers per group (one 32-byte row of the drift tile)
constexpr int kGatherBox = 256;        // indices per tensor box (rows of 1 KB: whole 128-byte lines)
constexpr int kGatherSlots = 16;       // lists walked side by side by one warp
constexpr int kGatherMaxLen = 32;      // longest list of one slot (longer cells are split)
constexpr int kGatherPrefixBytes = 2304; // shared memory in front of the schedule headers (scalars, fp64 sums)
constexpr int kGatherPadRows = 4;      // zero rows behind the tile, one per 32-byte bank group

// byte offset of the cell ids inside a schedule record with room for nr_max rounds
inline __host__ __device__ int fda_sched_cells_off(int nr_max) { return ((2 + 2 * nr_max) * 2 + 15) / 16 * 16; }
// bytes of one ring stage of the sketch kernel: a [workers][box] tile of w, a box of w_t0, a box of xi
inline int fda_gather_stage_bytes() { return kGatherWorkers * kGatherBox * 4 + 2 * kGatherBox * 4; }

struct fda_ctx {
    int device = 0;
    int n_sm = 0;
    int smem_optin = 0;        // largest dynamic shared memory per block (bytes)
    int l = 0, m = 0, lm = 0;
    int64_t d_max = 0;
    int K_max = 0;
    // sketch geometry (valid when l > 0)
    int columns = 0;           // lane-private columns per cell in the shared-memory bins
    // device scratch
    uint64_t *coeffs_dev = nullptr;   // 6*l
    uint16_t *tab = nullptr;          // l planes of tab_stride entries
    uint32_t *tab32 = nullptr;        // same hash as cell index | sign<<31 (staged sketch kernel)
    int64_t tab_stride = 0;
    int64_t tab32_stride = 0;         // entries per plane of tab32: the indices the staged kernel may be asked for
    float *part_sk = nullptr;         // per-block sketch partials
    size_t part_sk_floats = 0;
    double *part_np = nullptr;        // per-block (norm, projection) partials
    size_t part_np_doubles = 0;
    int max_blocks = 0;
    // gather schedule of the sorted-list sketch kernel (null when not built)
    unsigned char *sched = nullptr;   // [tile][row] records of sched_pitch bytes
    size_t sched_pitch = 0;
    uint16_t *sched_used = nullptr;   // [tile][row] 128-byte entry chunks a record uses
    int sched_nbox = 0;               // boxes of kGatherBox indices per tile
    int sched_nr_max = 0;             // rounds a record has room for
    int sched_hdr_bytes = 0;          // bytes of a record's header (round table + cell ids)
    int sched_max_chunks = 0;         // 128-byte entry chunks a record has room for
    int64_t sched_tiles = 0;
    float *mean_model = nullptr;      // d_max floats (average drift), allocated by the first fda_mean_state
    // tensor maps of the last staged launch (encoding four maps costs several microseconds of
    // host time, which matters for small models); valid while the key below matches
    alignas(64) unsigned char tmap_cache[4][128] = {};
    struct {
        const void *w = nullptr, *w_t0 = nullptr, *xi = nullptr;
        int64_t row_stride = 0, d = 0;
        int K = 0, bx = 0, Kg = 0;
    } tmap_key;
    unsigned int *err_flag = nullptr;  // set by a kernel whose bounded wait ran out
    double *combine_scratch = nullptr;        // 2 + FDA_MAX_ROWS doubles: S-bar[0..1] and the row norms
    unsigned int *combine_ticket = nullptr;   // blocks of the combine kernel that have finished (0 between launches)
    // staging for fda_round_host (lazy)
    float *stage_w = nullptr, *stage_w_t0 = nullptr, *stage_xi = nullptr, *stage_states = nullptr;
    fda_estimate *stage_est = nullptr;
    int64_t stage_stride = 0;
    uint64_t coeffs_host[6 * FDA_MAX_ROWS] = {0};
    const char *last_ls_kernel = "";   // which kernel served the last fda_local_state
    std::string err;
};

// ---- launchers (each returns the cudaError_t of its launches) -------------------------
cudaError_t fda_launch_build_table(const fda_ctx *ctx, cudaStream_t s);
cudaError_t fda_launch_read_probe(const fda_ctx *ctx, const float *src, int64_t n, float *sum_out,
                                  cudaStream_t s);
cudaError_t fda_launch_debug_hash(const fda_ctx *ctx, int64_t j0, int64_t n, uint16_t *buckets,
                                  int8_t *signs, cudaStream_t s);
cudaError_t fda_launch_local_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                   int64_t d, const float *w_t0, const float *xi, uint32_t flags,
                                   float *states, cudaStream_t s);
cudaError_t fda_launch_local_state_staged(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s);
cudaError_t fda_build_gather_schedule(fda_ctx *ctx, cudaStream_t s);   // allocates and fills ctx->sched when it fits
cudaError_t fda_launch_local_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s);
cudaError_t fda_launch_local_state_linear(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s);
cudaError_t fda_launch_mean_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                                  const float *w_t0, const float *xi, uint32_t flags, float *mean_state,
                                  cudaStream_t s);
cudaError_t fda_setup_local_state(fda_ctx *ctx);   // opt-in shared memory, pick geometry
cudaError_t fda_launch_combine(const fda_ctx *ctx, const float *states, int K, int variant,
                               float epsilon, float theta, fda_estimate *est_dev, cudaStream_t s);
cudaError_t fda_launch_average(const fda_ctx *ctx, float *w, int64_t row_stride, int K, int64_t d,
                               float *w_t0, float *xi_out, const fda_estimate *est_dev, uint32_t flags,
                               cudaStream_t s);

#endif
