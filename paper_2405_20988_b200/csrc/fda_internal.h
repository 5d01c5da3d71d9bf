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
// (fda_sched.cu).  Entries address rows of the drift tile ut[index][4 workers]: bits 0..12 row,
// bit 15 set when the sign is -1.  Index r of a tile lives in row r ^ ((r >> 3) & 3).
constexpr int kListWorkers = 4;        // workers per group: one 16-byte row of the drift tile
constexpr int kListSlots = 32;         // lists walked side by side by one warp (lane = list)
constexpr int kListOct = 8;            // lanes per pass of a 128-bit shared-memory load = 16-byte bank groups
constexpr int kListMaxLen = 64;        // longest list (longer cells are cut into pieces)
constexpr int kListPadRows = 8;        // zero rows behind the tile, one per bank group
constexpr int kListBatch = 1024;       // indices a producer step covers; tiles are multiples of it
constexpr int kListMaxTile = 7168;     // rows + pad rows must fit 13 bits
constexpr int kListMinTilesPerBlock = 1;
constexpr int kListSmemHead = 1088;    // counters and the producer warps' fp64 sums in front of the item tables

// byte offsets inside the schedule record of a tile with `items` items
inline __host__ __device__ size_t fda_sched_cells_off(uint32_t items) { return ((size_t)16 + 8 * (size_t)items + 63) / 64 * 64; }
inline __host__ __device__ size_t fda_sched_entries_off(uint32_t items)
{
    return (fda_sched_cells_off(items) + (size_t)items * kListSlots * 2 + 255) / 256 * 256;
}
// shared memory of the sketch kernel: one item-table buffer; everything for a tile of T indices
inline __host__ __device__ uint32_t fda_list_row(uint32_t r) { return r ^ ((r >> 3) & 3u); }
inline int fda_list_table_bytes(int ni_max) { return (16 + 8 * ni_max + 15) / 16 * 16; }
inline size_t fda_list_smem_bytes(int l, int m, int T, int ni_max)
{
    return kListSmemHead + 2 * (size_t)fda_list_table_bytes(ni_max) + (size_t)l * m * kListWorkers * 4 +
           2 * (size_t)(T + kListPadRows) * kListWorkers * 4;
}

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
    uint16_t *tab = nullptr;          // l planes of tab_stride entries; built by the first call that needs it
    int64_t tab_stride = 0;
    float *part_sk = nullptr;         // per-block sketch partials
    size_t part_sk_floats = 0;
    double *part_np = nullptr;        // per-block (norm, projection) partials
    size_t part_np_doubles = 0;
    int max_blocks = 0;
    // list schedule of the sorted-list sketch kernel (null when not built)
    unsigned char *sched = nullptr;   // records of the tiles, 256-byte aligned
    uint64_t *sched_off = nullptr;    // [tiles + 1] byte offsets of the records
    uint64_t sched_bytes = 0;         // size of the schedule
    uint64_t sched_skipped_bytes = 0; // size of a schedule that was not kept (memory limit)
    int64_t sched_limit_bytes = 0;    // caller's cap on the schedule (0: a third of the free memory)
    int sched_T = 0;                  // indices per tile
    int sched_ni_max = 0;             // items a record can have
    int64_t sched_tiles = 0;
    double sched_build_ms = 0.0;      // host time spent building it
    float *mean_model = nullptr;      // d_max floats (average drift), allocated by the first fda_mean_state
    // a second stream for the launches that fill the SMs the main launch of the list kernel leaves idle
    cudaStream_t side_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    double *combine_scratch = nullptr;        // 2 + FDA_MAX_ROWS doubles: S-bar[0..1] and the row norms
    unsigned int *combine_ticket = nullptr;   // blocks of the combine kernel that have finished (0 between launches)
    // staging for fda_round_host (lazy)
    float *stage_w = nullptr, *stage_w_t0 = nullptr, *stage_xi = nullptr, *stage_states = nullptr;
    fda_estimate *stage_est = nullptr;
    int64_t stage_stride = 0;
    uint64_t coeffs_host[6 * FDA_MAX_ROWS] = {0};
    const char *last_ls_kernel = "";   // which kernel served the last fda_local_state / fda_mean_state
    int last_ls_launches = 0;          // kernels the last fda_local_state launched
    std::string err;
};

// ---- launchers (each returns the cudaError_t of its launches) -------------------------
cudaError_t fda_ensure_table(fda_ctx *ctx, cudaStream_t s);   // allocates and fills ctx->tab on first use
cudaError_t fda_launch_read_probe(const fda_ctx *ctx, const float *src, int64_t n, float *sum_out,
                                  cudaStream_t s);
cudaError_t fda_launch_debug_hash(const fda_ctx *ctx, int64_t j0, int64_t n, uint16_t *buckets,
                                  int8_t *signs, cudaStream_t s);
cudaError_t fda_launch_local_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                   int64_t d, const float *w_t0, const float *xi, uint32_t flags,
                                   float *states, cudaStream_t s);
cudaError_t fda_build_list_schedule(fda_ctx *ctx, cudaStream_t s);   // allocates and fills ctx->sched when it fits
cudaError_t fda_launch_local_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s);
cudaError_t fda_launch_mean_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                         int64_t d, const float *w_t0, const float *xi,
                                         uint32_t flags, float *mean_state, cudaStream_t s);
cudaError_t fda_launch_mean_sketch_gather(fda_ctx *ctx, const float *mean_drift, int K, int64_t d, bool have_xi,
                                          uint32_t flags, int np_blocks, float *mean_state, cudaStream_t s);
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
