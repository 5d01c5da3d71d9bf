// Averaged state on the list schedule (fda_mean_state on a context that holds one).
//
// By the linearity of the sketch (Section 3.1, property (a)) the sketch of the mean drift
// u-bar = (1/K) sum_k u^(k) is the average of the K worker sketches, so the cells of S-bar cost l
// updates per index instead of K*l.  This kernel is the sibling of k_local_state_gather
// (fda_local_state_gather.cu) and walks the same schedule (fda_sched.cu): a block serves all K
// workers and a strided set of tiles, producers fill a tile in shared memory, walkers gather from
// it, one block-wide barrier per tile hands the two tile buffers over.  What differs:
//
//   * a row of the tile is one float - the sum over the workers of the drifts of the index - and a
//     cell of the bins one float, so a walker does a 32-bit shared-memory load per entry (the
//     schedule keeps the eight lanes of an octet in different banks mod 8; lanes of different
//     octets may still share a bank) and keeps one sum; everything is divided by K at the end;
//   * the single-column tile leaves most of the shared memory free, and the loads land there
//     instead of in registers: the rows of a quad of indices (the K workers, w_t0, xi) are copied
//     asynchronously, `depth` quads ahead per thread, and the thread that asked for them reads
//     them back when their group has landed (cp.async.wait_group: nothing here can wait for
//     ever).  The bytes in flight then depend neither on registers nor on the number of producer
//     warps.  Elements past d and the rows of a model that is not 16-byte aligned are copied
//     four bytes at a time, with zeros for what lies past the end;
//   * 8 producer and 24 walker warps at 64 registers.
//
// Two callers: the K rows of w (one pass, for few workers), or the single row of averaged drifts
// that k_mean_model has left in device memory (no w_t0; the two scalars then come from that
// kernel's partial sums).  Measured on B200, 5 x 250, K = 8, d = 198M, one pass: 1.50 ms (0.73 of
// the measured copy bandwidth).  On the way: loads landing in registers four rows at a time with
// a four-column tile and 12 + 16 warps 2.15 ms; single-column tile 2.07; landing zone with 8 + 20
// warps 1.73, with 8 + 24 warps 1.67 (6 + 26: 1.86; 12 + 16: 2.01; 4 + 24: 2.12; depth capped at
// 3 / 2: 1.76 / 1.95); without the L2 prefetch of the next tiles' rows that the per-worker kernel
// issues, 1.56; with every shared-memory region on a 128-byte boundary, 1.50.

#include "fda_internal.h"
#include "fda_list_kernel.cuh"

namespace {

using namespace fda_list;

constexpr int kPW = 8;                         // producer warps
constexpr int kWW = 24;                        // walker warps
constexpr int kThreads = (kPW + kWW) * 32;
constexpr int kBatch = kPW * 32 * 4;           // a batch is four consecutive indices per producer thread
constexpr uint32_t kRowPitch = kPW * 32u * 16u;   // one row of a landing-zone slot: 16 bytes per producer thread
constexpr int kMaxDepth = 8;

struct MeanParams {
    ListParams q;                    // rows, schedule, partial-sum buffers; q.K = rows that are read
    int base_zero;                   // the rows are drifts already (no w_t0 to subtract)
    int sketch_only;                 // leave part_np alone
    int depth;                       // quads a producer thread keeps in flight (1 .. kMaxDepth)
};

// 16 bytes from global memory straight into shared memory (no register in between), in groups
// that the issuing thread waits for by age.
__device__ __forceinline__ void cp_async16(uint32_t dst, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// four bytes (on == false: four zero bytes, src is not read)
__device__ __forceinline__ void cp_async4(uint32_t dst, const float *src, bool on)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(on ? 4 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// returns when at most n (0..7) of the thread's groups are still in flight
__device__ __forceinline__ void cp_async_wait_upto(int n)
{
    switch (n) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
    }
}
__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
// One entry: a 32-bit load of the row, the entry's sign flips the top bit.
__device__ __forceinline__ void gather1(uint32_t e, uint32_t base, float &a)
{
    float u;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(u) : "r"(base + ((e & 0x1fffu) << 2)));
    a += __uint_as_float(__float_as_uint(u) ^ ((e & 0x8000u) << 16));
}

// Shared-memory offsets: every region starts on a 128-byte boundary (the 16-byte stores and the
// asynchronous copies need 16; with the landing zone 48 bytes off a 128-byte boundary the pass ran
// 8 % slower).
__host__ __device__ inline uint32_t align128(uint32_t b) { return (b + 127u) & ~127u; }
__host__ __device__ inline uint32_t mean_bins_off(int tab_bytes) { return align128(kListSmemHead + 2u * (uint32_t)tab_bytes); }
__host__ __device__ inline uint32_t mean_ut_off(int lm, int tab_bytes) { return align128(mean_bins_off(tab_bytes) + (uint32_t)lm * 4u); }
__host__ __device__ inline uint32_t mean_ut_bytes(int T) { return align128((uint32_t)(T + kListPadRows) * 4u); }
// bytes in front of the landing zone: counters and sums, two item tables, bins, two tile buffers
inline size_t mean_smem_fixed(int l, int m, int T, int tab_bytes)
{
    return (size_t)mean_ut_off(l * m, tab_bytes) + 2 * (size_t)mean_ut_bytes(T);
}

// Shared-memory plan (bytes from the start of dynamic shared memory):
//   [0, 8)      item counters of the two tile buffers
//   [64, 192)   sums[producer warp][2] (fp64): sum_k ||u_k||^2 and <xi, sum_k u_k> over the tiles so far
//   [1088, ..)  two item tables (tab_bytes each): the head of a tile's schedule record
//   then        bins[l*m]
//   then        ut[2][T + 8]   (summed drifts; eight zero rows behind each)
//   then        the landing zone: depth slots of R rows of kRowPitch bytes
// (each region on a 128-byte boundary)
// AHEAD: entry chunks (four steps each) a walker loads before it walks them (five for sketches of
// seven or more rows, whose items are short; else eight - as in k_local_state_gather).
template <bool LINEAR, int AHEAD>
__global__ void __launch_bounds__(kThreads, 1) k_mean_state_gather(const MeanParams mp)
{
    const ListParams &p = mp.q;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = (int)blockIdx.x;
    const int T = p.T, lm = p.l * p.m;

    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    int *ctr = reinterpret_cast<int *>(smem_raw);
    double *sums = reinterpret_cast<double *>(smem_raw + 64);
    const uint32_t tab_off = kListSmemHead;
    const uint32_t bins_off = mean_bins_off(p.tab_bytes);
    const uint32_t ut_off = mean_ut_off(lm, p.tab_bytes);
    const uint32_t ut_bytes = mean_ut_bytes(T);
    const uint32_t lz_off = ut_off + 2u * ut_bytes;
    float *bins = reinterpret_cast<float *>(smem_raw + bins_off);

    for (int t = tid; t < lm; t += kThreads) bins[t] = 0.f;
    if (tid < 2 * kListPadRows)
        reinterpret_cast<float *>(smem_raw + ut_off + (size_t)(tid / kListPadRows) * ut_bytes)[T + tid % kListPadRows] = 0.f;
    if (tid < 2) ctr[tid] = 0;
    if (tid < kPW * 2) sums[tid] = 0.0;
    __syncthreads();

    const int64_t n_tiles = p.tiles > c ? (p.tiles - c + p.cpg - 1) / p.cpg : 0;

    if (warp < kPW) {
        // =============================== producers ===============================
        const int pt = tid;                                   // quad of indices inside a batch
        const bool vec_in = p.vec != 0;
        float nf = 0.f, pf = 0.f;
        // head of the schedule record of the tile being stored (the walkers' item table) and the
        // record offsets of the next tile, loaded one and two tiles ahead of their use
        uint4 tabv = make_uint4(0u, 0u, 0u, 0u);
        unsigned long long off0 = load_u64(p.sched_off + c), off1 = load_u64(p.sched_off + c + 1);
        if (pt * 16 < p.tab_bytes) tabv = load_u4(p.sched + off0 + pt * 16);
        if (n_tiles > 1) { off0 = load_u64(p.sched_off + c + p.cpg); off1 = load_u64(p.sched_off + c + p.cpg + 1); }

        // Slot s, row r of thread pt: lz + (s * R + r) * kRowPitch.
        const int D = mp.depth;
        const int R = p.K + (mp.base_zero ? 0 : 1) + (LINEAR ? 1 : 0);
        const uint32_t lz = smem_base + lz_off + (uint32_t)pt * 16u;
        const int64_t quads = n_tiles * p.nb;                 // this thread's quads
        int64_t s_i = 0;                                      // next quad to ask for
        int b_i = 0;
        int64_t j_i = (int64_t)c * T + 4 * pt;
        const int64_t wrap = (int64_t)(p.cpg - 1) * T;        // from the end of a tile to this block's next one
        // the slow copy: what lies past d becomes zero
        auto copy_ragged = [&](uint32_t dst, const float *row, int64_t j) {
            const int64_t left = p.d - j;
#pragma unroll
            for (int e = 0; e < 4; ++e) cp_async4(dst + 4u * e, e < left ? row + j + e : row, e < left);
        };
        auto issue = [&](int slot) {
            if (s_i < quads) {
                const uint32_t dst = lz + (uint32_t)(slot * R) * kRowPitch;
                if (vec_in && j_i + 4 <= p.d) {
                    const float *q = p.w + j_i;
                    for (int k = 0; k < p.K; ++k) cp_async16(dst + (uint32_t)k * kRowPitch, q + (int64_t)k * p.row_stride);
                    int r = p.K;
                    if (!mp.base_zero) { cp_async16(dst + (uint32_t)r * kRowPitch, p.w_t0 + j_i); ++r; }
                    if (LINEAR) cp_async16(dst + (uint32_t)r * kRowPitch, p.xi + j_i);
                } else {
                    for (int k = 0; k < p.K; ++k) copy_ragged(dst + (uint32_t)k * kRowPitch, p.w + (int64_t)k * p.row_stride, j_i);
                    int r = p.K;
                    if (!mp.base_zero) { copy_ragged(dst + (uint32_t)r * kRowPitch, p.w_t0, j_i); ++r; }
                    if (LINEAR) copy_ragged(dst + (uint32_t)r * kRowPitch, p.xi, j_i);
                }
                ++s_i;
                j_i += kBatch;
                if (++b_i == p.nb) { b_i = 0; j_i += wrap; }
            }
            cp_async_commit();                                 // (an empty group past the end keeps the count)
        };
        for (int s = 0; s < D; ++s) issue(s);
        int slot = 0;
        for (int64_t n = 0; n < n_tiles; ++n) {
            const int buf = (int)(n & 1);
            for (int b = 0; b < p.nb; ++b) {
                cp_async_wait_upto(D - 1);                     // the oldest group has landed
                const uint32_t src = lz + (uint32_t)(slot * R) * kRowPitch;
                int r = p.K;
                float4 w0 = make_float4(0.f, 0.f, 0.f, 0.f), a = make_float4(0.f, 0.f, 0.f, 0.f);
                if (!mp.base_zero) { w0 = lds128(src + (uint32_t)r * kRowPitch); ++r; }
#pragma unroll 4
                for (int k = 0; k < p.K; ++k) {
                    const float4 v = lds128(src + (uint32_t)k * kRowPitch);
                    const float ux = v.x - w0.x, uy = v.y - w0.y, uz = v.z - w0.z, uw = v.w - w0.w;
                    nf = fmaf(ux, ux, nf); nf = fmaf(uy, uy, nf);
                    nf = fmaf(uz, uz, nf); nf = fmaf(uw, uw, nf);
                    a.x += ux; a.y += uy; a.z += uz; a.w += uw;
                }
                if (LINEAR) {
                    const float4 x = lds128(src + (uint32_t)r * kRowPitch);
                    pf = fmaf(x.x, a.x, pf); pf = fmaf(x.y, a.y, pf);
                    pf = fmaf(x.z, a.z, pf); pf = fmaf(x.w, a.w, pf);
                }
                // rows 4*pt .. 4*pt+3 of the batch; row r is stored at r ^ ((r >> 3) & 3) (the
                // schedule's entries hold that row): one 16-byte store of the quad, its floats permuted
                const uint32_t r0 = (uint32_t)(b * kBatch + 4 * pt);
                const int sw = (int)((r0 >> 3) & 3u);
                store_row(smem_base + ut_off + (uint32_t)buf * ut_bytes + r0 * 4u,
                          comp(a, 0 ^ sw), comp(a, 1 ^ sw), comp(a, 2 ^ sw), comp(a, 3 ^ sw));
                issue(slot);                                   // the slot is free again
                slot = slot + 1 == D ? 0 : slot + 1;
            }
            // ---- the tile is stored: its sums, its item table, its counter, then the hand-over ----
            // (fp32 within the tile: a thread's few indices, then the warp's tree; fp64 across tiles)
            {
                float sa = nf, sb = LINEAR ? pf : 0.f;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    sa += __shfl_xor_sync(0xffffffffu, sa, off);
                    if (LINEAR) sb += __shfl_xor_sync(0xffffffffu, sb, off);
                }
                if (lane == 0) {
                    sums[warp * 2 + 0] += (double)sa;
                    if (LINEAR) sums[warp * 2 + 1] += (double)sb;
                }
                nf = 0.f; pf = 0.f;
            }
            // the table of this tile (loaded a tile ago), the loads of the next one, the offsets of
            // the one after: nothing here waits for memory
            if (pt * 16 < p.tab_bytes)
                *reinterpret_cast<uint4 *>(smem_raw + tab_off + (size_t)buf * p.tab_bytes + pt * 16) = tabv;
            if (pt == 0) ctr[buf] = 0;
            if (n + 1 < n_tiles) {
                const unsigned char *nrec = p.sched + off0;
                if (pt * 16 < p.tab_bytes) tabv = load_u4(nrec + pt * 16);
                for (uint64_t o = (uint64_t)pt * 128u; o < off1 - off0; o += (uint64_t)kPW * 32u * 128u)   // the record into L2 ahead of its walk
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(nrec + o));
            }
            if (n + 2 < n_tiles) {
                const int64_t t2 = c + (n + 2) * p.cpg;
                off0 = load_u64(p.sched_off + t2);
                off1 = load_u64(p.sched_off + t2 + 1);
            }
            block_barrier<kThreads>();
        }
        cp_async_wait_upto(0);
    } else {
        // =============================== walkers ===============================
        for (int64_t n = 0; n < n_tiles; ++n) {
            block_barrier<kThreads>();                                   // tile n is stored, tile n - 1 is walked
            const int buf = (int)(n & 1);
            const unsigned char *rec = p.sched + p.sched_off[c + n * p.cpg];
            const uint32_t *tab = reinterpret_cast<const uint32_t *>(smem_raw + tab_off + (size_t)buf * p.tab_bytes);
            const int n_items = (int)tab[0];
            const uint16_t *cells = reinterpret_cast<const uint16_t *>(rec + fda_sched_cells_off(n_items));
            const unsigned char *ent0 = rec + fda_sched_entries_off(n_items);
            const uint32_t base = smem_base + ut_off + (uint32_t)buf * ut_bytes;
            for (;;) {
                int it = 0;
                if (lane == 0) it = atomicAdd(&ctr[buf], 1);
                it = __shfl_sync(0xffffffffu, it, 0);
                if (it >= n_items) break;
                const uint32_t d0 = tab[4 + 2 * it], chunk0 = tab[5 + 2 * it];
                const int steps = (int)(d0 & 0xffffu);
                const uint32_t cell = cells[(size_t)(d0 >> 16) * kListSlots + lane];
                const uint2 *ent = reinterpret_cast<const uint2 *>(ent0 + (size_t)chunk0 * 256) + lane;
                const int nch = (steps + 3) >> 2;
                float a = 0.f;
                // all entry loads of (up to) AHEAD chunks first, then the walk
                for (int c0 = 0; c0 < nch; c0 += AHEAD) {
                    uint2 ch[AHEAD];
#pragma unroll
                    for (int q = 0; q < AHEAD; ++q)
                        if (c0 + q < nch) ch[q] = __ldg(ent + (size_t)(c0 + q) * kListSlots);
#pragma unroll
                    for (int q = 0; q < AHEAD; ++q) {
                        const int left = steps - 4 * (c0 + q);
                        if (left >= 4) {
                            gather1(ch[q].x & 0xffffu, base, a);
                            gather1(ch[q].x >> 16, base, a);
                            gather1(ch[q].y & 0xffffu, base, a);
                            gather1(ch[q].y >> 16, base, a);
                        } else if (left > 0) {
                            gather1(ch[q].x & 0xffffu, base, a);
                            if (left > 1) gather1(ch[q].x >> 16, base, a);
                            if (left > 2) gather1(ch[q].y & 0xffffu, base, a);
                        }
                    }
                }
                if ((cell & 0x7fffu) < (uint32_t)lm) {
                    float *b = bins + (cell & 0x7fffu);
                    if (cell & 0x8000u) atomicAdd(b, a);                // a cell with several lists
                    else *b += a;
                }
            }
        }
    }
    block_barrier<kThreads>();                                           // the last tile is walked

    // ---- flush: bins -> this block's partial sketch; the producer warps' sums, in warp order ----
    {
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)lm;
        for (int t = tid; t < lm; t += kThreads) out[t] = bins[t];
    }
    if (tid < 2 && !mp.sketch_only) {
        double t = 0.0;
        for (int q = 0; q < kPW; ++q) t += sums[q * 2 + tid];
        p.part_np[(size_t)blockIdx.x * 2 + tid] = t;
    }
}

// Averaged state: mean_state[e] = (sum over the blocks of the partials) / divisor, in fp64 and in a
// fixed order (block after block, eight loads in flight).  The two scalars are summed from
// part_np[b * 2 + e], b < np_blocks - this kernel's own partials, or those of the pass that
// averaged the drifts - and divided by K.
__global__ void k_finalize_mean_gather(const float *__restrict__ part_sk, const double *__restrict__ part_np,
                                       int blocks, int np_blocks, int lm, int K, uint32_t flags, bool have_xi,
                                       double cell_div, float *__restrict__ mean_state)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && warp < 2) {          // the scalars: lanes stride the partials, fixed shuffle tree
        const int e = warp;
        const bool on = (e == 0) ? (flags & FDA_STATE_NORM) != 0 : ((flags & FDA_STATE_LINEAR) != 0 && have_xi);
        double acc = 0.0;
        if (on)
            for (int b = lane; b < np_blocks; b += 32) acc += part_np[(size_t)b * 2 + e];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) mean_state[e] = (float)(acc / (double)K);
    }
    const int cell = blockIdx.x * blockDim.x + threadIdx.x;
    if (cell >= lm) return;
    double acc = 0.0;
    if (flags & FDA_STATE_SKETCH) {
        const float *src = part_sk + cell;
        int b = 0;
        for (; b + 8 <= blocks; b += 8) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = src[(size_t)(b + u) * lm];
#pragma unroll
            for (int u = 0; u < 8; ++u) acc += (double)v[u];
        }
        for (; b < blocks; ++b) acc += (double)src[(size_t)b * lm];
    }
    mean_state[2 + cell] = (float)(acc / cell_div);
}

// rows == K: the averaged state of the K rows of w in one pass.  rows == 1 and base_zero: w is the
// row of averaged drifts; the cells come from it, the two scalars from np_blocks partial pairs that
// the averaging pass left at the start of ctx->part_np.
cudaError_t launch_mean(fda_ctx *ctx, const float *w, int64_t row_stride, int rows, bool base_zero, int K, int64_t d,
                        const float *w_t0, const float *xi, bool have_xi, uint32_t flags, int np_blocks,
                        float *mean_state, cudaStream_t s)
{
    if (!(flags & FDA_STATE_SKETCH) || ctx->l == 0 || !ctx->sched) return cudaErrorNotSupported;
    const float *xi_used = (!base_zero && (flags & FDA_STATE_LINEAR)) ? xi : nullptr;

    MeanParams mp{};
    ListParams &p = mp.q;
    p.w = w; p.w_t0 = w_t0; p.xi = xi_used; p.row_stride = row_stride;
    p.K = rows; p.d = d; p.have_xi = xi_used != nullptr;
    mp.base_zero = base_zero;
    mp.sketch_only = base_zero;
    p.vec = ((((uintptr_t)w | (uintptr_t)(base_zero ? w : w_t0) | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) &&
            (row_stride % 4 == 0);
    p.l = ctx->l; p.m = ctx->m;
    p.T = ctx->sched_T;
    p.sched = ctx->sched; p.sched_off = ctx->sched_off;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np;
    p.tiles = (d + p.T - 1) / p.T;
    p.tab_bytes = fda_list_table_bytes(ctx->sched_ni_max);
    p.groups = 1;
    int64_t cpg = ctx->n_sm;
    if (cpg > p.tiles) cpg = p.tiles;
    p.cpg = (int)cpg;
    const int blocks = p.cpg;
    if ((size_t)blocks * ctx->lm > ctx->part_sk_floats || blocks > ctx->max_blocks ||
        (size_t)blocks * 2 > ctx->part_np_doubles)
        return cudaErrorNotSupported;
    if (p.T % kBatch != 0 || kPW * 32 * 16 < p.tab_bytes) return cudaErrorNotSupported;
    p.nb = p.T / kBatch;
    // what the single-column tile leaves free becomes the producers' landing zone
    const size_t fixed = mean_smem_fixed(p.l, p.m, p.T, p.tab_bytes);
    const size_t per_quad = (size_t)kRowPitch * (size_t)(rows + (base_zero ? 0 : 1) + (xi_used ? 1 : 0));
    const size_t depth = (size_t)ctx->smem_optin > fixed ? ((size_t)ctx->smem_optin - fixed) / per_quad : 0;
    // too many rows to keep three quads per thread in flight: the pass would wait for its loads
    if (depth < (size_t)(base_zero ? 1 : 3)) return cudaErrorNotSupported;
    mp.depth = (int)(depth < (size_t)kMaxDepth ? depth : (size_t)kMaxDepth);
    const size_t smem = fixed + (size_t)mp.depth * per_quad;

    auto kern = ctx->l >= 7 ? (xi_used ? k_mean_state_gather<true, 5> : k_mean_state_gather<false, 5>)
                            : (xi_used ? k_mean_state_gather<true, kChunksAhead> : k_mean_state_gather<false, kChunksAhead>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, kThreads, smem, s>>>(mp);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int fblocks = ((ctx->lm > 64 ? ctx->lm : 64) + 127) / 128;      // at least two warps for the scalars
    k_finalize_mean_gather<<<fblocks, 128, 0, s>>>(ctx->part_sk, ctx->part_np, blocks, base_zero ? np_blocks : blocks,
                                                    ctx->lm, K, flags, have_xi, base_zero ? 1.0 : (double)K, mean_state);
    return cudaGetLastError();
}

}  // namespace

// The averaged state S-bar of fda_mean_state in one pass over the K rows.  Returns
// cudaErrorNotSupported when the request does not fit this path (the caller then uses the other
// kernels); any other value is the result of the launches.
cudaError_t fda_launch_mean_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                         int64_t d, const float *w_t0, const float *xi,
                                         uint32_t flags, float *mean_state, cudaStream_t s)
{
    const bool have_xi = (flags & FDA_STATE_LINEAR) && xi;
    return launch_mean(ctx, w, row_stride, K, false, K, d, w_t0, xi, have_xi, flags, 0, mean_state, s);
}

// The cells of S-bar from the vector of averaged drifts (d floats, 16-byte aligned), the scalars
// from the np_blocks partial pairs at the start of ctx->part_np; same return convention.
cudaError_t fda_launch_mean_sketch_gather(fda_ctx *ctx, const float *mean_drift, int K, int64_t d, bool have_xi,
                                          uint32_t flags, int np_blocks, float *mean_state, cudaStream_t s)
{
    return launch_mean(ctx, mean_drift, (d + 3) / 4 * 4, 1, true, K, d, nullptr, nullptr, have_xi, flags, np_blocks,
                       mean_state, s);
}
