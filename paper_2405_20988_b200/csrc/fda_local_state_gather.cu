// Sketch pass over sorted per-cell lists (the main path of fda_local_state with a sketch).
//
// What the pass computes is stated in fda_local_state.cu (Section 3: drift and ||u||^2;
// Section 3.1: sk(u); Section 3.2: <xi,u>).  This file turns the scatter
// sk[i][h_i(j)] += s_i(j) u[j] into a gather: the bucket and sign of an index never change,
// so the context holds, for every tile of T indices, the indices of each sketch row sorted by
// cell and laid out as a program for a warp (the schedule of fda_sched.cu).  A lane keeps the
// sum of one cell in registers, walks the cell's list and reads the drifts it needs from a
// tile in shared memory; a cell of the bins is touched once per tile and list instead of once
// per update, with plain loads and stores, because a cell belongs to one list (cells that had
// to be cut into pieces are added atomically).  One update costs one 4-byte shared-memory read.
//
// A block serves a group of 4 workers and a strided set of tiles, with two kinds of warps:
//   producers  8 warps (4 for sketches of 7 or more rows).  A thread owns four consecutive indices
//              of a batch (1024 indices with 8 warps): it loads the four workers' values and w_t0
//              (xi) with 128-bit loads into registers (the landing zone: nothing else is staged),
//              subtracts, adds up ||u||^2 and <xi,u> (fp32 within a tile, fp64 across tiles) and
//              stores the four drifts of an index as one 16-byte row of the tile: ut[index][4].
//              The next batch is asked for as soon as the registers are free.  Measured on B200:
//              what a block streams from memory grows with the number of warps that have loads
//              in flight (4.6 TB/s with 8 warps per SM, 6.5 with 16, 7.0 with 24), not with the
//              loads a warp has in flight; deeper software pipelines here changed nothing, and
//              32-bit loads ran at a quarter of the speed;
//   walkers    20 warps (24).  They take the tile's items (32 lists, one per lane) from a counter,
//              longest first; per step a lane loads one 16-bit entry's row with a 128-bit load
//              (the schedule orders the entries so that the eight lanes of a pass through
//              shared memory hit eight different bank groups) and adds it with the entry's
//              sign; when the item ends the 32 sums are added to the bins.
// The tile is double buffered: while the walkers are on tile n the producers fill the other
// buffer with tile n + 1, and one block-wide barrier per tile hands the buffers over.  Nothing
// in this kernel waits on another block or spins on memory.

#include <algorithm>

#include "fda_internal.h"

namespace {

constexpr int GW = kListWorkers;
constexpr int kChunksAhead = 8;                // entry chunks (four steps each) a walker loads before it walks them
constexpr int kMaxProducerWarps = 16;          // the fp64 sums in shared memory have room for that many

struct ListParams {
    const float *w, *w_t0, *xi;
    int64_t row_stride;
    int K;
    int64_t d;
    int have_xi;
    int vec;                         // 16-byte aligned inputs: the producers load 128 bits at a time
    int l, m;
    int groups, cpg;                 // block = c * groups + g
    int T, nb;                       // indices and batches per tile
    int64_t tiles;                   // tiles that hold indices below d
    int tab_bytes;                   // bytes of one item-table buffer in shared memory
    const unsigned char *sched;
    const uint64_t *sched_off;
    float *part_sk;                  // [block][cell][GW]
    double *part_np;                 // [block][GW][2]
    int base_zero;                   // averaged state only: the rows are drifts already (no w_t0 to subtract)
    int depth;                       // averaged state only: quads a producer thread keeps in flight in its
                                     // shared-memory landing zone (1..8)
    int sketch_only;                 // averaged state only: leave part_np alone
};

template <int THREADS>
__device__ __forceinline__ void block_barrier()
{
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
}

// Loads and stores of the producers as volatile statements: the compiler keeps them in program
// order, so a batch's loads are issued kDepth batches before its values are used.
__device__ __forceinline__ float4 load4_stream(const float *ptr)
{
    float4 v;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ float4 load4_keep(const float *ptr)
{
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ float load1(const float *ptr, bool on)
{
    float v;
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\tmov.b32 %0, 0;\n\t@p ld.global.f32 %0, [%1];\n\t}"
                 : "=f"(v) : "l"(ptr), "r"((int)on));
    return v;
}
// four floats from ptr: one 128-bit load when `vec` (aligned, all four below the end), else the
// `n` valid ones with 32-bit loads and zeros behind them
template <bool STREAM>
__device__ __forceinline__ float4 load_quad(const float *ptr, bool vec, int n)
{
    if (vec) return STREAM ? load4_stream(ptr) : load4_keep(ptr);
    float4 v;
    v.x = load1(ptr, n > 0); v.y = load1(ptr + 1, n > 1); v.z = load1(ptr + 2, n > 2); v.w = load1(ptr + 3, n > 3);
    return v;
}
__device__ __forceinline__ uint4 load_u4(const void *ptr)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ unsigned long long load_u64(const void *ptr)
{
    unsigned long long v;
    asm volatile("ld.global.nc.u64 %0, [%1];" : "=l"(v) : "l"(ptr));
    return v;
}
__device__ __forceinline__ void store_row(uint32_t addr, float x, float y, float z, float w)
{
    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ float comp(const float4 &v, int q) { return q == 0 ? v.x : (q == 1 ? v.y : (q == 2 ? v.z : v.w)); }

// One schedule entry: gather the row (four workers) and add it with the entry's sign.  The
// sums stay packed as fp32 pairs, the sign is a multiplication by (+-1, +-1) (exact).
__device__ __forceinline__ void gather_row(uint32_t row_off, uint32_t sign_one, uint32_t base,
                                           unsigned long long &a01, unsigned long long &a23)
{
    unsigned long long u0, u1, ss;
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(u0), "=l"(u1) : "r"(base + row_off));
    asm("mov.b64 %0, {%1,%1};" : "=l"(ss) : "r"(sign_one));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a01) : "l"(u0), "l"(ss));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a23) : "l"(u1), "l"(ss));
}
// low / high half of a 32-bit word holding two entries (bits 0..12 row, bit 15 sign)
__device__ __forceinline__ void gather_lo(uint32_t w, uint32_t base, unsigned long long &a01, unsigned long long &a23)
{
    gather_row((w & 0x1fffu) << 4, ((w << 16) & 0x80000000u) ^ 0x3f800000u, base, a01, a23);
}
__device__ __forceinline__ void gather_hi(uint32_t w, uint32_t base, unsigned long long &a01, unsigned long long &a23)
{
    gather_row((w >> 12) & 0x1fff0u, (w & 0x80000000u) ^ 0x3f800000u, base, a01, a23);
}

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

// One entry of a single-column tile (the averaged state): a 32-bit load, the sign flips the top bit.
__device__ __forceinline__ void gather1(uint32_t e, uint32_t base, float &a)
{
    float u;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(u) : "r"(base + ((e & 0x1fffu) << 2)));
    a += __uint_as_float(__float_as_uint(u) ^ ((e & 0x8000u) << 16));
}

// Shared-memory plan (bytes from the start of dynamic shared memory):
//   [0, 8)    item counters of the two tile buffers
//   [64, 1088) sums[producer warp][worker][2] (fp64): ||u||^2 and <xi,u> over the tiles so far
//   [1088, ..) two item tables (tab_bytes each): the head of a tile's schedule record
//   then      bins[l*m][4]
//   then      ut[2][T + 8][4]   (drift tiles, index-major; eight zero rows behind each)
// PW producer warps and WW walker warps: the split that is fastest depends on how much walking a
// loaded index pays for (l updates per worker).
// MEAN (the averaged state of fda_mean_state; by linearity, Section 3.1 (a), the sketch of the
// mean drift): one block group serves all K workers, a row of the tile is one float, the sum of all
// workers' drifts of the index, and a cell of the bins one float, so the walk costs l 4-byte reads
// per index instead of K*l; the sums are divided by K at the end.
template <bool LINEAR, bool MEAN, int PW, int WW>
__global__ void __launch_bounds__((PW + WW) * 32, 1) k_local_state_gather(const ListParams p)
{
    constexpr int kProducerWarps = PW;
    constexpr int kThreads = (PW + WW) * 32;
    constexpr int kBatch = PW * 32 * 4;                       // a batch is four consecutive indices per producer thread
    constexpr int kDepth = 1;                                 // batches a producer thread keeps in flight
    static_assert(PW <= (MEAN ? 4 * kMaxProducerWarps : kMaxProducerWarps), "room for the fp64 sums of the producer warps");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = (int)blockIdx.x % p.groups, c = (int)blockIdx.x / p.groups;
    const int T = p.T, lm = p.l * p.m;

    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    int *ctr = reinterpret_cast<int *>(smem_raw);
    double *sums = reinterpret_cast<double *>(smem_raw + 64);
    const uint32_t tab_off = kListSmemHead;
    const uint32_t bins_off = tab_off + 2u * (uint32_t)p.tab_bytes;
    constexpr int COLS = MEAN ? 1 : GW;                       // floats per row of the drift tile and per cell of the bins
    const uint32_t ut_off = bins_off + (uint32_t)lm * 16u;    // (MEAN uses a quarter of the bins and of each tile buffer)
    const uint32_t ut_bytes = (uint32_t)(T + kListPadRows) * 4u * COLS;
    float *bins = reinterpret_cast<float *>(smem_raw + bins_off);

    for (int t = tid; t < lm * COLS; t += kThreads) bins[t] = 0.f;
    for (int t = tid; t < 2 * kListPadRows * COLS; t += kThreads) {
        const int b = t / (kListPadRows * COLS), r = t % (kListPadRows * COLS);
        reinterpret_cast<float *>(smem_raw + ut_off + (size_t)b * ut_bytes)[T * COLS + r] = 0.f;
    }
    if (tid < 2) ctr[tid] = 0;
    if (tid < kMaxProducerWarps * GW * 2) sums[tid] = 0.0;
    __syncthreads();

    const int64_t n_tiles = p.tiles > c ? (p.tiles - c + p.cpg - 1) / p.cpg : 0;

    if (warp < kProducerWarps) {
        // =============================== producers ===============================
        const int pt = tid;                                   // quad of indices inside a batch
        const bool vec_in = p.vec != 0;
        float nf[GW], pf[GW];
#pragma unroll
        for (int k = 0; k < GW; ++k) { nf[k] = 0.f; pf[k] = 0.f; }
        // rows of the group (MEAN: the group is all K workers, g = 0)
        const float *wbase = p.w + (size_t)(g * GW) * (size_t)p.row_stride;

        // The rows of a tile two tiles ahead of the one being stored, into L2 (one bulk prefetch per
        // worker row, w_t0 and xi): the producers' loads then find their data in L2.
        auto prefetch_tile = [&](int64_t n) {
            const int n_rows = MEAN ? p.K : GW;
            if (n >= n_tiles || !vec_in || pt >= n_rows + 2) return;
            const int64_t j = (c + n * p.cpg) * (int64_t)T;
            int64_t cnt = p.d - j;
            if (cnt > T) cnt = T;
            const uint32_t bytes = (uint32_t)(cnt * 4) & ~15u;
            for (int r = pt; r < n_rows + 2; r += kProducerWarps * 32) {
                const float *src = r < n_rows ? (g * GW + r < p.K ? wbase + (int64_t)r * p.row_stride + j : nullptr)
                                              : (r == n_rows ? (MEAN && p.base_zero ? nullptr : p.w_t0 + j) : (LINEAR ? p.xi + j : nullptr));
                if (src && bytes)
                    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
            }
        };
        prefetch_tile(0);
        prefetch_tile(1);
        // head of the schedule record of the tile being stored (the walkers' item table) and the
        // record offsets of the next tile, loaded one and two tiles ahead of their use
        uint4 tabv = make_uint4(0u, 0u, 0u, 0u);
        unsigned long long off0 = load_u64(p.sched_off + c), off1 = load_u64(p.sched_off + c + 1);
        if (pt * 16 < p.tab_bytes) tabv = load_u4(p.sched + off0 + pt * 16);
        if (n_tiles > 1) { off0 = load_u64(p.sched_off + c + p.cpg); off1 = load_u64(p.sched_off + c + p.cpg + 1); }

        // ---- tile n of this block is stored: its sums, its item table, its counter, then the hand-over ----
        auto end_of_tile = [&](int64_t n) {
            const int buf = (int)(n & 1);
            // (fp32 within the tile: a thread's few indices, then the warp's tree; fp64 across tiles)
            if (MEAN) {
                float a = nf[0], bq = LINEAR ? pf[0] : 0.f;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    a += __shfl_xor_sync(0xffffffffu, a, off);
                    if (LINEAR) bq += __shfl_xor_sync(0xffffffffu, bq, off);
                }
                if (lane == 0) {
                    sums[warp * 2 + 0] += (double)a;
                    if (LINEAR) sums[warp * 2 + 1] += (double)bq;
                }
                nf[0] = 0.f; pf[0] = 0.f;
            } else {
#pragma unroll
                for (int k = 0; k < GW; ++k) {
                    float a = nf[k], bq = LINEAR ? pf[k] : 0.f;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) {
                        a += __shfl_xor_sync(0xffffffffu, a, off);
                        if (LINEAR) bq += __shfl_xor_sync(0xffffffffu, bq, off);
                    }
                    if (lane == 0) {
                        sums[(warp * GW + k) * 2 + 0] += (double)a;
                        if (LINEAR) sums[(warp * GW + k) * 2 + 1] += (double)bq;
                    }
                    nf[k] = 0.f; pf[k] = 0.f;
                }
            }
            // the table of this tile (loaded a tile ago), the loads of the next one, the offsets
            // of the one after: nothing here waits for memory
            if (pt * 16 < p.tab_bytes)
                *reinterpret_cast<uint4 *>(smem_raw + tab_off + (size_t)buf * p.tab_bytes + pt * 16) = tabv;
            if (pt == 0) ctr[buf] = 0;
            if (n + 1 < n_tiles) {
                const unsigned char *nrec = p.sched + off0;
                if (pt * 16 < p.tab_bytes) tabv = load_u4(nrec + pt * 16);
                for (uint64_t o = (uint64_t)pt * 128u; o < off1 - off0; o += (uint64_t)kProducerWarps * 32u * 128u)   // the record into L2 ahead of its walk
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(nrec + o));
            }
            if (n + 2 < n_tiles) {
                const int64_t t2 = c + (n + 2) * p.cpg;
                off0 = load_u64(p.sched_off + t2);
                off1 = load_u64(p.sched_off + t2 + 1);
            }
            prefetch_tile(n + 2);
            block_barrier<kThreads>();
        };

        if constexpr (!MEAN) {
            // workers past K alias the group's first row (their sums are computed and never written
            // out), so the loop below needs no per-worker predicate
            int64_t roff[GW];
#pragma unroll
            for (int k = 0; k < GW; ++k) roff[k] = g * GW + k < p.K ? (int64_t)k * p.row_stride : 0;
            float4 wv[kDepth][GW], w0v[kDepth], xv[kDepth];       // four consecutive indices each
            int64_t n_i = 0, n_c = 0;                             // tile being loaded / stored
            int b_i = 0, b_c = 0;                                 // batch inside it
            int64_t j_i = (int64_t)c * T + 4 * pt;                // first index of this thread's next loads
            int64_t end_i = (int64_t)(c + 1) * T;                 // end of the tile they belong to
            const int64_t wrap = (int64_t)(p.cpg - 1) * T;        // from the end of a tile to this block's next one
            auto issue = [&](int slot) {
                if (n_i < n_tiles) {
                    const float *q = wbase + j_i;
                    if (vec_in && end_i <= p.d) {                 // a whole tile of aligned rows: 128-bit loads
#pragma unroll
                        for (int k = 0; k < GW; ++k) wv[slot][k] = load4_stream(q + roff[k]);
                        w0v[slot] = load4_keep(p.w_t0 + j_i);
                        if (LINEAR) xv[slot] = load4_keep(p.xi + j_i);
                    } else {                                      // the last tile of the model, or unaligned rows
                        const int64_t left = p.d - j_i;
                        const int n = left >= 4 ? 4 : (left > 0 ? (int)left : 0);
                        const bool vec = vec_in && n == 4;
#pragma unroll
                        for (int k = 0; k < GW; ++k) wv[slot][k] = load_quad<true>(q + roff[k], vec, n);
                        w0v[slot] = load_quad<false>(p.w_t0 + j_i, vec, n);
                        if (LINEAR) xv[slot] = load_quad<false>(p.xi + j_i, vec, n);
                    }
                    j_i += kBatch;
                    if (++b_i == p.nb) { b_i = 0; ++n_i; j_i += wrap; end_i += wrap + T; }
                }
            };
            auto consume = [&](int slot) {
                const int buf = (int)(n_c & 1);
                // rows 4*pt .. 4*pt+3 of the batch; row r is stored at r ^ ((r >> 3) & 3), so that the
                // eight lanes of a store pass hit eight different bank groups (the schedule's entries
                // hold the swizzled row)
                const uint32_t r0 = (uint32_t)(b_c * kBatch + 4 * pt);
                const uint32_t dst0 = smem_base + ut_off + (uint32_t)buf * ut_bytes + r0 * 16u;
                const uint32_t sw = (r0 >> 3) & 3u;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float w0 = comp(w0v[slot], q);
                    const float u0 = comp(wv[slot][0], q) - w0;
                    const float u1 = comp(wv[slot][1], q) - w0;
                    const float u2 = comp(wv[slot][2], q) - w0;
                    const float u3 = comp(wv[slot][3], q) - w0;
                    nf[0] = fmaf(u0, u0, nf[0]); nf[1] = fmaf(u1, u1, nf[1]);
                    nf[2] = fmaf(u2, u2, nf[2]); nf[3] = fmaf(u3, u3, nf[3]);
                    if (LINEAR) {
                        const float xq = comp(xv[slot], q);
                        pf[0] = fmaf(xq, u0, pf[0]); pf[1] = fmaf(xq, u1, pf[1]);
                        pf[2] = fmaf(xq, u2, pf[2]); pf[3] = fmaf(xq, u3, pf[3]);
                    }
                    store_row(dst0 + (((uint32_t)q ^ sw) << 4), u0, u1, u2, u3);
                }
                if (++b_c == p.nb) {
                    end_of_tile(n_c);
                    b_c = 0;
                    ++n_c;
                }
            };
#pragma unroll
            for (int s = 0; s < kDepth; ++s) issue(s);
            while (n_c < n_tiles) {
#pragma unroll
                for (int s = 0; s < kDepth; ++s) {
                    if (n_c < n_tiles) { consume(s); issue(s); }
                }
            }
        } else {
            // The single-column tile leaves most of the shared memory free, so the loads land there
            // instead of in registers: the rows of a quad of indices (the K workers, w_t0, xi) are
            // copied asynchronously, `depth` quads ahead per thread, and the thread that asked for
            // them reads them back when their group has landed.  The bytes in flight then depend
            // neither on registers nor on the number of producer warps (with the loads in registers,
            // four rows at a time, the same pass took 2.07 instead of 1.73 ms at K = 8, d = 198M).
            // Slot s, row r of thread pt: lz + ((s * R + r) * threads + pt) * 16.  Elements past d and
            // the rows of a model that is not 16-byte aligned are copied four bytes at a time, with
            // zeros for what lies past the end.
            const int D = p.depth;
            const int R = p.K + (p.base_zero ? 0 : 1) + (LINEAR ? 1 : 0);
            constexpr uint32_t kRowPitch = (uint32_t)kProducerWarps * 32u * 16u;
            const uint32_t lz = smem_base + ut_off + 2u * ut_bytes + (uint32_t)pt * 16u;
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
            auto issue_lz = [&](int slot) {
                if (s_i < quads) {
                    const uint32_t dst = lz + (uint32_t)(slot * R) * kRowPitch;
                    if (vec_in && j_i + 4 <= p.d) {
                        const float *q = p.w + j_i;
                        for (int k = 0; k < p.K; ++k) cp_async16(dst + (uint32_t)k * kRowPitch, q + (int64_t)k * p.row_stride);
                        int r = p.K;
                        if (!p.base_zero) { cp_async16(dst + (uint32_t)r * kRowPitch, p.w_t0 + j_i); ++r; }
                        if (LINEAR) cp_async16(dst + (uint32_t)r * kRowPitch, p.xi + j_i);
                    } else {
                        for (int k = 0; k < p.K; ++k) copy_ragged(dst + (uint32_t)k * kRowPitch, p.w + (int64_t)k * p.row_stride, j_i);
                        int r = p.K;
                        if (!p.base_zero) { copy_ragged(dst + (uint32_t)r * kRowPitch, p.w_t0, j_i); ++r; }
                        if (LINEAR) copy_ragged(dst + (uint32_t)r * kRowPitch, p.xi, j_i);
                    }
                    ++s_i;
                    j_i += kBatch;
                    if (++b_i == p.nb) { b_i = 0; j_i += wrap; }
                }
                cp_async_commit();                                 // (an empty group past the end keeps the count)
            };
            for (int s = 0; s < D; ++s) issue_lz(s);
            int slot = 0;
            for (int64_t n = 0; n < n_tiles; ++n) {
                const int buf = (int)(n & 1);
                for (int b = 0; b < p.nb; ++b) {
                    cp_async_wait_upto(D - 1);                     // the oldest group has landed
                    const uint32_t src = lz + (uint32_t)(slot * R) * kRowPitch;
                    int r = p.K;
                    float4 w0 = make_float4(0.f, 0.f, 0.f, 0.f), a = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (!p.base_zero) { w0 = lds128(src + (uint32_t)r * kRowPitch); ++r; }
#pragma unroll 4
                    for (int k = 0; k < p.K; ++k) {
                        const float4 v = lds128(src + (uint32_t)k * kRowPitch);
                        const float ux = v.x - w0.x, uy = v.y - w0.y, uz = v.z - w0.z, uw = v.w - w0.w;
                        nf[0] = fmaf(ux, ux, nf[0]); nf[0] = fmaf(uy, uy, nf[0]);
                        nf[0] = fmaf(uz, uz, nf[0]); nf[0] = fmaf(uw, uw, nf[0]);
                        a.x += ux; a.y += uy; a.z += uz; a.w += uw;
                    }
                    if (LINEAR) {
                        const float4 x = lds128(src + (uint32_t)r * kRowPitch);
                        pf[0] = fmaf(x.x, a.x, pf[0]); pf[0] = fmaf(x.y, a.y, pf[0]);
                        pf[0] = fmaf(x.z, a.z, pf[0]); pf[0] = fmaf(x.w, a.w, pf[0]);
                    }
                    // rows 4*pt .. 4*pt+3 of the batch; row r is stored at r ^ ((r >> 3) & 3): one 16-byte
                    // store of the quad, its floats permuted
                    const uint32_t r0 = (uint32_t)(b * kBatch + 4 * pt);
                    const int sw = (int)((r0 >> 3) & 3u);
                    store_row(smem_base + ut_off + (uint32_t)buf * ut_bytes + r0 * 4u,
                              comp(a, 0 ^ sw), comp(a, 1 ^ sw), comp(a, 2 ^ sw), comp(a, 3 ^ sw));
                    issue_lz(slot);                                // the slot is free again
                    slot = slot + 1 == D ? 0 : slot + 1;
                }
                end_of_tile(n);
            }
            cp_async_wait_upto(0);
        }
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
                if constexpr (MEAN) {
                    // one column: a 32-bit load per entry.  The schedule keeps the eight lanes of an
                    // octet in different banks mod 8; lanes of different octets may still share a bank.
                    float a = 0.f;
                    for (int c0 = 0; c0 < nch; c0 += kChunksAhead) {
                        uint2 ch[kChunksAhead];
#pragma unroll
                        for (int q = 0; q < kChunksAhead; ++q)
                            if (c0 + q < nch) ch[q] = __ldg(ent + (size_t)(c0 + q) * kListSlots);
#pragma unroll
                        for (int q = 0; q < kChunksAhead; ++q) {
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
                        if (cell & 0x8000u) atomicAdd(b, a);            // a cell with several lists
                        else *b += a;
                    }
                } else {
                    unsigned long long a01 = 0ull, a23 = 0ull;
                    // all entry loads of (up to) eight chunks first, then the walk: the entries come
                    // from global memory (L2), one round trip per eight chunks instead of one per chunk
                    for (int c0 = 0; c0 < nch; c0 += kChunksAhead) {
                        uint2 ch[kChunksAhead];
    #pragma unroll
                        for (int q = 0; q < kChunksAhead; ++q)
                            if (c0 + q < nch) ch[q] = __ldg(ent + (size_t)(c0 + q) * kListSlots);
    #pragma unroll
                        for (int q = 0; q < kChunksAhead; ++q) {
                            const int left = steps - 4 * (c0 + q);
                            if (left >= 4) {
                                gather_lo(ch[q].x, base, a01, a23);
                                gather_hi(ch[q].x, base, a01, a23);
                                gather_lo(ch[q].y, base, a01, a23);
                                gather_hi(ch[q].y, base, a01, a23);
                            } else if (left > 0) {
                                gather_lo(ch[q].x, base, a01, a23);
                                if (left > 1) gather_hi(ch[q].x, base, a01, a23);
                                if (left > 2) gather_lo(ch[q].y, base, a01, a23);
                            }
                        }
                    }
                    float4 acc;
                    asm("mov.b64 {%0,%1}, %2;" : "=f"(acc.x), "=f"(acc.y) : "l"(a01));
                    asm("mov.b64 {%0,%1}, %2;" : "=f"(acc.z), "=f"(acc.w) : "l"(a23));
                    if ((cell & 0x7fffu) < (uint32_t)lm) {
                        float *b = bins + (cell & 0x7fffu) * GW;
                        if (cell & 0x8000u) {                           // a cell with several lists
                            atomicAdd(b + 0, acc.x); atomicAdd(b + 1, acc.y);
                            atomicAdd(b + 2, acc.z); atomicAdd(b + 3, acc.w);
                        } else {
                            float4 o = *reinterpret_cast<float4 *>(b);
                            o.x += acc.x; o.y += acc.y; o.z += acc.z; o.w += acc.w;
                            *reinterpret_cast<float4 *>(b) = o;
                        }
                    }
                }
            }
        }
    }
    block_barrier<kThreads>();                                           // the last tile is walked

    // ---- flush: bins -> this block's partial sketch ----
    {
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)lm * COLS;
        for (int t = tid; t < lm * COLS; t += kThreads) out[t] = bins[t];
    }
    // ---- block partial of (||u||^2, <xi,u>) per worker: the producer warps' sums, in warp order ----
    // (MEAN: one pair per block, the sum over all workers)
    if (tid < (MEAN ? 2 : GW * 2) && !(MEAN && p.sketch_only)) {
        double t = 0.0;
        for (int q = 0; q < kProducerWarps; ++q) t += sums[q * (MEAN ? 2 : GW * 2) + tid];
        p.part_np[(size_t)blockIdx.x * GW * 2 + tid] = t;
    }
}

// states[k][.] = sum of the partials of worker k's blocks in fp64, in a fixed order: four
// adjacent lanes share one output, lane s adds the blocks s, s + 4, ... of the worker's group in
// order (eight loads in flight), and the four sums are added as (s0 + s1) + (s2 + s3).
__global__ void k_finalize_gather(const ListParams p, int blocks, uint32_t flags, float *__restrict__ states)
{
    const int lm = p.l * p.m, slen = 2 + lm;
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    const int64_t total = (int64_t)p.groups * slen * GW * 4;
    const int64_t padded = (total + 31) & ~(int64_t)31;                 // whole warps take part in the shuffles
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < padded;
         t += (int64_t)gridDim.x * blockDim.x) {
        const bool valid = t < total;
        const int sub = (int)(t & 3);
        const int64_t o = t >> 2;
        const int kl = (int)(o % GW);
        const int e = (int)((o / GW) % slen);
        const int g = (int)(o / ((int64_t)GW * slen));
        const int k = g * GW + kl;
        const int nb = (blocks - g + p.groups - 1) / p.groups;        // blocks of this group: g, g + groups, ...
        double acc = 0.0;
        if (!valid) {
        } else if (e < 2) {
            const bool on = (e == 0) ? (flags & FDA_STATE_NORM) != 0
                                     : ((flags & FDA_STATE_LINEAR) != 0 && p.have_xi);
            if (on)
                for (int j = sub; j < nb; j += 4) acc += p.part_np[((size_t)(g + j * p.groups) * GW + kl) * 2 + e];
        } else if (sketch) {
            const size_t step = (size_t)lm * GW * p.groups;             // from one block of the group to the next
            const float *src = p.part_sk + (size_t)g * lm * GW + (size_t)(e - 2) * GW + kl + (size_t)sub * step;
            int j = sub;
            for (; j + 28 < nb; j += 32, src += 32 * step) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = src[(size_t)(4 * u) * step];
#pragma unroll
                for (int u = 0; u < 8; ++u) acc += (double)v[u];
            }
            for (; j < nb; j += 4, src += 4 * step) acc += (double)src[0];
        }
        const double pair = acc + __shfl_xor_sync(0xffffffffu, acc, 1);      // lanes 0,1: s0 + s1; lanes 2,3: s2 + s3
        const double other = __shfl_xor_sync(0xffffffffu, pair, 2);
        if (valid && sub == 0 && k < p.K) states[(size_t)k * slen + e] = (float)(pair + other);
    }
}

// Averaged state: mean_state[e] = (sum over the blocks of the partials) / divisor, in fp64 and in a
// fixed order (block after block, eight loads in flight).  The two scalars are summed from np_src[b * np_pitch + e], b < np_blocks - this
// kernel's own partials, or those of the pass that averaged the drifts - and divided by K.
__global__ void k_finalize_gather_mean(const ListParams p, int blocks, uint32_t flags, const double *__restrict__ np_src,
                                       int np_blocks, int np_pitch, double cell_div, float *__restrict__ mean_state)
{
    const int lm = p.l * p.m;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && warp < 2) {          // the scalars: lanes stride the partials, fixed shuffle tree
        const int e = warp;
        const bool on = (e == 0) ? (flags & FDA_STATE_NORM) != 0 : ((flags & FDA_STATE_LINEAR) != 0 && p.have_xi);
        double acc = 0.0;
        if (on)
            for (int b = lane; b < np_blocks; b += 32) acc += np_src[(size_t)b * np_pitch + e];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) mean_state[e] = (float)(acc / (double)p.K);
    }
    const int cell = blockIdx.x * blockDim.x + threadIdx.x;
    if (cell >= lm) return;
    double acc = 0.0;
    if (flags & FDA_STATE_SKETCH) {
        const float *src = p.part_sk + cell;
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

template <bool MEAN, int PW, int WW>
cudaError_t launch_lists(ListParams &p, int blocks, size_t smem, int smem_optin, cudaStream_t s)
{
    if (p.T % (PW * 128) != 0 || PW * 32 * 16 < p.tab_bytes) return cudaErrorNotSupported;
    p.nb = p.T / (PW * 128);
    p.depth = 0;
    if (MEAN) {
        // what the single-column tile leaves free becomes the producers' landing zone
        const size_t used = kListSmemHead + 2 * (size_t)p.tab_bytes + (size_t)p.l * p.m * 16 +
                            2 * (size_t)(p.T + kListPadRows) * 4;
        const size_t per_quad = (size_t)PW * 32 * 16 * (size_t)(p.K + (p.base_zero ? 0 : 1) + (p.have_xi ? 1 : 0));
        const size_t depth = (size_t)smem_optin > used ? ((size_t)smem_optin - used) / per_quad : 0;
        if (depth < 1) return cudaErrorNotSupported;              // too many rows for this route
        p.depth = (int)(depth < 8 ? depth : 8);
        smem = used + (size_t)p.depth * per_quad;
    }
    auto kern = p.have_xi ? k_local_state_gather<true, MEAN, PW, WW> : k_local_state_gather<false, MEAN, PW, WW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, (PW + WW) * 32, smem, s>>>(p);
    return cudaGetLastError();
}

enum ListMode { kPerWorker, kMeanFused, kMeanOfVector };

// kPerWorker: states[K][.] of the K rows of w.  kMeanFused: the averaged state of the K rows in one
// pass.  kMeanOfVector: w is one row that holds the average drift already (w_t0 unused); the cells
// of the averaged state come from it, the two scalars from np_blocks partial pairs that the
// averaging pass left at the start of ctx->part_np, and K only divides those.
cudaError_t launch_list_kernel(fda_ctx *ctx, ListMode mode, const float *w, int64_t row_stride, int K, int64_t d,
                               const float *w_t0, const float *xi, bool have_xi, uint32_t flags, float *out,
                               int np_blocks, cudaStream_t s)
{
    if (!(flags & FDA_STATE_SKETCH) || ctx->l == 0 || !ctx->sched) return cudaErrorNotSupported;
    const float *xi_used = (mode != kMeanOfVector && (flags & FDA_STATE_LINEAR)) ? xi : nullptr;
    const bool mean = mode != kPerWorker;
    const int rows = mode == kMeanOfVector ? 1 : K;

    ListParams p{};
    p.w = w; p.w_t0 = w_t0; p.xi = xi_used; p.row_stride = row_stride;
    p.K = rows; p.d = d; p.have_xi = xi_used != nullptr;
    p.base_zero = mode == kMeanOfVector;
    p.sketch_only = mode == kMeanOfVector;
    p.vec = ((((uintptr_t)w | (uintptr_t)(p.base_zero ? w : w_t0) | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) &&
            (row_stride % 4 == 0);
    p.l = ctx->l; p.m = ctx->m;
    p.T = ctx->sched_T;
    p.sched = ctx->sched; p.sched_off = ctx->sched_off;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np;
    p.tiles = (d + p.T - 1) / p.T;
    p.tab_bytes = fda_list_table_bytes(ctx->sched_ni_max);
    p.groups = mean ? 1 : (K + GW - 1) / GW;
    if (p.groups > ctx->n_sm) return cudaErrorNotSupported;
    int64_t cpg = ctx->n_sm / p.groups;
    if (cpg > p.tiles) cpg = p.tiles;
    // short jobs stay with the other kernels
    if (p.tiles < (int64_t)kListMinTilesPerBlock * cpg) return cudaErrorNotSupported;
    p.cpg = (int)cpg;
    const int blocks = p.groups * p.cpg;
    if ((size_t)blocks * ctx->lm * GW > ctx->part_sk_floats || blocks > ctx->max_blocks ||
        (size_t)blocks * GW * 2 > ctx->part_np_doubles)
        return cudaErrorNotSupported;
    const size_t smem = fda_list_smem_bytes(p.l, p.m, p.T, ctx->sched_ni_max);
    if (smem > (size_t)ctx->smem_optin) return cudaErrorNotSupported;

    cudaError_t e = cudaErrorNotSupported;
    if (mean) {
        // 8 producer + 24 walker warps: the single accumulator of the walk and the landing zone of the
        // loads leave room for 32 warps at 64 registers (K = 8, d = 198M, 5 x 250: 1.67 ms; 1.73 with
        // 8 + 20, 1.86 with 6 + 26, 2.01 with 12 + 16, 2.12 with 4 + 24).
        e = launch_lists<true, 8, 24>(p, blocks, smem, ctx->smem_optin, s);
        if (e != cudaSuccess) return e;
        const int fblocks = ((ctx->lm > 64 ? ctx->lm : 64) + 127) / 128;      // at least two warps for the scalars
        p.K = K;
        p.have_xi = have_xi;
        if (mode == kMeanFused)
            k_finalize_gather_mean<<<fblocks, 128, 0, s>>>(p, blocks, flags, ctx->part_np, blocks, GW * 2, (double)K, out);
        else
            k_finalize_gather_mean<<<fblocks, 128, 0, s>>>(p, blocks, flags, ctx->part_np, np_blocks, 2, 1.0, out);
        return cudaGetLastError();
    }
    // 8 producer + 20 walker warps, or 4 + 24 when a loaded index pays for more walking.  Measured:
    // 7 x 500, K = 60, d = 20M: 3.34 ms with 4 + 24 against 3.71 ms with 8 + 20; 5 x 250, K = 8,
    // d = 198M: 3.49 against 2.49 ms; 5 x 250, K = 30, d = 7M: 0.535 against 0.387 ms.
    if (ctx->l >= 7) e = launch_lists<false, 4, 24>(p, blocks, smem, ctx->smem_optin, s);
    else e = launch_lists<false, 8, 20>(p, blocks, smem, ctx->smem_optin, s);
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)p.groups * (2 + ctx->lm) * GW * 4;
    int fb = (int)((total + 255) / 256);
    if (fb > ctx->n_sm * 8) fb = ctx->n_sm * 8;
    k_finalize_gather<<<fb, 256, 0, s>>>(p, blocks, flags, out);
    return cudaGetLastError();
}

}  // namespace

// Returns cudaErrorNotSupported when the request does not fit this path (the caller then uses
// the other kernels); any other value is the result of the launches.
cudaError_t fda_launch_local_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s)
{
    return launch_list_kernel(ctx, kPerWorker, w, row_stride, K, d, w_t0, xi, false, flags, states, 0, s);
}

// The averaged state S-bar of fda_mean_state on the same kernel, in one pass over the K rows; same
// return convention.
cudaError_t fda_launch_mean_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                         int64_t d, const float *w_t0, const float *xi,
                                         uint32_t flags, float *mean_state, cudaStream_t s)
{
    const bool have_xi = (flags & FDA_STATE_LINEAR) && xi;
    return launch_list_kernel(ctx, kMeanFused, w, row_stride, K, d, w_t0, xi, have_xi, flags, mean_state, 0, s);
}

// The cells of S-bar from the vector of averaged drifts (d floats, 16-byte aligned), the scalars
// from the np_blocks partial pairs at the start of ctx->part_np; same return convention.
cudaError_t fda_launch_mean_sketch_gather(fda_ctx *ctx, const float *mean_drift, int K, int64_t d, bool have_xi,
                                          uint32_t flags, int np_blocks, float *mean_state, cudaStream_t s)
{
    return launch_list_kernel(ctx, kMeanOfVector, mean_drift, (d + 3) / 4 * 4, K, d, nullptr, nullptr, have_xi, flags,
                              mean_state, np_blocks, s);
}
