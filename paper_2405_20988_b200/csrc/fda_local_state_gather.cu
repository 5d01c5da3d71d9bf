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
//
// fda_mean_state_gather.cu holds the sibling of this kernel that computes the averaged state of
// fda_mean_state from the same schedule.

#include <algorithm>

#include "fda_internal.h"
#include "fda_list_kernel.cuh"

namespace {

using namespace fda_list;

// Shared-memory plan (bytes from the start of dynamic shared memory):
//   [0, 8)    item counters of the two tile buffers
//   [64, 1088) sums[producer warp][worker][2] (fp64): ||u||^2 and <xi,u> over the tiles so far
//   [1088, ..) two item tables (tab_bytes each): the head of a tile's schedule record
//   then      bins[l*m][4]
//   then      ut[2][T + 8][4]   (drift tiles, index-major; eight zero rows behind each)
// PW producer warps and WW walker warps: the split that is fastest depends on how much walking a
// loaded index pays for (l updates per worker).
template <bool LINEAR, int PW, int WW>
__global__ void __launch_bounds__((PW + WW) * 32, 1) k_local_state_gather(const ListParams p)
{
    constexpr int kProducerWarps = PW;
    constexpr int kThreads = (PW + WW) * 32;
    constexpr int kBatch = PW * 32 * 4;                       // a batch is four consecutive indices per producer thread
    constexpr int kDepth = 1;                                 // batches a producer thread keeps in flight
    // entry chunks (four steps each) a walker loads before it walks them: seven (items of 5 x 250
    // average 28 steps), or five with the 4 + 24 split, whose items average eleven steps.  Measured:
    // 7 x 500, K = 60, d = 20M: 2.94 ms with 5, 2.98 with 4, 2.96 with 6, 3.01 with 7, 3.06 with 8;
    // 5 x 250, K = 8, d = 198M with 8 + 20 warps: 2.474 ms with 7, 2.481 with 8, 2.51 with 6, 2.52 with 10
    constexpr int kAhead = (WW == 24) ? 5 : 7;
    static_assert(PW <= kMaxProducerWarps, "the fp64 sums have room for kMaxProducerWarps warps");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = (int)blockIdx.x % p.groups, c = (int)blockIdx.x / p.groups;
    const int T = p.T, lm = p.l * p.m;

    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    int *ctr = reinterpret_cast<int *>(smem_raw);
    double *sums = reinterpret_cast<double *>(smem_raw + 64);
    const uint32_t tab_off = kListSmemHead;
    const uint32_t bins_off = tab_off + 2u * (uint32_t)p.tab_bytes;
    const uint32_t ut_off = bins_off + (uint32_t)lm * 16u;
    const uint32_t ut_bytes = (uint32_t)(T + kListPadRows) * 16u;
    float *bins = reinterpret_cast<float *>(smem_raw + bins_off);

    for (int t = tid; t < lm * GW; t += kThreads) bins[t] = 0.f;
    for (int t = tid; t < 2 * kListPadRows * GW; t += kThreads) {
        const int b = t / (kListPadRows * GW), r = t % (kListPadRows * GW);
        reinterpret_cast<float *>(smem_raw + ut_off + (size_t)b * ut_bytes)[T * GW + r] = 0.f;
    }
    if (tid < 2) ctr[tid] = 0;
    if (tid < kProducerWarps * GW * 2) sums[tid] = 0.0;
    __syncthreads();

    const int64_t n_tiles = p.tiles > c ? (p.tiles - c + p.cpg - 1) / p.cpg : 0;

    if (warp < kProducerWarps) {
        // =============================== producers ===============================
        const int pt = tid;                                   // quad of indices inside a batch
        // rows of the group; workers past K alias the group's first row (their sums are computed
        // and never written out), so the loop below needs no per-worker predicate
        const float *wbase = p.w + (size_t)(g * GW) * (size_t)p.row_stride;
        int64_t roff[GW];
#pragma unroll
        for (int k = 0; k < GW; ++k) roff[k] = g * GW + k < p.K ? (int64_t)k * p.row_stride : 0;
        float4 wv[kDepth][GW], w0v[kDepth], xv[kDepth];       // four consecutive indices each
        float nf[GW], pf[GW];
#pragma unroll
        for (int k = 0; k < GW; ++k) { nf[k] = 0.f; pf[k] = 0.f; }
        int64_t n_i = 0, n_c = 0;                             // tile being loaded / stored
        int b_i = 0, b_c = 0;                                 // batch inside it
        int64_t j_i = (int64_t)c * T + 4 * pt;                // first index of this thread's next loads
        int64_t end_i = (int64_t)(c + 1) * T;                 // end of the tile they belong to
        const int64_t wrap = (int64_t)(p.cpg - 1) * T;        // from the end of a tile to this block's next one
        const bool vec_in = p.vec != 0;

        // The rows of a tile two tiles ahead of the one being stored, into L2 (one bulk prefetch per
        // worker row, w_t0 and xi): the producers' loads then find their data in L2.
        auto prefetch_tile = [&](int64_t n) {
            if (n >= n_tiles || !vec_in || pt >= GW + 2) return;
            const int64_t j = (c + n * p.cpg) * (int64_t)T;
            int64_t cnt = p.d - j;
            if (cnt > T) cnt = T;
            const uint32_t bytes = (uint32_t)(cnt * 4) & ~15u;
            const float *src = pt < GW ? (g * GW + pt < p.K ? wbase + (int64_t)pt * p.row_stride + j : nullptr)
                                       : (pt == GW ? p.w_t0 + j : (LINEAR ? p.xi + j : nullptr));
            if (src && bytes)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
        };
        prefetch_tile(0);
        prefetch_tile(1);
        // head of the schedule record of the tile being stored (the walkers' item table) and the
        // record offsets of the next tile, loaded one and two tiles ahead of their use
        uint4 tabv = make_uint4(0u, 0u, 0u, 0u);
        unsigned long long off0 = load_u64(p.sched_off + c), off1 = load_u64(p.sched_off + c + 1);
        if (pt * 16 < p.tab_bytes) tabv = load_u4(p.sched + off0 + pt * 16);
        if (n_tiles > 1) { off0 = load_u64(p.sched_off + c + p.cpg); off1 = load_u64(p.sched_off + c + p.cpg + 1); }
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
                // ---- the tile is stored: its item table, its counter, then the hand-over ----
                // (fp32 within the tile: a thread's few indices, then the warp's tree; fp64 across tiles)
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
                // the table of this tile (loaded a tile ago), the loads of the next one, the offsets
                // of the one after: nothing here waits for memory
                if (pt * 16 < p.tab_bytes)
                    *reinterpret_cast<uint4 *>(smem_raw + tab_off + (size_t)buf * p.tab_bytes + pt * 16) = tabv;
                if (pt == 0) ctr[buf] = 0;
                if (n_c + 1 < n_tiles) {
                    const unsigned char *nrec = p.sched + off0;
                    if (pt * 16 < p.tab_bytes) tabv = load_u4(nrec + pt * 16);
                    for (uint64_t o = (uint64_t)pt * 128u; o < off1 - off0; o += (uint64_t)kProducerWarps * 32u * 128u)   // the record into L2 ahead of its walk
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(nrec + o));
                }
                if (n_c + 2 < n_tiles) {
                    const int64_t t2 = c + (n_c + 2) * p.cpg;
                    off0 = load_u64(p.sched_off + t2);
                    off1 = load_u64(p.sched_off + t2 + 1);
                }
                prefetch_tile(n_c + 2);
                block_barrier<kThreads>();
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
                unsigned long long a01 = 0ull, a23 = 0ull;
                // all entry loads of (up to) kAhead chunks first, then the walk: the entries come
                // from global memory (L2), one round trip per kAhead chunks instead of one per chunk
                for (int c0 = 0; c0 < nch; c0 += kAhead) {
                    uint2 ch[kAhead];
#pragma unroll
                    for (int q = 0; q < kAhead; ++q)
                        if (c0 + q < nch) ch[q] = __ldg(ent + (size_t)(c0 + q) * kListSlots);
#pragma unroll
                    for (int q = 0; q < kAhead; ++q) {
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
    block_barrier<kThreads>();                                           // the last tile is walked

    // ---- flush: bins -> this block's partial sketch ----
    {
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)lm * GW;
        for (int t = tid; t < lm * GW; t += kThreads) out[t] = bins[t];
    }
    // ---- block partial of (||u||^2, <xi,u>) per worker: the producer warps' sums, in warp order ----
    if (tid < GW * 2) {
        double t = 0.0;
        for (int q = 0; q < kProducerWarps; ++q) t += sums[q * GW * 2 + tid];
        p.part_np[(size_t)blockIdx.x * GW * 2 + tid] = t;
    }
}

// The partial sums of a call come from up to three launches of the kernel (the main one and the
// two that fill the SMs it leaves idle, see fda_launch_local_state_gather): launch q served the
// groups g_first .. g_first + groups - 1 with cpg blocks each, block c * groups + (g - g_first)
// writing slot slot_base + that number.
struct ListParts {
    int n;
    int slot_base[3], g_first[3], groups[3], cpg[3];
};

// states[k][.] = sum of the partials of worker k's blocks in fp64, in a fixed order: four
// adjacent lanes share one output, lane s adds the blocks s, s + 4, ... of the worker's group in
// each launch in order (eight loads in flight), and the four sums are added as (s0 + s1) + (s2 + s3).
__global__ void k_finalize_gather(const ListParams p, const ListParts parts, uint32_t flags, float *__restrict__ states)
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
        double acc = 0.0;
        for (int q = 0; q < parts.n; ++q) {
            const int gl = g - parts.g_first[q];
            if (!valid || gl < 0 || gl >= parts.groups[q]) continue;
            const int nb = parts.cpg[q];                                // blocks of this group: gl, gl + groups, ...
            const size_t first = (size_t)(parts.slot_base[q] + gl);
            if (e < 2) {
                const bool on = (e == 0) ? (flags & FDA_STATE_NORM) != 0
                                         : ((flags & FDA_STATE_LINEAR) != 0 && p.have_xi);
                if (on)
                    for (int j = sub; j < nb; j += 4)
                        acc += p.part_np[((first + (size_t)j * parts.groups[q]) * GW + kl) * 2 + e];
            } else if (sketch) {
                const size_t step = (size_t)lm * GW * parts.groups[q];  // from one block of the group to the next
                const float *src = p.part_sk + first * lm * GW + (size_t)(e - 2) * GW + kl + (size_t)sub * step;
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
        }
        const double pair = acc + __shfl_xor_sync(0xffffffffu, acc, 1);      // lanes 0,1: s0 + s1; lanes 2,3: s2 + s3
        const double other = __shfl_xor_sync(0xffffffffu, pair, 2);
        if (valid && sub == 0 && k < p.K) states[(size_t)k * slen + e] = (float)(pair + other);
    }
}

template <int PW, int WW>
cudaError_t launch_lists(ListParams &p, int blocks, size_t smem, int smem_optin, cudaStream_t s)
{
    if (p.T % (PW * 128) != 0 || PW * 32 * 16 < p.tab_bytes) return cudaErrorNotSupported;
    p.nb = p.T / (PW * 128);
    auto kern = p.have_xi ? k_local_state_gather<true, PW, WW> : k_local_state_gather<false, PW, WW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, (PW + WW) * 32, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

// Returns cudaErrorNotSupported when the request does not fit this path (the caller then uses
// the other kernels); any other value is the result of the launches.
cudaError_t fda_launch_local_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s)
{
    if (!(flags & FDA_STATE_SKETCH) || ctx->l == 0 || !ctx->sched) return cudaErrorNotSupported;
    const float *xi_used = (flags & FDA_STATE_LINEAR) ? xi : nullptr;

    ListParams p{};
    p.w = w; p.w_t0 = w_t0; p.xi = xi_used; p.row_stride = row_stride;
    p.K = K; p.d = d; p.have_xi = xi_used != nullptr;
    p.vec = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) && (row_stride % 4 == 0);
    p.l = ctx->l; p.m = ctx->m;
    p.T = ctx->sched_T;
    p.sched = ctx->sched; p.sched_off = ctx->sched_off;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np;
    p.tiles = (d + p.T - 1) / p.T;
    p.tab_bytes = fda_list_table_bytes(ctx->sched_ni_max);
    p.groups = (K + GW - 1) / GW;
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

    // 8 producer + 20 walker warps, or 4 + 24 when a loaded index pays for more walking.  Measured:
    // 7 x 500, K = 60, d = 20M: 3.34 ms with 4 + 24 against 3.71 ms with 8 + 20; 5 x 250, K = 8,
    // d = 198M: 3.49 against 2.49 ms; 5 x 250, K = 30, d = 7M: 0.535 against 0.387 ms.
    auto launch = [&](ListParams &q, int grid, cudaStream_t st) {
        return ctx->l >= 7 ? launch_lists<4, 24>(q, grid, smem, ctx->smem_optin, st)
                           : launch_lists<8, 20>(q, grid, smem, ctx->smem_optin, st);
    };
    ListParts parts{};
    parts.n = 1;
    parts.slot_base[0] = 0; parts.g_first[0] = 0; parts.groups[0] = p.groups; parts.cpg[0] = p.cpg;

    // When the groups do not divide the SMs (K = 60: 15 groups x 9 blocks on 148 SMs) the SMs left
    // over get the last tiles of every group, from the same kernel launched on a second stream with
    // shifted pointers: first one block for each of the first `extra` groups, then the other groups
    // on as many blocks each as fit.  The main launch stops at tile t1; all launches write their own
    // slots of the partial sums.  Taken when the second of those launches still has a block per group
    // and the job is long enough for the gain (tiles / cpg against t1 / cpg tile walks) to show.
    const int extra = ctx->n_sm - blocks;
    const int rest = p.groups - extra;                         // groups of the second tail launch (extra < groups)
    int64_t t1 = p.tiles;
    int cpg_b = 0;
    if (extra > 0 && rest > 0 && extra / rest >= 1 && ctx->side_stream && p.tiles >= 64 * (int64_t)p.cpg) {
        cpg_b = extra / rest;
        // tail walks per block: n_tail + n_tail / cpg_b; main walks per block: (tiles - n_tail) / cpg
        const double per_tail = 1.0 + 1.0 / (double)cpg_b;
        int64_t n_tail = (int64_t)((double)p.tiles / (1.0 + (double)p.cpg * per_tail));
        n_tail = n_tail / cpg_b * cpg_b;
        const int64_t main_walks = (p.tiles - n_tail + p.cpg - 1) / p.cpg;
        const size_t slots = (size_t)blocks + extra + (size_t)rest * cpg_b;
        if (n_tail >= 4 * cpg_b && main_walks + 2 < (p.tiles + p.cpg - 1) / p.cpg &&
            slots * ctx->lm * GW <= ctx->part_sk_floats && slots * GW * 2 <= ctx->part_np_doubles)
            t1 = p.tiles - n_tail;
    }
    cudaError_t e;
    if (t1 < p.tiles) {
        const int64_t shift = t1 * p.T;                        // elements in front of the tail (a multiple of 1024)
        ListParams ta = p;
        ta.w = p.w + shift; ta.w_t0 = p.w_t0 + shift; ta.xi = p.xi ? p.xi + shift : nullptr;
        ta.d = p.d - shift; ta.tiles = p.tiles - t1; ta.sched_off = p.sched_off + t1;
        ListParams tb = ta;
        ta.K = extra * GW; ta.groups = extra; ta.cpg = 1;
        ta.part_sk = p.part_sk + (size_t)blocks * ctx->lm * GW; ta.part_np = p.part_np + (size_t)blocks * GW * 2;
        tb.w = ta.w + (size_t)extra * GW * (size_t)row_stride; tb.K = K - extra * GW; tb.groups = rest; tb.cpg = cpg_b;
        tb.part_sk = ta.part_sk + (size_t)extra * ctx->lm * GW; tb.part_np = ta.part_np + (size_t)extra * GW * 2;
        parts.n = 3;
        parts.slot_base[1] = blocks; parts.g_first[1] = 0; parts.groups[1] = extra; parts.cpg[1] = 1;
        parts.slot_base[2] = blocks + extra; parts.g_first[2] = extra; parts.groups[2] = rest; parts.cpg[2] = cpg_b;
        ListParams main = p;
        main.tiles = t1; main.d = shift;
        e = cudaEventRecord(ctx->ev_fork, s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0);
        if (e == cudaSuccess) e = launch(ta, extra, ctx->side_stream);
        if (e == cudaSuccess) e = launch(tb, rest * cpg_b, ctx->side_stream);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_join, ctx->side_stream);
        if (e == cudaSuccess) e = launch(main, blocks, s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ctx->ev_join, 0);
    } else {
        e = launch(p, blocks, s);
    }
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)p.groups * (2 + ctx->lm) * GW * 4;
    int fb = (int)((total + 255) / 256);
    if (fb > ctx->n_sm * 8) fb = ctx->n_sm * 8;
    k_finalize_gather<<<fb, 256, 0, s>>>(p, parts, flags, states);
    ctx->last_ls_launches = parts.n + 1;
    return cudaGetLastError();
}
