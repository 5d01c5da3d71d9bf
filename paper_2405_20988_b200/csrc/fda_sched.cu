// Gather schedule of the sorted-list sketch kernel (Section 3.1: sk(u)[i][h_i(j)] += s_i(j) u[j]).
//
// The hash of an index depends on (row, index) only, so the order in which a tile's updates
// are applied can be fixed once, when the context is created.  For every (tile, sketch row)
// this file sorts the tile's indices by cell and lays the per-cell lists out as a program for
// one warp of the sketch kernel:
//
//   * an item is the list of one cell (cells with more than kGatherMaxLen indices are split
//     into several items, flagged so that their sums are added atomically);
//   * items are ordered by length and taken kGatherSlots at a time: a round.  The warp walks
//     the 16 lists of a round side by side, one entry per slot and step, and adds the 16 sums
//     to the bins when the round ends.  A round has as many steps as its longest list (made
//     even); shorter lists are padded with entries that point at zero rows;
//   * inside a round the four slots that share a quarter-warp are ordered so that, step by
//     step, their entries fall into different 32-byte bank groups of the drift tile wherever
//     the lists allow it (row mod 4 distinct): a 128-bit gather then takes one pass through
//     shared memory per quarter-warp.
//
// Record of one (tile, row), `sched_pitch` bytes, 16-bit words unless stated:
//   [0] rounds  [1] 0  [2 .. 2+NR) steps of round r  [2+NR .. 2+2NR) first chunk of round r
//   then, 16-byte aligned, cells[r][16]: cell index i*m + c of slot q (bit 15: add atomically;
//   l*m: unused slot), and from `sched_hdr_bytes` on, chunks of 128 bytes: chunk[slot][4] entries,
//   entry = row of the drift tile (bits 0..12) | sign << 15, steps 4c .. 4c+3 of the round.
#include "fda_hash.cuh"
#include "fda_internal.h"

namespace {

constexpr int kBuildThreads = 256;

struct SchedParams {
    const uint64_t *coeffs;
    int l, m;
    uint64_t magic;
    int T;                 // indices per tile
    int nr_max, hdr_bytes, max_chunks;
    size_t pitch;
    unsigned char *sched;
    uint16_t *used;        // [tile][row] entry chunks of the record
};

// Shared memory of the builder (dynamic): see the carve-up in the kernel.
__global__ void __launch_bounds__(kBuildThreads) k_build_schedule(const SchedParams p)
{
    extern __shared__ __align__(16) unsigned char sm[];
    const int tid = threadIdx.x;
    const int64_t rec = blockIdx.x;
    const int i = (int)(rec % p.l);
    const int64_t tile = rec / p.l;
    const int T = p.T, m = p.m;
    const int ni_max = (m < T ? m : T) + T / kGatherMaxLen;

    int *cnt = reinterpret_cast<int *>(sm);                 // [m]   indices per cell
    int *start = cnt + m;                                   // [m+1] first position of a cell's list
    int *fill = start + m + 1;                              // [m]
    int *ifirst = fill + m;                                 // [m+1] first item of a cell
    int *it_start = ifirst + m + 1;                         // [ni_max]
    int *it_len = it_start + ni_max;                        // [ni_max]
    int *it_cell = it_len + ni_max;                         // [ni_max]
    int *order = it_cell + ni_max;                          // [nr_max*16] item of rank r (-1: none)
    int *cls = order + p.nr_max * kGatherSlots;             // [kGatherMaxLen+2] first rank of a length class
    int *rsteps = cls + kGatherMaxLen + 2;                  // [nr_max]
    int *rchunk = rsteps + p.nr_max;                        // [nr_max+1]
    int *chunk_sum = rchunk + p.nr_max + 1;                 // [kBuildThreads+1] scratch of the scans
    uint32_t *key = reinterpret_cast<uint32_t *>(chunk_sum + kBuildThreads + 1);   // [T] cell<<16 | entry
    uint16_t *sorted = reinterpret_cast<uint16_t *>(key + T);                        // [T] entries by cell

    const uint64_t c[6] = {p.coeffs[6 * i + 0], p.coeffs[6 * i + 1], p.coeffs[6 * i + 2],
                           p.coeffs[6 * i + 3], p.coeffs[6 * i + 4], p.coeffs[6 * i + 5]};
    for (int t = tid; t < m; t += kBuildThreads) { cnt[t] = 0; fill[t] = 0; }
    for (int t = tid; t < p.nr_max * kGatherSlots; t += kBuildThreads) order[t] = -1;
    if (tid < kGatherMaxLen + 2) cls[tid] = 0;
    __syncthreads();

    // ---- hash every index of the tile, count the cells ----
    for (int jl = tid; jl < T; jl += kBuildThreads) {
        const uint32_t j = (uint32_t)(tile * T + jl);       // below 2^31 + T
        const uint32_t b = fda::bucket_of(c, j, (uint32_t)m, p.magic);
        const uint32_t sg = fda::sign_is_negative(c, j) ? 0x8000u : 0u;
        key[jl] = (b << 16) | sg | (uint32_t)jl;
        atomicAdd(&cnt[b], 1);
    }
    __syncthreads();

    // ---- exclusive scans over the cells: list positions and item numbers ----
    const int per = (m + kBuildThreads - 1) / kBuildThreads;
    {
        int s0 = 0, s1 = 0;
        for (int t = tid * per; t < min(m, (tid + 1) * per); ++t) {
            s0 += cnt[t];
            s1 += (cnt[t] + kGatherMaxLen - 1) / kGatherMaxLen;
        }
        chunk_sum[tid] = s0;
        __syncthreads();
        // two scans share one scratch array: do them one after the other
        if (tid == 0) { int a = 0; for (int t = 0; t < kBuildThreads; ++t) { const int v = chunk_sum[t]; chunk_sum[t] = a; a += v; } }
        __syncthreads();
        int a = chunk_sum[tid];
        for (int t = tid * per; t < min(m, (tid + 1) * per); ++t) { start[t] = a; a += cnt[t]; }
        if (tid == kBuildThreads - 1) start[m] = T;
        __syncthreads();
        chunk_sum[tid] = s1;
        __syncthreads();
        if (tid == 0) { int b = 0; for (int t = 0; t < kBuildThreads; ++t) { const int v = chunk_sum[t]; chunk_sum[t] = b; b += v; } chunk_sum[kBuildThreads] = b; }
        __syncthreads();
        int b = chunk_sum[tid];
        for (int t = tid * per; t < min(m, (tid + 1) * per); ++t) { ifirst[t] = b; b += (cnt[t] + kGatherMaxLen - 1) / kGatherMaxLen; }
        if (tid == 0) ifirst[m] = chunk_sum[kBuildThreads];
        __syncthreads();
    }
    const int ni = ifirst[m];
    for (int t = tid; t < m; t += kBuildThreads) fill[t] = 0;
    __syncthreads();

    // ---- scatter the entries to their cells (order inside a cell is fixed by the sort below) ----
    for (int jl = tid; jl < T; jl += kBuildThreads) {
        const uint32_t k = key[jl];
        const int b = (int)(k >> 16);
        const int pos = start[b] + atomicAdd(&fill[b], 1);
        sorted[pos] = (uint16_t)(k & 0xffffu);
    }
    // ---- items: pieces of at most kGatherMaxLen entries ----
    for (int b = tid; b < m; b += kBuildThreads) {
        const int n = cnt[b], pieces = (n + kGatherMaxLen - 1) / kGatherMaxLen;
        for (int q = 0; q < pieces; ++q) {
            const int it = ifirst[b] + q;
            it_start[it] = start[b] + q * kGatherMaxLen;
            it_len[it] = min(kGatherMaxLen, n - q * kGatherMaxLen);
            it_cell[it] = (i * m + b) | (pieces > 1 ? 0x8000 : 0);
        }
    }
    __syncthreads();
    // ---- sort each item by (row mod 4, row): fixes the order and groups the bank groups ----
    // (when a cell is split its entries were dealt to the pieces in arrival order; every piece is
    // sorted by itself, and split cells are added atomically anyway)
    for (int it = tid; it < ni; it += kBuildThreads) {
        uint16_t *e = sorted + it_start[it];
        const int n = it_len[it];
        for (int a = 1; a < n; ++a) {
            const uint16_t v = e[a];
            const uint32_t kv = ((uint32_t)(v & 3u) << 13) | (v & 0x1fffu);
            int b = a - 1;
            while (b >= 0) {
                const uint16_t w = e[b];
                const uint32_t kw = ((uint32_t)(w & 3u) << 13) | (w & 0x1fffu);
                if (kw <= kv) break;
                e[b + 1] = w;
                --b;
            }
            e[b + 1] = v;
        }
        atomicAdd(&cls[it_len[it]], 1);
    }
    __syncthreads();
    // ---- rank the items: longest first, ties by item number ----
    if (tid == 0) {
        int a = 0;
        for (int len = kGatherMaxLen; len >= 1; --len) { const int v = cls[len]; cls[len] = a; a += v; }
    }
    __syncthreads();
    if (tid >= 1 && tid <= kGatherMaxLen) {
        int r = cls[tid];
        for (int it = 0; it < ni; ++it)
            if (it_len[it] == tid) order[r++] = it;
    }
    __syncthreads();
    const int nrounds = (ni + kGatherSlots - 1) / kGatherSlots;
    if (tid == 0) {
        int a = 0;
        for (int r = 0; r < nrounds; ++r) {
            const int steps = (it_len[order[r * kGatherSlots]] + 1) & ~1;
            rsteps[r] = steps;
            rchunk[r] = a;
            a += (steps + 3) / 4;
        }
        rchunk[nrounds] = a;
    }
    __syncthreads();

    // ---- header ----
    unsigned char *recp = p.sched + (size_t)rec * p.pitch;
    uint16_t *hdr = reinterpret_cast<uint16_t *>(recp);
    const int cells_off = fda_sched_cells_off(p.nr_max);
    uint16_t *cells = reinterpret_cast<uint16_t *>(recp + cells_off);
    if (tid == 0) { hdr[0] = (uint16_t)nrounds; hdr[1] = 0; p.used[rec] = (uint16_t)rchunk[nrounds]; }
    for (int r = tid; r < p.nr_max; r += kBuildThreads) {
        hdr[2 + r] = (uint16_t)(r < nrounds ? rsteps[r] : 0);
        hdr[2 + p.nr_max + r] = (uint16_t)(r < nrounds ? rchunk[r] : 0);
    }
    for (int t = tid; t < p.nr_max * kGatherSlots; t += kBuildThreads) {
        const int it = order[t];
        cells[t] = (uint16_t)(it >= 0 ? it_cell[it] : p.l * m);
    }

    // ---- entries: one thread per (round, quarter-warp) orders its four lists step by step ----
    uint16_t *ent = reinterpret_cast<uint16_t *>(recp + p.hdr_bytes);
    for (int rq = tid; rq < nrounds * 4; rq += kBuildThreads) {
        const int r = rq >> 2, qq = rq & 3;
        const int steps = rsteps[r];
        int pos[4][4], left[4][4], remain[4];       // per slot and bank group: next entry, entries left
        for (int s = 0; s < 4; ++s) {
            const int it = order[r * kGatherSlots + qq * 4 + s];
            remain[s] = it >= 0 ? it_len[it] : 0;
            for (int g = 0; g < 4; ++g) { pos[s][g] = 0; left[s][g] = 0; }
            if (it >= 0) {
                const uint16_t *e = sorted + it_start[it];
                for (int a = 0; a < remain[s]; ++a) left[s][e[a] & 3]++;
                int a = it_start[it];
                for (int g = 0; g < 4; ++g) { pos[s][g] = a; a += left[s][g]; }
            }
        }
        for (int t = 0; t < steps; ++t) {
            // Give the four slots different bank groups: of the 24 ways to do so take the one that
            // lets the most lists advance (lists with no step to spare count first), then the one
            // that draws on the fullest queues.  A list that cannot advance waits (a zero row)
            // if it has a step to spare; otherwise it takes its fullest queue and the gather of
            // this step needs a second pass through shared memory.
            unsigned used = 0;
            int choice[4] = {-1, -1, -1, -1};
            {
                int best_score = -1, best_perm = 0;
                for (int perm = 0; perm < 24; ++perm) {
                    // perm -> groups g0..g3, all different
                    int avail[4] = {0, 1, 2, 3}, gsel[4], x = perm;
                    for (int s = 0, n = 4; s < 4; ++s, --n) {
                        const int k = x % n; x /= n;
                        gsel[s] = avail[k];
                        for (int a = k; a + 1 < n; ++a) avail[a] = avail[a + 1];
                    }
                    int score = 0;
                    for (int s = 0; s < 4; ++s) {
                        if (remain[s] == 0 || left[s][gsel[s]] == 0) continue;
                        const bool must = remain[s] >= steps - t;
                        score += (must ? 4096 : 256) + left[s][gsel[s]];
                    }
                    if (score > best_score) { best_score = score; best_perm = perm; }
                }
                int avail[4] = {0, 1, 2, 3}, x = best_perm;
                for (int s = 0, n = 4; s < 4; ++s, --n) {
                    const int k = x % n; x /= n;
                    const int gs = avail[k];
                    for (int a = k; a + 1 < n; ++a) avail[a] = avail[a + 1];
                    if (remain[s] > 0 && left[s][gs] > 0) { choice[s] = gs; used |= 1u << gs; }
                }
                for (int s = 0; s < 4; ++s) {
                    if (choice[s] != -1 || remain[s] == 0 || remain[s] < steps - t) continue;
                    int best = 0;                               // no step to spare: a conflict
                    for (int gq = 1; gq < 4; ++gq)
                        if (left[s][gq] > left[s][best]) best = gq;
                    choice[s] = best;
                }
            }
            for (int s = 0; s < 4; ++s) {
                uint16_t e;
                if (choice[s] >= 0) {
                    const int g = choice[s];
                    e = sorted[pos[s][g]++];
                    left[s][g]--;
                    remain[s]--;
                } else {
                    int g = 0;
                    while (g < 3 && (used & (1u << g))) ++g;       // a zero row in a free bank group
                    used |= 1u << g;
                    e = (uint16_t)(T + g);
                }
                ent[((size_t)(rchunk[r] + (t >> 2)) * kGatherSlots + qq * 4 + s) * 4 + (t & 3)] = e;
            }
        }
    }
}

}  // namespace

// Shared memory the sketch kernel needs beside its ring for a tile of nbox boxes.
static size_t gather_fixed_smem(int l, int m, int nbox, int *nr_max, int *hdr_bytes)
{
    const int T = nbox * kGatherBox;
    const int ni_max = (m < T ? m : T) + T / kGatherMaxLen;
    *nr_max = (ni_max + kGatherSlots - 1) / kGatherSlots;
    *hdr_bytes = (fda_sched_cells_off(*nr_max) + *nr_max * kGatherSlots * 2 + 127) / 128 * 128;
    return kGatherPrefixBytes + 128 + 2 * (size_t)l * *hdr_bytes + ((size_t)l * m + 1) * kGatherWorkers * 4 +
           (size_t)(T + kGatherPadRows) * kGatherWorkers * 4;
}

cudaError_t fda_build_gather_schedule(fda_ctx *ctx, cudaStream_t s)
{
    if (ctx->l == 0 || ctx->lm + 1 >= 0x8000) return cudaSuccess;
    // The largest tile that leaves room for two ring stages.  Measured on B200 at 5 x 250, K = 8,
    // d = 198M: 4.32 / 3.85 / 3.60 / 3.62 ms with tiles of 2560 / 3072 / 3584 / 4096 indices - longer
    // lists (fewer rounds per update) pay more than a deeper ring.
    int nbox = 0, nr_max = 0, hdr_bytes = 0;
    for (int nb = 16; nb >= 6; nb -= 2) {      // an even number of boxes: the kernel stages two at a time
        const size_t fixed = gather_fixed_smem(ctx->l, ctx->m, nb, &nr_max, &hdr_bytes);
        if (fixed + 2 * (size_t)fda_gather_stage_bytes() * 2 <= (size_t)ctx->smem_optin) { nbox = nb; break; }
    }
    // Lists shorter than 8 entries on average do not pay for their rounds: measured at 7 x 500 with
    // tiles of 1536 indices, 8.7 ms against 6.9 ms for the compare-and-swap kernel (K = 60, d = 20M).
    if (nbox == 0 || nbox * kGatherBox < 8 * ctx->m) return cudaSuccess;
    const int T = nbox * kGatherBox;
    const int max_chunks = (kGatherMaxLen + T / kGatherSlots) / 4 + nr_max + 2;
    const size_t pitch = (size_t)hdr_bytes + (size_t)max_chunks * 128;
    const int64_t tiles = (ctx->d_max + T - 1) / T;
    const size_t total = (size_t)tiles * ctx->l * pitch;
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) { cudaGetLastError(); return cudaSuccess; }
    if (total > free_b / 3) return cudaSuccess;            // leave the memory to the models
    if ((int64_t)tiles * ctx->l > 0x7fffffffLL) return cudaSuccess;

    const int ni_max = (ctx->m < T ? ctx->m : T) + T / kGatherMaxLen;
    const size_t bsmem = sizeof(int) * ((size_t)4 * ctx->m + 2 + 3 * (size_t)ni_max + (size_t)nr_max * kGatherSlots +
                                        kGatherMaxLen + 2 + 2 * (size_t)nr_max + 1 + kBuildThreads + 1) +
                         (size_t)T * 6 + 16;
    if (bsmem > (size_t)ctx->smem_optin) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_build_schedule, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bsmem);
    if (e != cudaSuccess) return e;
    unsigned char *buf = nullptr;
    uint16_t *used = nullptr;
    if (cudaMalloc(&buf, total) != cudaSuccess) { cudaGetLastError(); return cudaSuccess; }
    if (cudaMalloc(&used, sizeof(uint16_t) * (size_t)tiles * ctx->l) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(buf);
        return cudaSuccess;
    }
    SchedParams p{};
    p.coeffs = ctx->coeffs_dev; p.l = ctx->l; p.m = ctx->m; p.magic = ~0ull / (uint64_t)ctx->m;
    p.T = T; p.nr_max = nr_max; p.hdr_bytes = hdr_bytes; p.max_chunks = max_chunks; p.pitch = pitch; p.sched = buf; p.used = used;
    k_build_schedule<<<(unsigned)(tiles * ctx->l), kBuildThreads, bsmem, s>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) { cudaFree(buf); cudaFree(used); return e; }
    ctx->sched = buf; ctx->sched_used = used; ctx->sched_pitch = pitch; ctx->sched_nbox = nbox; ctx->sched_nr_max = nr_max;
    ctx->sched_hdr_bytes = hdr_bytes; ctx->sched_max_chunks = max_chunks; ctx->sched_tiles = tiles;
    return cudaSuccess;
}
