// List schedule of the sketch kernel (Section 3.1: sk(u)[i][h_i(j)] += s_i(j) u[j]).
//
// The hash of an index depends on (row, index) only, so the order in which a tile's updates
// are applied can be fixed once, when the context is created.  For every tile of T indices
// this file sorts the indices of each sketch row by cell and lays the per-cell lists out as a
// program for the warps of k_local_state_gather:
//
//   * a list holds the indices of one cell (a cell with more than kListMaxLen indices is cut
//     into pieces, flagged so that their sums are added atomically);
//   * a warp walks 32 lists side by side, one per lane: an item.  A lane reads the drift of one
//     index and four workers with one 128-bit shared-memory load per step.  Eight lanes share a
//     pass through shared memory, and the pass is conflict free when their eight rows fall into
//     eight different 16-byte bank groups, i.e. when the indices differ mod 8;
//   * so the lists are grouped by eight (an octet): starting from the longest list left, the
//     builder adds the longest lists whose indices keep every residue class mod 8 of the octet
//     at or below the length of the first one (a class with c indices needs c passes whatever
//     the order), counting a list whose cell shares a bank group with a cell already in the
//     octet (a conflict when the sums are flushed) as two entries shorter.  The entries of an octet are then ordered by decomposing the bipartite
//     multigraph (lists x residue classes, one edge per index, made regular with padding edges)
//     into perfect matchings: in every step each lane reads a different residue class, and a
//     lane with nothing left reads a zero row of a class nobody else reads;
//   * octets are ordered by their number of steps and taken four at a time, items are ordered by
//     steps over all sketch rows of the tile (the kernel hands them out longest first).
//
// Record of one tile (byte offsets; all records are 256-byte aligned, their offsets are in a
// table of tiles + 1 64-bit values):
//   [0]  u32 items   [4] u32 bytes of the record   [8] u32 entry chunks   [12] u32 0
//   [16] items x { u16 steps, u16 cell block, u32 first chunk }, longest first
//   then, 64-byte aligned, cell blocks: [32] u16 cell index i*m + c of the lane's list (bit 15:
//   add atomically; l*m: the lane has no list)
//   then, 256-byte aligned, chunks of 256 bytes: [lane][4] u16 entries, steps 4c .. 4c+3 of an
//   item; entry = row of the drift tile (bits 0..12; index r of the tile is stored in row
//   r ^ ((r >> 3) & 3); T + r is the zero row of class r) | sign << 15.
#include <vector>

#include "fda_hash.cuh"
#include "fda_internal.h"

namespace {

constexpr int kBT = 256;                  // threads of a builder block
constexpr int ML = kListMaxLen;
constexpr int NRES = kListOct;            // residue classes = lanes per shared-memory pass
constexpr int kWindow = 64;               // candidates looked at for every place in an octet
#ifndef FDA_SPREAD
#define FDA_SPREAD 8
#endif
constexpr int kMatchBytes = 304;          // shared memory of the thread that orders an octet's entries
constexpr int kSpread = FDA_SPREAD;       // every kSpread-th thread of the block orders the entries of an octet

struct SchedParams {
    const uint64_t *coeffs;
    int l, m;
    uint64_t magic;
    int T;
    int nl_max;            // lists of a (tile, row)
    int no_max;            // octets of a (tile, row)
    int ni_row_max;        // items of a (tile, row)
    uint32_t *rec_items;   // [tile]  written by the counting pass, read by the writing pass
    uint32_t *rec_chunks;  // [tile]
    const uint64_t *rec_off;   // [tile + 1] byte offsets of the records (writing pass)
    unsigned char *sched;
};

struct Carve {
    unsigned char *p;
    template <typename T> __device__ T *take(size_t n)
    {
        p = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(p) + 15) & ~(uintptr_t)15);
        T *r = reinterpret_cast<T *>(p);
        p += n * sizeof(T);
        return r;
    }
};

// shared memory of a builder block (must match the carve-up in the kernel)
size_t build_smem(int l, int m, int T, int nl_max, int no_max, int ni_row_max)
{
    auto a16 = [](size_t b) { return (b + 15) / 16 * 16; };
    size_t s = 0;
    s += a16(sizeof(int) * m) * 3 + a16(sizeof(int) * (m + 1)) * 2;      // cnt, fill, npiece | start, lfirst
    s += a16(sizeof(uint32_t) * T) * 2;                                   // key, bycell
    s += a16(sizeof(uint16_t) * T);                                       // sorted
    s += a16(sizeof(uint16_t) * nl_max) * 4;                              // ls_start, ls_len, ls_cell, order
    s += a16(8 * (size_t)nl_max);                                         // ls_res
    s += a16(sizeof(int) * (ML + 2)) + a16(sizeof(int) * (kBT + 1));      // cls, scan scratch
    s += a16(sizeof(uint16_t) * 8 * no_max) + a16(sizeof(uint16_t) * no_max) * 2;   // oc_list, oc_cost, oc_order
    s += a16(sizeof(uint32_t) * (size_t)l * ni_row_max) * 3;              // it_steps, it_chunk, it_rank
    s += 64;
    return s + 64;
}

// One block per tile.  WRITE = false: count the items and entry chunks of the record;
// WRITE = true: write the record at its offset.
template <bool WRITE>
__global__ void __launch_bounds__(kBT) k_build_schedule(const SchedParams p)
{
    extern __shared__ __align__(16) unsigned char sm[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t tile = blockIdx.x;
    const int T = p.T, m = p.m, NL = p.nl_max, NO = p.no_max;

    Carve cv{sm};
    int *cnt = cv.take<int>(m);
    int *fill = cv.take<int>(m);
    int *npiece = cv.take<int>(m);
    int *start = cv.take<int>(m + 1);
    int *lfirst = cv.take<int>(m + 1);
    uint32_t *key = cv.take<uint32_t>(T);          // by index: cell << 16 | sign << 15 | index
    uint32_t *bycell = cv.take<uint32_t>(T);       // the same words grouped by cell
    uint16_t *sorted = cv.take<uint16_t>(T);       // entries (sign << 15 | index), list after list
    uint16_t *ls_start = cv.take<uint16_t>(NL);
    uint16_t *ls_len = cv.take<uint16_t>(NL);
    uint16_t *ls_cell = cv.take<uint16_t>(NL);
    uint16_t *order = cv.take<uint16_t>(NL);       // lists, longest first
    unsigned char *ls_res = cv.take<unsigned char>(8 * (size_t)NL);   // indices per residue class
    int *cls = cv.take<int>(ML + 2);
    int *scan = cv.take<int>(kBT + 1);
    uint16_t *oc_list = cv.take<uint16_t>(8 * (size_t)NO);
    uint16_t *oc_cost = cv.take<uint16_t>(NO);
    uint16_t *oc_order = cv.take<uint16_t>(NO);    // octets, most steps first
    uint32_t *it_steps = cv.take<uint32_t>((size_t)p.l * p.ni_row_max);
    uint32_t *it_chunk = cv.take<uint32_t>((size_t)p.l * p.ni_row_max);
    uint32_t *it_rank = cv.take<uint32_t>((size_t)p.l * p.ni_row_max);
    int *tot = cv.take<int>(8);                    // [0] items so far, [1] chunks so far, [2] lists, [3] octets

    unsigned char *rec = nullptr;
    uint32_t rec_ni = 0;
    size_t cells_off = 0, ent_off = 0;
    if (WRITE) {
        rec = p.sched + p.rec_off[tile];
        rec_ni = p.rec_items[tile];
        cells_off = fda_sched_cells_off(rec_ni);
        ent_off = fda_sched_entries_off(rec_ni);
    }
    if (tid == 0) { tot[0] = 0; tot[1] = 0; }
    __syncthreads();

    for (int i = 0; i < p.l; ++i) {
        const uint64_t c[6] = {p.coeffs[6 * i + 0], p.coeffs[6 * i + 1], p.coeffs[6 * i + 2],
                               p.coeffs[6 * i + 3], p.coeffs[6 * i + 4], p.coeffs[6 * i + 5]};
        for (int t = tid; t < m; t += kBT) { cnt[t] = 0; fill[t] = 0; }
        if (tid < ML + 2) cls[tid] = 0;
        __syncthreads();

        // ---- hash every index of the tile, count the cells ----
        for (int jl = tid; jl < T; jl += kBT) {
            const uint32_t j = (uint32_t)(tile * T + jl);       // below 2^31 + T
            const uint32_t b = fda::bucket_of(c, j, (uint32_t)m, p.magic);
            const uint32_t sg = fda::sign_is_negative(c, j) ? 0x8000u : 0u;
            key[jl] = (b << 16) | sg | (uint32_t)jl;
            atomicAdd(&cnt[b], 1);
        }
        __syncthreads();

        // ---- exclusive scans over the cells: positions and list numbers ----
        const int per = (m + kBT - 1) / kBT;
        {
            int s0 = 0, s1 = 0;
            for (int t = tid * per; t < min(m, (tid + 1) * per); ++t) {
                const int np = (cnt[t] + ML - 1) / ML;
                npiece[t] = np;
                s0 += cnt[t];
                s1 += np;
            }
            scan[tid] = s0;
            __syncthreads();
            if (tid == 0) { int a = 0; for (int t = 0; t < kBT; ++t) { const int v = scan[t]; scan[t] = a; a += v; } }
            __syncthreads();
            int a = scan[tid];
            for (int t = tid * per; t < min(m, (tid + 1) * per); ++t) { start[t] = a; a += cnt[t]; }
            if (tid == kBT - 1) start[m] = T;
            __syncthreads();
            scan[tid] = s1;
            __syncthreads();
            if (tid == 0) { int b = 0; for (int t = 0; t < kBT; ++t) { const int v = scan[t]; scan[t] = b; b += v; } scan[kBT] = b; }
            __syncthreads();
            int b = scan[tid];
            for (int t = tid * per; t < min(m, (tid + 1) * per); ++t) { lfirst[t] = b; b += npiece[t]; }
            if (tid == 0) { lfirst[m] = scan[kBT]; tot[2] = scan[kBT]; }
            __syncthreads();
        }
        const int nl = tot[2];

        // ---- group by cell (arrival order), then order every cell's run by index ----
        for (int jl = tid; jl < T; jl += kBT) {
            const uint32_t k = key[jl];
            const int b = (int)(k >> 16);
            bycell[start[b] + atomicAdd(&fill[b], 1)] = k;
        }
        __syncthreads();
        for (int pos = tid; pos < T; pos += kBT) {
            const uint32_t k = bycell[pos];
            const int b = (int)(k >> 16);
            const uint32_t idx = k & 0x1fffu;
            int rank = 0;
            for (int q = start[b]; q < start[b + 1]; ++q) rank += ((bycell[q] & 0x1fffu) < idx) ? 1 : 0;
            sorted[start[b] + rank] = (uint16_t)((k & 0x8000u) | fda_list_row(idx));   // the row the index is stored in
        }
        // ---- lists: a cell's run in pieces of nearly equal length ----
        for (int b = tid; b < m; b += kBT) {
            const int n = cnt[b], pieces = npiece[b];
            if (pieces == 0) continue;
            const int base = n / pieces, rem = n % pieces;
            for (int q = 0; q < pieces; ++q) {
                const int it = lfirst[b] + q;
                ls_start[it] = (uint16_t)(start[b] + q * base + min(q, rem));
                ls_len[it] = (uint16_t)(base + (q < rem ? 1 : 0));
                ls_cell[it] = (uint16_t)((i * m + b) | (pieces > 1 ? 0x8000 : 0));
            }
        }
        __syncthreads();
        // ---- inside a list: by residue class, then by index (a stable counting sort) ----
        for (int it = tid; it < nl; it += kBT) {
            uint16_t *e = sorted + ls_start[it];
            const int n = ls_len[it];
            uint16_t tmp[ML];
            int c8[NRES];
#pragma unroll
            for (int r = 0; r < NRES; ++r) c8[r] = 0;
            for (int a = 0; a < n; ++a) { tmp[a] = e[a]; c8[e[a] & (NRES - 1)]++; }
            int pos8[NRES], a0 = 0;
#pragma unroll
            for (int r = 0; r < NRES; ++r) { ls_res[8 * it + r] = (unsigned char)c8[r]; pos8[r] = a0; a0 += c8[r]; }
            for (int a = 0; a < n; ++a) e[pos8[tmp[a] & (NRES - 1)]++] = tmp[a];
            atomicAdd(&cls[n], 1);
        }
        __syncthreads();
        // ---- lists by length, longest first, ties by list number ----
        if (tid == 0) {
            int a = 0;
            for (int len = ML; len >= 1; --len) { const int v = cls[len]; cls[len] = a; a += v; }
        }
        __syncthreads();
        if (tid >= 1 && tid <= ML) {
            int r = cls[tid];
            for (int it = 0; it < nl; ++it)
                if (ls_len[it] == tid) order[r++] = (uint16_t)it;
        }
        __syncthreads();

        // ---- octets (one warp): the longest list left opens an octet; every further place goes
        // to the longest of the next kWindow lists that keeps all residue classes within the
        // opener's length (ties: a cell whose bank group the octet's flush does not use yet,
        // then the flattest classes); if none fits, to the one that raises the classes least ----
        const int no = (nl + NRES - 1) / NRES;
        if (tid < 32) {
            // order[head ..) are the lists not yet placed, longest first: a list taken from the
            // window is removed by moving the ones before it up by one, so the order is kept
            int head = 0;
            for (int o = 0; o < no; ++o) {
                const int first = order[head];
                int cols[NRES];
#pragma unroll
                for (int r = 0; r < NRES; ++r) cols[r] = ls_res[8 * first + r];
                const int L = ls_len[first];
                unsigned cellmask = 1u << (ls_cell[first] & 7);
                if (lane == 0) oc_list[8 * o] = (uint16_t)first;
                ++head;
                for (int place = 1; place < NRES; ++place) {
                    uint32_t best = 0xffffffffu;
#pragma unroll
                    for (int half = 0; half < kWindow / 32; ++half) {
                        const int slot = half * 32 + lane;
                        const int pos = head + slot;
                        if (pos < nl) {
                            const int cand = order[pos];
                            int mx = 0, sq = 0;
#pragma unroll
                            for (int r = 0; r < NRES; ++r) {
                                const int v = cols[r] + ls_res[8 * cand + r];
                                mx = max(mx, v);
                                sq += v * v;
                            }
                            uint32_t k;
                            if (mx <= L) {
                                const uint32_t conflict = (cellmask >> (ls_cell[cand] & 7)) & 1u;
                                // a flush conflict (two cells of the octet in one bank group) costs about
                                // as much as two idle steps of a lane
                                k = ((uint32_t)(L - ls_len[cand] + 2 * (int)conflict) << 23) |
                                    ((uint32_t)min(sq, 0xffff) << 6) | (uint32_t)slot;
                            } else {
                                k = 0x80000000u | ((uint32_t)min(mx, 0x3ff) << 21) |
                                    ((uint32_t)min(sq >> 6, 0x7fff) << 6) | (uint32_t)slot;
                            }
                            best = min(best, k);
                        }
                    }
                    best = __reduce_min_sync(0xffffffffu, best);
                    if (best == 0xffffffffu) {                       // no list left
                        if (lane == 0) oc_list[8 * o + place] = 0xffffu;
                        continue;
                    }
                    const int w = (int)(best & 63u);
                    const int cand = order[head + w];
#pragma unroll
                    for (int r = 0; r < NRES; ++r) cols[r] += ls_res[8 * cand + r];
                    cellmask |= 1u << (ls_cell[cand] & 7);
                    // close the gap: order[head .. head+w) moves up by one, head advances
                    uint16_t mv[kWindow / 32];
#pragma unroll
                    for (int half = 0; half < kWindow / 32; ++half) {
                        const int slot = half * 32 + lane;
                        mv[half] = slot < w ? order[head + slot] : (uint16_t)0;
                    }
                    __syncwarp();
#pragma unroll
                    for (int half = 0; half < kWindow / 32; ++half) {
                        const int slot = half * 32 + lane;
                        if (slot < w) order[head + slot + 1] = mv[half];
                    }
                    if (lane == 0) oc_list[8 * o + place] = (uint16_t)cand;
                    ++head;
                    __syncwarp();
                }
                int cost = L;
#pragma unroll
                for (int r = 0; r < NRES; ++r) cost = max(cost, cols[r]);
                if (lane == 0) oc_cost[o] = (uint16_t)cost;
            }
            if (lane == 0) tot[3] = no;
        }
        __syncthreads();
        // ---- octets by steps (most first, ties by number); four of them make an item ----
        for (int o = tid; o < no; o += kBT) {
            int rank = 0;
            const int co = oc_cost[o];
            for (int q = 0; q < no; ++q) rank += (oc_cost[q] > co || (oc_cost[q] == co && q < o)) ? 1 : 0;
            oc_order[rank] = (uint16_t)o;
        }
        __syncthreads();
        const int ni_row = (no + 3) / 4;
        const int item0 = tot[0], chunk0 = tot[1];
        __syncthreads();
        if (tid == 0) {
            int a = chunk0;
            for (int q = 0; q < ni_row; ++q) {
                const int steps = oc_cost[oc_order[4 * q]];
                it_steps[item0 + q] = (uint32_t)steps;
                it_chunk[item0 + q] = (uint32_t)a;
                a += (steps + 3) / 4;
            }
            tot[0] = item0 + ni_row;
            tot[1] = a;
        }
        __syncthreads();

        if (WRITE) {
            // ---- cell blocks ----
            uint16_t *cells = reinterpret_cast<uint16_t *>(rec + cells_off);
            for (int t = tid; t < ni_row * kListSlots; t += kBT) {
                const int q = t / kListSlots, ln = t % kListSlots;
                const int pos = 4 * q + ln / NRES;
                uint16_t cell = (uint16_t)(p.l * m);
                if (pos < no) {
                    const int li = oc_list[8 * oc_order[pos] + (ln % NRES)];
                    if (li != 0xffff) cell = ls_cell[li];
                }
                cells[(size_t)(item0 + q) * kListSlots + ln] = cell;
            }
            // ---- entries: one thread per octet place of the row's items ----
            uint16_t *ent = reinterpret_cast<uint16_t *>(rec + ent_off);
            // (spread over the warps of the block: the matching is serial code on private tables,
            // and threads of one warp would run its data-dependent paths one after the other)
            for (int pos = tid / kSpread; (tid % kSpread) == 0 && pos < 4 * ni_row; pos += kBT / kSpread) {
                const int q = pos / 4, lane0 = (pos % 4) * NRES;
                const int steps = (int)it_steps[item0 + q];
                const int padded = (steps + 3) & ~3;
                uint16_t *dst = ent + (size_t)it_chunk[item0 + q] * (kListSlots * 4);
                auto put = [&](int t, int s, uint16_t e) {
                    dst[(size_t)(t >> 2) * (kListSlots * 4) + (lane0 + s) * 4 + (t & 3)] = e;
                };
                int delta = 0;
                if (pos < no) {
                    const int o = oc_order[pos];
                    delta = oc_cost[o];
                    // C: indices of list s in class r; D: padding edges that make the graph regular.
                    // The tables live in shared memory (the hash words of the row are no longer
                    // needed): as private arrays they spill to local memory, which the block's
                    // shared-memory footprint leaves almost no L1 for.
                    unsigned char *mt = reinterpret_cast<unsigned char *>(key) + (size_t)pos * kMatchBytes;
                    unsigned char *C = mt, *D = mt + 64;
                    unsigned short *cur = reinterpret_cast<unsigned short *>(mt + 128);
                    signed char *match = reinterpret_cast<signed char *>(mt + 256);
                    signed char *matchR = match + 8, *prevS = match + 16, *queue = match + 24;
                    unsigned char *defL = mt + 288, *defR = mt + 296;
                    for (int r = 0; r < NRES; ++r) defR[r] = (unsigned char)delta;
                    for (int s = 0; s < NRES; ++s) {
                        const int li = oc_list[8 * o + s];
                        int a0 = li != 0xffff ? ls_start[li] : 0, len = 0;
                        for (int r = 0; r < NRES; ++r) {
                            const int v = li != 0xffff ? ls_res[8 * li + r] : 0;
                            C[s * NRES + r] = (unsigned char)v;
                            D[s * NRES + r] = 0;
                            cur[s * NRES + r] = (unsigned short)a0;
                            a0 += v;
                            len += v;
                            defR[r] = (unsigned char)(defR[r] - v);
                        }
                        defL[s] = (unsigned char)(delta - len);
                    }
                    for (int s = 0, r = 0; s < NRES && r < NRES;) {
                        const int x = min((int)defL[s], (int)defR[r]);
                        D[s * NRES + r] = (unsigned char)(D[s * NRES + r] + x);
                        defL[s] = (unsigned char)(defL[s] - x);
                        defR[r] = (unsigned char)(defR[r] - x);
                        if (defL[s] == 0) ++s; else ++r;
                    }
                    for (int s = 0; s < NRES; ++s) match[s] = -1;
                    for (int t = 0; t < delta; ++t) {
                        // keep the edges of the last matching that still exist, complete it with
                        // augmenting paths (a regular bipartite multigraph has a perfect matching)
                        for (int r = 0; r < NRES; ++r) matchR[r] = -1;
                        for (int s = 0; s < NRES; ++s) {
                            const int r = match[s];
                            if (r >= 0 && (C[s * NRES + r] | D[s * NRES + r]) != 0) matchR[r] = (signed char)s; else match[s] = -1;
                        }
                        for (int s0 = 0; s0 < NRES; ++s0) {
                            if (match[s0] >= 0) continue;
                            int qh = 0, qt = 0;
                            unsigned vis = 0;
                            queue[qt++] = (signed char)s0;
                            bool done = false;
                            while (qh < qt && !done) {
                                const int s = queue[qh++];
                                for (int r = 0; r < NRES && !done; ++r) {
                                    if ((vis >> r) & 1u) continue;
                                    if ((C[s * NRES + r] | D[s * NRES + r]) == 0) continue;
                                    vis |= 1u << r;
                                    prevS[r] = (signed char)s;
                                    if (matchR[r] < 0) {
                                        int rc = r;
                                        for (;;) {
                                            const int sp = prevS[rc];
                                            const int nr = match[sp];
                                            match[sp] = (signed char)rc;
                                            matchR[rc] = (signed char)sp;
                                            if (sp == s0) break;
                                            rc = nr;
                                        }
                                        done = true;
                                    } else {
                                        queue[qt++] = matchR[r];
                                    }
                                }
                            }
                        }
                        for (int s = 0; s < NRES; ++s) {
                            const int r = match[s];
                            uint16_t e;
                            if (r < 0) {                                  // cannot happen; keep the record valid
                                e = (uint16_t)(T + s);
                            } else if (C[s * NRES + r] != 0) {
                                e = sorted[cur[s * NRES + r]++];
                                C[s * NRES + r]--;
                            } else {
                                e = (uint16_t)(T + r);
                                D[s * NRES + r]--;
                            }
                            put(t, s, e);
                        }
                    }
                }
                for (int t = delta; t < padded; ++t)
                    for (int s = 0; s < NRES; ++s) put(t, s, (uint16_t)(T + s));
            }
        }
        __syncthreads();
    }

    // ---- items of the tile by steps, most first (ties by creation order) ----
    const int ni = tot[0], nch = tot[1];
    for (int q = tid; q < ni; q += kBT) {
        int rank = 0;
        const uint32_t sq = it_steps[q];
        for (int r = 0; r < ni; ++r) rank += (it_steps[r] > sq || (it_steps[r] == sq && r < q)) ? 1 : 0;
        it_rank[q] = (uint32_t)rank;
    }
    __syncthreads();
    if (!WRITE) {
        if (tid == 0) { p.rec_items[tile] = (uint32_t)ni; p.rec_chunks[tile] = (uint32_t)nch; }
    } else {
        uint32_t *hdr = reinterpret_cast<uint32_t *>(rec);
        if (tid == 0) {
            hdr[0] = (uint32_t)ni;
            hdr[1] = (uint32_t)(ent_off + (size_t)nch * 256);
            hdr[2] = (uint32_t)nch;
            hdr[3] = (ni == (int)rec_ni && nch == (int)p.rec_chunks[tile]) ? 0u : 1u;   // 1: the two passes disagree
        }
        for (int q = tid; q < ni; q += kBT) {
            uint32_t *dsc = hdr + 4 + 2 * it_rank[q];
            dsc[0] = (it_steps[q] & 0xffffu) | ((uint32_t)q << 16);
            dsc[1] = it_chunk[q];
        }
    }
}

}  // namespace

// Geometry of the schedule for a sketch of l x m: the largest tile (a multiple of kListBatch
// indices) whose two drift buffers fit beside the bins, or 0 when the lists would be too short.
static int list_tile_indices(const fda_ctx *ctx, int *ni_max_out)
{
    const int l = ctx->l, m = ctx->m;
    if (l == 0 || ctx->lm + 1 >= 0x8000) return 0;
    for (int T = kListMaxTile; T >= 2 * kListBatch; T -= kListBatch) {
        const int nl = (m < T ? m : T) + T / kListMaxLen;
        const int ni_max = l * ((nl + kListSlots - 1) / kListSlots);
        if (fda_list_smem_bytes(l, m, T, ni_max) > (size_t)ctx->smem_optin) continue;
        // Lists shorter than six entries on average do not pay for their flushes.
        if (T < 6 * m) return 0;
        *ni_max_out = ni_max;
        return T;
    }
    return 0;
}

cudaError_t fda_build_list_schedule(fda_ctx *ctx, cudaStream_t s)
{
    int ni_max = 0;
    const int T = list_tile_indices(ctx, &ni_max);
    if (T == 0) return cudaSuccess;
    const int64_t tiles = (ctx->d_max + T - 1) / T;
    if (tiles > 0x7fffffffLL) return cudaSuccess;

    SchedParams p{};
    p.coeffs = ctx->coeffs_dev; p.l = ctx->l; p.m = ctx->m; p.magic = ~0ull / (uint64_t)ctx->m;
    p.T = T;
    p.nl_max = (ctx->m < T ? ctx->m : T) + T / kListMaxLen;
    p.no_max = (p.nl_max + kListOct - 1) / kListOct;
    p.ni_row_max = (p.nl_max + kListSlots - 1) / kListSlots;
    const size_t bsmem = build_smem(p.l, p.m, T, p.nl_max, p.no_max, p.ni_row_max);
    if (bsmem > (size_t)ctx->smem_optin) return cudaSuccess;
    // the matching tables of a row's octets reuse the two arrays of hash words (8 bytes per index)
    if ((size_t)4 * p.ni_row_max * kMatchBytes > 2 * sizeof(uint32_t) * (size_t)T) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_build_schedule<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bsmem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_build_schedule<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bsmem);
    if (e != cudaSuccess) return e;

    uint32_t *items = nullptr, *chunks = nullptr;
    uint64_t *off = nullptr;
    unsigned char *buf = nullptr;
    auto cleanup = [&]() { cudaFree(items); cudaFree(chunks); cudaFree(off); cudaFree(buf); };
    if (cudaMalloc(&items, sizeof(uint32_t) * tiles) != cudaSuccess ||
        cudaMalloc(&chunks, sizeof(uint32_t) * tiles) != cudaSuccess ||
        cudaMalloc(&off, sizeof(uint64_t) * (tiles + 1)) != cudaSuccess) {
        cudaGetLastError();
        cleanup();
        return cudaSuccess;
    }
    p.rec_items = items; p.rec_chunks = chunks;
    k_build_schedule<false><<<(unsigned)tiles, kBT, bsmem, s>>>(p);
    e = cudaGetLastError();
    std::vector<uint32_t> h_items((size_t)tiles), h_chunks((size_t)tiles);
    std::vector<uint64_t> h_off((size_t)tiles + 1);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_items.data(), items, sizeof(uint32_t) * tiles, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_chunks.data(), chunks, sizeof(uint32_t) * tiles, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { cleanup(); return e; }
    uint64_t total = 0;
    for (int64_t t = 0; t < tiles; ++t) {
        h_off[t] = total;
        if ((int)h_items[t] > ni_max) { cleanup(); return cudaSuccess; }      // cannot happen; stay with the other kernels
        total += fda_sched_entries_off(h_items[t]) + (uint64_t)h_chunks[t] * 256;
    }
    h_off[tiles] = total;
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess || total > free_b / 3 ||
        (ctx->sched_limit_bytes > 0 && total > (uint64_t)ctx->sched_limit_bytes)) {
        cudaGetLastError();
        cleanup();
        ctx->sched_skipped_bytes = total;
        return cudaSuccess;                                                   // leave the memory to the models
    }
    if (cudaMalloc(&buf, total) != cudaSuccess) { cudaGetLastError(); cleanup(); ctx->sched_skipped_bytes = total; return cudaSuccess; }
    e = cudaMemcpyAsync(off, h_off.data(), sizeof(uint64_t) * (tiles + 1), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) { cleanup(); return e; }
    p.rec_off = off; p.sched = buf;
    k_build_schedule<true><<<(unsigned)tiles, kBT, bsmem, s>>>(p);
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(items); cudaFree(chunks);
    if (e != cudaSuccess) { cudaFree(off); cudaFree(buf); return e; }
    ctx->sched = buf; ctx->sched_off = off; ctx->sched_bytes = total; ctx->sched_T = T;
    ctx->sched_ni_max = ni_max; ctx->sched_tiles = tiles;
    return cudaSuccess;
}
