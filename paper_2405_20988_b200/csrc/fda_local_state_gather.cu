// Sketch pass with sorted per-cell lists (the main path of fda_local_state for aligned inputs).
//
// What the pass computes is stated in fda_local_state.cu (Section 3: drift and ||u||^2;
// Section 3.1: sk(u); Section 3.2: <xi,u>).  This file turns the scatter
// sk[i][h_i(j)] += s_i(j) u[j] into a gather: the bucket and sign of an index never change,
// so the context holds, for every (tile, sketch row), the tile's indices sorted by cell (the
// schedule of fda_sched.cu).  A warp then keeps the sums of 16 cells in registers, walks their
// lists and reads the drifts it needs from a transposed tile in shared memory; a cell of the
// bins is touched once per tile and list instead of once per update, with plain loads and
// stores, because a cell belongs to one list (cells that had to be split are added atomically).
// One update costs one 4-byte shared-memory read: measured on B200, 19-20 updates per clock
// and SM against 6 for compare-and-swap adds into the bins.
//
// A block serves a group of up to 8 workers and a strided set of tiles.  Per tile:
//   phase 1  16 loader warps bring the tile in with 16-byte asynchronous copies, 512 indices of
//            the 8 workers per step, each warp into its own part of a small ring (it reads back
//            only what it copied itself, so the ring needs no barrier, only the warp's own copy
//            groups); they subtract w_t0, add up ||u||^2 and <xi,u>, and store u transposed:
//            ut[index][worker], 32 bytes per index.  One more warp fetches the schedule headers
//            of the next tile and prefetches this tile's entries into L2;
//   phase 2  all 32 warps walk the lists: item (round r, sketch row i) goes to warp
//            (r*l + i) mod 32; the warp loads the item's entries, gathers and adds the 16 sums
//            to the bins.
// Lane = (slot q, half h): slot q walks one list, the two halves hold workers 4h .. 4h+3, so a
// gather is one 128-bit load per lane and a quarter-warp reads four 32-byte rows.
// The phases are separated by __syncthreads; nothing in this kernel waits on another block or
// on a barrier object.  Measured on B200 while this was built: tensor copies (TMA) of
// [8][252] or [8][256] boxes into a ring delivered 8-11 bytes per clock and SM here, no better
// than these copies; staging the tile in registers with scalar coalesced loads was slower
// (0.62 against 0.44 ms at d = 20M, K = 8).

#include <algorithm>

#include "fda_internal.h"

namespace {

constexpr int GW = kGatherWorkers;
constexpr int kLoaderWarps = 16;               // warps that stage and transpose the tile
constexpr int kWarps = 32;                     // + one warp that fetches the schedule headers; all walk the lists
constexpr int kThreads = kWarps * 32;
constexpr uint32_t kPrefix = kGatherPrefixBytes;   // counters and the warps' (norm, projection) sums
constexpr int kSlab = 2 * kGatherBox;          // indices staged per step: 32 per loader warp
constexpr uint32_t kUnitBytes = 1280;          // one warp's part of a stage: W [8][32], W0 [32], XI [32]
constexpr int kMaxStages = 6;                  // slab stages of the ring (copy groups pending per thread)
static_assert(kGatherMaxLen == 32, "walk_item is instantiated for up to 8 chunks of four steps");
static_assert(kLoaderWarps * 32 == kSlab, "a slab is 32 indices per loader warp");
static_assert(kLoaderWarps * (int)kUnitBytes == 2 * (kGatherWorkers * kGatherBox * 4 + 2 * kGatherBox * 4),
              "ring stage size differs from the one the tile size was chosen with");

struct GatherParams {
    const float *w, *w_t0, *xi;
    int64_t row_stride;
    int K;
    int64_t d;
    int have_xi;
    int l, m;
    int groups, cpg;                 // block = c * groups + g
    int nbox, stages, T;
    int64_t tiles;                   // tiles that hold indices below d
    int nr_max, hdr_bytes;
    size_t pitch;
    const unsigned char *sched;
    const uint16_t *used;            // [tile][row] entry chunks of a record
    float *part_sk;                  // [block][cell][GW]
    double *part_np;                 // [block][GW][2]
};

// Two schedule entries (the halves of one 32-bit word): gather the two rows and add them with
// their signs.  The sums stay packed as fp32 pairs from the first step to the flush, the loaded
// row arrives as two 64-bit registers, and the sign is a multiplication by (+-1, +-1) (exact),
// so a step is: one field extract, one address, one load, sign word, pair, two packed FMAs.
__device__ __forceinline__ void gather_pair(uint32_t w, uint32_t lane_base, unsigned long long &a01,
                                            unsigned long long &a23)
{
    uint32_t r1;
    asm("bfe.u32 %0, %1, 16, 13;" : "=r"(r1) : "r"(w));
    const uint32_t ad0 = lane_base + ((w & 0x1fffu) << 5), ad1 = lane_base + (r1 << 5);
    unsigned long long u0, u1, v0, v1, ss0, ss1;
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(u0), "=l"(u1) : "r"(ad0));
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(v0), "=l"(v1) : "r"(ad1));
    const uint32_t s0 = ((w << 16) & 0x80000000u) ^ 0x3f800000u;      // bit 15: sign of the low entry
    const uint32_t s1 = (w & 0x80000000u) ^ 0x3f800000u;              // bit 31: sign of the high entry
    asm("mov.b64 %0, {%1,%1};" : "=l"(ss0) : "r"(s0));
    asm("mov.b64 %0, {%1,%1};" : "=l"(ss1) : "r"(s1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a01) : "l"(u0), "l"(ss0));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a23) : "l"(u1), "l"(ss0));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a01) : "l"(v0), "l"(ss1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a23) : "l"(v1), "l"(ss1));
}

// One item: NCH chunks of four steps for this lane's slot (the last chunk holds two or four;
// `steps` is even).  All loads of the entries first, then the walk.
template <int NCH>
__device__ __forceinline__ float4 walk_item(const uint2 *ent, int steps, uint32_t lane_base)
{
    uint2 ch[NCH];
#pragma unroll
    for (int cc = 0; cc < NCH; ++cc) ch[cc] = __ldg(ent + cc * kGatherSlots);
    unsigned long long a01 = 0ull, a23 = 0ull;
#pragma unroll
    for (int cc = 0; cc < NCH; ++cc) {
        gather_pair(ch[cc].x, lane_base, a01, a23);
        if (cc + 1 < NCH || 4 * NCH - 2 < steps) gather_pair(ch[cc].y, lane_base, a01, a23);
    }
    float4 acc;
    asm("mov.b64 {%0,%1}, %2;" : "=f"(acc.x), "=f"(acc.y) : "l"(a01));
    asm("mov.b64 {%0,%1}, %2;" : "=f"(acc.z), "=f"(acc.w) : "l"(a23));
    return acc;
}

// 16-byte asynchronous copy global -> shared; bytes past `src_bytes` (0..16) arrive as zero
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// wait until at most `n` of this thread's copy groups are pending (n is uniform, below kMaxStages)
__device__ __forceinline__ void cp_async_wait(int n)
{
    switch (n) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
    }
}

// Shared-memory plan (bytes from the start of dynamic shared memory):
//   [136,140) rounds of the tile   [256, 2304) sums[loader warp][worker][2] (fp64)
//   [2304, ...) two buffers with the headers of a tile's l schedule records, hdr_bytes each
//   then        bins[l*m + 1][8]  (the last row takes the sums of unused slots)
//   then        ut[T + 4][8]      (drift tile, index-major; four zero rows behind it)
//   then, 128-byte aligned, the ring: per stage and loader warp W [8][32], W0 [32], XI [32]
template <bool LINEAR>
__global__ void __launch_bounds__(kThreads, 1) k_local_state_gather(const GatherParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 1, h = lane & 1;
    const int g = (int)blockIdx.x % p.groups, c = (int)blockIdx.x / p.groups;
    const int S = p.stages, nslab = p.nbox / 2, T = p.T, lm = p.l * p.m;

    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    int *nr_tile_p = reinterpret_cast<int *>(smem_raw + 136);
    const uint32_t hdr_buf_bytes = (uint32_t)(p.l * p.hdr_bytes);       // two header buffers: tile n uses n & 1
    double *sums = reinterpret_cast<double *>(smem_raw + 256);
    const uint32_t bins_off = kPrefix + 2u * hdr_buf_bytes;
    const uint32_t ut_off = bins_off + (uint32_t)(lm + 1) * 32u;
    const uint32_t ring_off = (ut_off + (uint32_t)(T + kGatherPadRows) * 32u + 127u) & ~127u;
    float *bins = reinterpret_cast<float *>(smem_raw + bins_off);
    float *ut = reinterpret_cast<float *>(smem_raw + ut_off);
    const uint32_t ut_addr = smem_base + ut_off;

    for (int t = tid; t < (lm + 1) * GW; t += kThreads) bins[t] = 0.f;
    for (int t = tid; t < kGatherPadRows * GW; t += kThreads) ut[T * GW + t] = 0.f;
    for (int t = tid; t < kLoaderWarps * GW * 2; t += kThreads) sums[t] = 0.0;
    __syncthreads();

    const int64_t my_tiles = p.tiles > c ? (p.tiles - c + p.cpg - 1) / p.cpg : 0;
    const int64_t total_slabs = my_tiles * nslab;

    // ---- loader state (warps below kLoaderWarps).  A slab is 512 indices of the 8 workers; a
    // warp owns 32 of them: it copies them into its own part of the ring, 16 bytes per lane
    // (two copies of 4 rows x 128 bytes, one for w_t0 and xi), and later reads them back itself,
    // so the ring needs no barrier, only the warp's own copy groups. ----
    const uint32_t my_ring = smem_base + ring_off + (uint32_t)warp * kUnitBytes;
    const uint32_t slab_stage_bytes = kLoaderWarps * kUnitBytes;
    // Running pointers of this lane's copies (lane = 8 * row + 16-byte piece): rows cr and 4 + cr of
    // the group at this lane's column, and the column of w_t0 (lanes 0..7) or xi (lanes 8..15).
    const int cr = lane >> 3, cpiece = lane & 7;
    const bool k0ok = g * GW + cr < p.K, k1ok = g * GW + 4 + cr < p.K;
    const int64_t col0 = (int64_t)c * T + 32 * warp;         // first index of this warp in its first slab
    const float *wp0 = p.w + (size_t)(g * GW + cr) * (size_t)p.row_stride + col0 + 4 * cpiece;
    const float *wp1 = wp0 + 4 * (size_t)p.row_stride;
    const float *vp = ((LINEAR && lane >= 8) ? p.xi : p.w_t0) + col0 + 4 * cpiece;
    int64_t rem = p.d - (col0 + 4 * cpiece);                 // floats of the row from this lane's column on
    const int64_t wrap = (int64_t)(p.cpg - 1) * T;           // from the end of a tile to this block's next tile
    const uint32_t lane_dst = my_ring + 16u * (uint32_t)lane;
    int ld_sb = 0, ld_stage = 0, rd_stage = 0;
    int ld_left = (int)total_slabs;                          // fits: below 2^31 / 512 slabs in all
    auto load_slab = [&]() {                                 // one copy group, empty when nothing is left
        if (ld_left > 0) {
            --ld_left;
            const uint32_t nb = rem >= 4 ? 16u : (rem > 0 ? 4u * (uint32_t)rem : 0u);
            const uint32_t dst = lane_dst + (uint32_t)ld_stage * slab_stage_bytes;
            cp_async16(dst, (k0ok && nb) ? wp0 : p.w_t0, k0ok ? nb : 0u);
            cp_async16(dst + 512u, (k1ok && nb) ? wp1 : p.w_t0, k1ok ? nb : 0u);
            if (lane < (LINEAR ? 16 : 8)) cp_async16(dst + 1024u, nb ? vp : p.w_t0, nb);
            int64_t adv = kSlab;
            if (++ld_sb == nslab) { ld_sb = 0; adv += wrap; }
            wp0 += adv; wp1 += adv; vp += adv; rem -= adv;
            if (++ld_stage == S) ld_stage = 0;
        }
        cp_async_commit();
    };
    if (warp < kLoaderWarps)
        for (int st = 0; st < S - 1; ++st) load_slab();

    // the extra warp fetches the schedule headers one tile ahead (asynchronous copies into the
    // other header buffer) and keeps the entry-chunk counts of the tile to come (lane i: row i)
    auto fetch_headers = [&](int64_t tile_, int buf) {
        const unsigned char *src0 = p.sched + (size_t)tile_ * p.l * p.pitch;
        for (int i = 0; i < p.l; ++i) {
            const unsigned char *src = src0 + (size_t)i * p.pitch;
            const uint32_t dst = smem_base + kPrefix + (uint32_t)buf * hdr_buf_bytes + (uint32_t)(i * p.hdr_bytes);
            for (int t = lane; t < p.hdr_bytes / 16; t += 32) cp_async16(dst + 16u * t, src + 16 * t, 16u);
        }
    };
    int my_used = 0;
    if (warp == kLoaderWarps && my_tiles > 0) {
        if (lane < p.l) my_used = p.used[(int64_t)c * p.l + lane];
        fetch_headers(c, 0);
    }
    const uint32_t gather_base = ut_addr + (uint32_t)h * 16u;

    for (int64_t n = 0; n < my_tiles; ++n) {
        const int64_t tile = c + n * p.cpg;
        const unsigned char *rec0 = p.sched + (size_t)tile * p.l * p.pitch;
        const unsigned char *hdr = smem_raw + kPrefix + (size_t)(n & 1) * hdr_buf_bytes;
        // ================= phase 1: ring -> drift tile =================
        if (warp < kLoaderWarps) {
            float nf[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}}, pf[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            for (int sb = 0; sb < nslab; ++sb) {
                load_slab();                     // the slab S-1 ahead, into the stage read last time
                cp_async_wait(S - 1);            // this thread's copies of the slab to read have landed
                __syncwarp();                    // ... and so have the other lanes'
                const float *src = reinterpret_cast<const float *>(smem_raw + ring_off + (uint32_t)warp * kUnitBytes +
                                                                   (uint32_t)rd_stage * slab_stage_bytes);
                if (++rd_stage == S) rd_stage = 0;
                // two steps: lanes h = 0 take index q with workers 4*hh .. 4*hh+3, lanes h = 1 index
                // 16 + q with the other four (rows of the unit are 32 floats: the halves use
                // different banks); the second step swaps the worker halves.  All ten loads first.
                const int xl = 16 * h + q;
                const float w0 = src[256 + xl];
                const float xv = LINEAR ? src[288 + xl] : 0.f;
                float wv[2][4];
#pragma unroll
                for (int step = 0; step < 2; ++step)
#pragma unroll
                    for (int e = 0; e < 4; ++e) wv[step][e] = src[(4 * (h ^ step) + e) * 32 + xl];
#pragma unroll
                for (int step = 0; step < 2; ++step) {
                    const int hh = h ^ step;
                    const float u0 = wv[step][0] - w0, u1 = wv[step][1] - w0, u2 = wv[step][2] - w0, u3 = wv[step][3] - w0;
                    nf[step][0] = fmaf(u0, u0, nf[step][0]); nf[step][1] = fmaf(u1, u1, nf[step][1]);
                    nf[step][2] = fmaf(u2, u2, nf[step][2]); nf[step][3] = fmaf(u3, u3, nf[step][3]);
                    if (LINEAR) {
                        pf[step][0] = fmaf(xv, u0, pf[step][0]); pf[step][1] = fmaf(xv, u1, pf[step][1]);
                        pf[step][2] = fmaf(xv, u2, pf[step][2]); pf[step][3] = fmaf(xv, u3, pf[step][3]);
                    }
                    *reinterpret_cast<float4 *>(ut + (size_t)(sb * kSlab + 32 * warp + xl) * GW + 4 * hh) =
                        make_float4(u0, u1, u2, u3);
                }
                __syncwarp();                    // all reads of this stage are done before it is refilled
            }
            // lane h holds workers 4*(h^step) + e in nf[step][e]: fold to workers 4*h + e, add up the
            // warp's 16 index columns and keep the tile's sums in fp64 (lanes 0 and 1 own the slots)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float a = nf[0][e] + __shfl_xor_sync(0xffffffffu, nf[1][e], 1);
                float bq = LINEAR ? pf[0][e] + __shfl_xor_sync(0xffffffffu, pf[1][e], 1) : 0.f;
#pragma unroll
                for (int off = 2; off < 32; off <<= 1) {
                    a += __shfl_xor_sync(0xffffffffu, a, off);
                    if (LINEAR) bq += __shfl_xor_sync(0xffffffffu, bq, off);
                }
                if (lane < 2) {
                    sums[(warp * GW + 4 * lane + e) * 2 + 0] += (double)a;
                    if (LINEAR) sums[(warp * GW + 4 * lane + e) * 2 + 1] += (double)bq;
                }
            }
        } else if (warp == kLoaderWarps) {
            // ---- one more warp: this tile's headers have arrived; L2 prefetch of its entries;
            // headers and chunk counts of the next tile ----
            asm volatile("cp.async.wait_all;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                int nr = 0;
                for (int i = 0; i < p.l; ++i)
                    nr = max(nr, (int)*reinterpret_cast<const uint16_t *>(hdr + (size_t)i * p.hdr_bytes));
                *nr_tile_p = nr;
            }
            for (int i = 0; i < p.l; ++i) {
                const int chunks = __shfl_sync(0xffffffffu, my_used, i);
                const unsigned char *ent = rec0 + (size_t)i * p.pitch + p.hdr_bytes;
                for (int t = lane; t < chunks; t += 32)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(ent + (size_t)t * 128));
            }
            if (n + 1 < my_tiles) {
                if (lane < p.l) my_used = p.used[(tile + p.cpg) * p.l + lane];
                fetch_headers(tile + p.cpg, (int)((n + 1) & 1));
            }
        }
        __syncthreads();
        // ================= phase 2: walk the lists =================
        // Item (round r, sketch row i) number r*l + i goes to warp (r*l + i) mod kWarps: rounds are
        // ordered by length, so every warp gets long and short ones.
        {
            const int nr_tile = *nr_tile_p;
            int r = warp / p.l, i = warp - r * p.l;
            const int dr = kWarps / p.l, di = kWarps - dr * p.l;
            for (; r < nr_tile; r += dr, i += di) {
                if (i >= p.l) { i -= p.l; ++r; if (r >= nr_tile) break; }
                const unsigned char *hrow = hdr + (size_t)i * p.hdr_bytes;
                const uint16_t *hi = reinterpret_cast<const uint16_t *>(hrow);
                if (r >= (int)hi[0]) continue;
                const int steps = hi[2 + r];
                const int coff = hi[2 + p.nr_max + r];
                const uint32_t cell = reinterpret_cast<const uint16_t *>(hrow + fda_sched_cells_off(p.nr_max))[r * kGatherSlots + q];
                const uint2 *ent = reinterpret_cast<const uint2 *>(rec0 + (size_t)i * p.pitch + p.hdr_bytes +
                                                                   (size_t)coff * 128) + q;
                float4 acc;
                switch ((steps + 3) >> 2) {                     // straight-line code per chunk count
                    case 1: acc = walk_item<1>(ent, steps, gather_base); break;
                    case 2: acc = walk_item<2>(ent, steps, gather_base); break;
                    case 3: acc = walk_item<3>(ent, steps, gather_base); break;
                    case 4: acc = walk_item<4>(ent, steps, gather_base); break;
                    case 5: acc = walk_item<5>(ent, steps, gather_base); break;
                    case 6: acc = walk_item<6>(ent, steps, gather_base); break;
                    case 7: acc = walk_item<7>(ent, steps, gather_base); break;
                    default: acc = walk_item<8>(ent, steps, gather_base); break;
                }
                float *b = bins + (cell & 0x7fffu) * GW + h * 4;
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
        __syncthreads();
    }

    // ---- flush: bins -> this block's partial sketch ----
    __syncthreads();
    {
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)lm * GW;
        for (int t = tid; t < lm * GW; t += kThreads) out[t] = bins[t];
    }
    // ---- block partial of (||u||^2, <xi,u>) per worker ----
    if (tid < GW * 2) {
        double t = 0.0;
        for (int wv = 0; wv < kLoaderWarps; ++wv) t += sums[wv * GW * 2 + tid];
        p.part_np[(size_t)blockIdx.x * GW * 2 + tid] = t;
    }
}

// states[k][.] = sum of the partials of worker k's blocks in fp64, in a fixed order: four
// adjacent lanes share one output, lane s adds the blocks s, s + 4, ... of the worker's group in
// order (eight loads in flight), and the four sums are added as (s0 + s1) + (s2 + s3).
__global__ void k_finalize_gather(const GatherParams p, int blocks, uint32_t flags, float *__restrict__ states)
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

}  // namespace

// Returns cudaErrorNotSupported when the request does not fit this path (the caller then uses
// the other kernels); any other value is the result of the launches.
cudaError_t fda_launch_local_state_gather(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s)
{
    if (!(flags & FDA_STATE_SKETCH) || ctx->l == 0 || !ctx->sched) return cudaErrorNotSupported;
    const float *xi_used = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
    const bool aligned = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) &&
                         (row_stride % 4 == 0);
    if (!aligned) return cudaErrorNotSupported;

    GatherParams p{};
    p.w = w; p.w_t0 = w_t0; p.xi = xi_used; p.row_stride = row_stride;
    p.K = K; p.d = d; p.have_xi = xi_used != nullptr;
    p.l = ctx->l; p.m = ctx->m;
    p.nbox = ctx->sched_nbox; p.T = p.nbox * kGatherBox;
    p.nr_max = ctx->sched_nr_max; p.hdr_bytes = ctx->sched_hdr_bytes;
    p.pitch = ctx->sched_pitch; p.sched = ctx->sched; p.used = ctx->sched_used;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np;
    p.tiles = (d + p.T - 1) / p.T;
    p.groups = (K + GW - 1) / GW;
    if (p.groups > ctx->n_sm) return cudaErrorNotSupported;
    int64_t cpg = ctx->n_sm / p.groups;
    // short jobs (measured at d = 1.2M, K = 10: 78 against 69 microseconds) stay with the other kernels
    if (p.tiles < 8 * cpg) return cudaErrorNotSupported;
    p.cpg = (int)cpg;
    const int blocks = p.groups * p.cpg;
    if ((size_t)blocks * ctx->lm * GW > ctx->part_sk_floats || blocks > ctx->max_blocks ||
        (size_t)blocks * GW * 2 > ctx->part_np_doubles)
        return cudaErrorNotSupported;

    const size_t ring_off = (kPrefix + 2 * (size_t)p.l * p.hdr_bytes + ((size_t)ctx->lm + 1) * 32 +
                             (size_t)(p.T + kGatherPadRows) * 32 + 127) / 128 * 128;
    const size_t stage_bytes = (size_t)kLoaderWarps * kUnitBytes;
    if (p.nbox % 2 != 0 || (size_t)ctx->smem_optin < ring_off + 2 * stage_bytes) return cudaErrorNotSupported;
    int stages = (int)(((size_t)ctx->smem_optin - ring_off) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    p.stages = stages;
    const size_t smem = ring_off + (size_t)stages * stage_bytes;

    auto kern = xi_used ? k_local_state_gather<true> : k_local_state_gather<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, kThreads, smem, s>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)p.groups * (2 + ctx->lm) * GW * 4;
    int fb = (int)((total + 255) / 256);
    if (fb > ctx->n_sm * 8) fb = ctx->n_sm * 8;
    k_finalize_gather<<<fb, 256, 0, s>>>(p, blocks, flags, states);
    return cudaGetLastError();
}
