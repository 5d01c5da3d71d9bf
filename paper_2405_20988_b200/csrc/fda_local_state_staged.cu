// Sketch pass with TMA-staged tiles (the main path of fda_local_state for aligned inputs).
//
// What the pass computes is stated in fda_local_state.cu (Section 3: drift and ||u||^2;
// Section 3.1: sk(u); Section 3.2: <xi,u>).  This file differs in how data reaches the lanes.
//
// Measured on B200: fp32 adds into shared memory are compare-and-swap loops (there is no
// native instruction), and the data pipe of the load/store unit is the binding resource of
// the pass.  A lane = worker mapping that loads w straight from global memory spends ~40 %
// of that pipe on 32-row uncoalesced 16-byte loads, so each tile is staged in shared memory
// by the TMA engine instead and read back with conflict-free 128-bit loads.  Row-by-row
// bulk copies (cp.async.bulk) were measured at one copy per 230-420 clocks per SM, which
// starves tiles made of 30+ short rows; 16-byte cp.async from all threads loads the same
// pipe the scatter needs.  Hence tiled tensor copies: one cp.async.bulk.tensor.2d brings a
// [workers x BX] box, with BX/4 odd so that the dense box rows fall on
// different banks, and zero-fills everything outside the tensor (ragged end, missing rows).
// No multicast is used anywhere.
//
// Block roles.  A block serves (row subset, worker group, tile chunk).  When the l x m bins
// with 32 lane-private columns do not fit beside the ring, the sketch rows are split over
// several blocks ("roles"); every role re-reads the tile through L2 and only role 0
// accumulates the norm and the projection.
//
// Pipeline.  Warp 0 produces (one elected lane issues the tensor copies of a tile), the other
// warps consume.  full[s] completes when a tile's bytes have landed, empty[s] when every
// consumer warp has released the stage.  Every wait is bounded: when it runs out the thread
// raises the context's error word and stops waiting, so the kernel always returns.
//
// Updates.  Four shared-memory updates per lane are in flight (four loads, four adds, four
// compare-and-swaps); an update whose compare-and-swap lost a race is redone with an
// atomic add.  Lanes own their column, so races only occur between warps that hit the same
// cell, or between two of a lane's own four updates.  (Giving each sketch row to one warp and
// updating with plain load-add-store, which needs no retries and is bit-reproducible, was
// measured 3.4x slower here: too few warps to hide the shared-memory latency.)
#include <cuda.h>

#include <algorithm>

#include "fda_internal.h"

namespace {

constexpr int kMaxThreads = 1024;
constexpr int kMaxUnits = 64;
constexpr int kMaxBoxes = 4;                   // tensor boxes per tile
constexpr uint32_t kWaitLimit = 1u << 24;      // polls of an mbarrier before giving up

struct StagedParams {
    int K;
    int64_t d;
    bool have_xi;
    int l, m;
    int Kg, groups;
    int roles, rows_per_role;        // role r owns rows [r*rows_per_role, min(l, ...))
    int bx, nb;                      // box width (floats, bx/4 odd) and boxes per tile
    int stages;                      // depth of the shared-memory ring
    int64_t tiles;                   // ceil(d / (bx*nb))
    uint32_t wbox_bytes, vbox_bytes, hbox_bytes;   // 128-byte aligned sizes of one box
    int unit_first_block[kMaxUnits + 1];           // unit = role*groups + group
    float *part_sk;                  // [block][local cell][LWK], block pitch = part_pitch floats
    size_t part_pitch;
    double *part_np;                 // [block][LWK][2]
    unsigned int *err_flag;
};

__device__ __forceinline__ float flip(float v, uint32_t signbit)
{
    return __uint_as_float(__float_as_uint(v) ^ signbit);
}
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t cas_shared(uint32_t addr, uint32_t expect, uint32_t val)
{
    uint32_t old;
    asm volatile("atom.shared.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "r"(addr), "r"(expect), "r"(val) : "memory");
    return old;
}
__device__ __forceinline__ void red_shared_add(uint32_t addr, float v)
{
    asm volatile("red.shared.add.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t addr, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t addr)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t addr, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    return ok != 0;
}
// Tiled 2-D tensor copy global -> shared (no multicast).  dst 128-byte aligned; x times the
// element size a multiple of 16 bytes; elements outside the tensor arrive as zero.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t mbar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(mbar) : "memory");
}

// N updates of lane-private cells: N loads, N adds, N compare-and-swaps in flight; the ones that
// lost a race are redone with an atomic add.  (The kernel is close to its instruction-issue
// limit: this straight-line retry replaced a loop that merged the lanes' retries into fewer
// atomic instructions and was 6 % slower.)
template <int N>
__device__ __forceinline__ void apply_updates(const uint32_t (&addr)[N], const float (&val)[N])
{
    float old[N];
    uint32_t got[N];
#pragma unroll
    for (int e = 0; e < N; ++e) old[e] = lds_f32(addr[e]);
    uint32_t diff = 0;
#pragma unroll
    for (int e = 0; e < N; ++e) {
        got[e] = cas_shared(addr[e], __float_as_uint(old[e]), __float_as_uint(old[e] + val[e]));
        diff |= got[e] ^ __float_as_uint(old[e]);
    }
    if (diff) {
#pragma unroll
        for (int e = 0; e < N; ++e)
            if (got[e] != __float_as_uint(old[e])) red_shared_add(addr[e], val[e]);
    }
}

// Shared-memory plan (bytes from the start of dynamic shared memory):
//   [0, 64)                  mbarriers: full[s] at 8*s, empty[s] at 32 + 8*s
//   [128, 128 + bins_bytes)  bins[local cell][32]
//   then `stages` stages, each holding, for box b < nb:
//        W  [Kg][bx] floats        at b*wbox_bytes
//        W0 [bx] floats            at nb*wbox_bytes + b*vbox_bytes
//        XI [bx] floats            at nb*(wbox_bytes + vbox_bytes) + b*vbox_bytes
//        H  [rows_per_role][bx] uint32    at nb*(wbox_bytes + 2*vbox_bytes) + b*hbox_bytes
// A lane takes one index quad per pass: four updates in flight per lane and sketch row.  Two
// quads (eight in flight) or two rows at once (sixteen) were measured slower: what pays is
// many warps with short windows between load and compare-and-swap, which keeps the share of
// lost races down.
template <int LWK, bool LINEAR, int ROWS /* sketch rows, 0 = read at run time */>
__global__ void __launch_bounds__(kMaxThreads, 1)
k_local_state_staged(const StagedParams p, const __grid_constant__ CUtensorMap tm_w,
                     const __grid_constant__ CUtensorMap tm_w0, const __grid_constant__ CUtensorMap tm_xi,
                     const __grid_constant__ CUtensorMap tm_tab)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr int JS = 32 / LWK;
    constexpr int QPL = 1;                      // index quads per lane and pass
    constexpr int NB = 4 * QPL;                 // updates in flight per lane
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int ncons = nwarps - 1;               // consumer warps
    const int cw = warp - 1;                    // consumer index (-1: producer)
    const int kl = lane % LWK, s = lane / LWK;

    // ---- which (role, group, chunk) am I ----
    int unit = 0;
    while (unit + 1 < p.roles * p.groups && (int)blockIdx.x >= p.unit_first_block[unit + 1]) ++unit;
    const int role = unit / p.groups, g = unit % p.groups;
    const int c = (int)blockIdx.x - p.unit_first_block[unit];
    const int cpg = p.unit_first_block[unit + 1] - p.unit_first_block[unit];
    const int row0 = role * p.rows_per_role;
    const int rows = min(p.rows_per_role, p.l - row0);
    const int kg_here = min(p.Kg, p.K - g * p.Kg);
    const bool active = kl < kg_here;
    const bool do_np = role == 0;

    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
    const uint32_t bins_addr = smem_base + 128;
    const int local_cells = p.rows_per_role * p.m;
    const uint32_t bins_bytes = (uint32_t)local_cells * 32u * 4u;
    const int S = p.stages, nb = p.nb, bx = p.bx;
    const uint32_t w0_off = (uint32_t)nb * p.wbox_bytes;
    const uint32_t xi_off = w0_off + (uint32_t)nb * p.vbox_bytes;
    const uint32_t h_off = xi_off + (uint32_t)nb * p.vbox_bytes;
    const uint32_t stage_bytes = h_off + (uint32_t)nb * p.hbox_bytes;
    const uint32_t stage0 = bins_addr + bins_bytes;
    const int tile = bx * nb;

    float *bins = reinterpret_cast<float *>(smem_raw + 128);
    for (int i = tid; i < local_cells * 32; i += blockDim.x) bins[i] = 0.f;
    if (tid == 0) {
        for (int st = 0; st < S; ++st) {
            mbar_init(smem_base + 8u * st, 1);
            mbar_init(smem_base + 32u + 8u * st, (uint32_t)ncons);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int64_t my_tiles = p.tiles > c ? (p.tiles - c + cpg - 1) / cpg : 0;
    // a tensor copy always delivers its whole box (zero-filled where outside the tensor)
    const uint32_t tx_bytes = (uint32_t)nb * ((uint32_t)(p.Kg * bx) * 4u + (uint32_t)bx * 4u * (LINEAR ? 2u : 1u) +
                                              (uint32_t)(p.rows_per_role * bx) * 4u);

    double acc_n = 0.0, acc_p = 0.0;
    // table words hold the cell of the whole sketch: take off this role's first cell (the table
    // is padded past the last tile, so every word read is a valid cell of the row it belongs to)
    const uint32_t col_addr = bins_addr + (uint32_t)lane * 4u - (((uint32_t)(row0 * p.m)) << 7);
    const int qpb = bx / 4;                                        // quads per box
    const int quads = qpb * nb;                                    // quads per tile
    const int quads_per_pass = ncons * JS * QPL;
    const int passes = (quads + quads_per_pass - 1) / quads_per_pass;

    // one staged tile -> bins (+ norm / projection partials); consumer warps only
    // q / qpb for q < 1024 and qpb < 64 by multiplication (exact on that range)
    const uint32_t qpb_inv = (65536u + (uint32_t)qpb - 1u) / (uint32_t)qpb;
    auto process = [&](uint32_t base, int64_t j0) {
        if (!active) return;
        float tile_n = 0.f, tile_p = 0.f;      // fp32 over one tile (a few quads per lane), fp64 across tiles
        for (int ps = 0; ps < passes; ++ps) {
            float u[NB];
            uint32_t haddr[QPL];
            bool any = false;
            float pp = 0.f;
#pragma unroll
            for (int v = 0; v < QPL; ++v) {
                const int q = (ps * ncons + cw) * (JS * QPL) + v * JS + s;       // quad inside the tile
                const bool in = q < quads;
                any |= in;
                const int b = in ? (int)(((uint32_t)q * qpb_inv) >> 16) : 0, xq = in ? q - b * qpb : 0;
                haddr[v] = base + h_off + (uint32_t)b * p.hbox_bytes + 16u * (uint32_t)xq;
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), w0 = a;
                if (in) {
                    a = lds_f32x4(base + (uint32_t)b * p.wbox_bytes + ((uint32_t)(kl * bx) + 4u * (uint32_t)xq) * 4u);
                    w0 = lds_f32x4(base + w0_off + (uint32_t)b * p.vbox_bytes + 16u * (uint32_t)xq);
                }
                u[4 * v + 0] = a.x - w0.x; u[4 * v + 1] = a.y - w0.y;
                u[4 * v + 2] = a.z - w0.z; u[4 * v + 3] = a.w - w0.w;
                if (LINEAR && in && do_np) {
                    const float4 x = lds_f32x4(base + xi_off + (uint32_t)b * p.vbox_bytes + 16u * (uint32_t)xq);
                    pp = fmaf(x.x, u[4 * v + 0], pp); pp = fmaf(x.y, u[4 * v + 1], pp);
                    pp = fmaf(x.z, u[4 * v + 2], pp); pp = fmaf(x.w, u[4 * v + 3], pp);
                }
            }
            if (!any) continue;
            if (do_np) {
                float pn = 0.f;
#pragma unroll
                for (int e = 0; e < NB; ++e) pn = fmaf(u[e], u[e], pn);
                tile_n += pn;
                if (LINEAR) tile_p += pp;
            }
            auto row_updates = [&](int i, uint32_t *addr, float *val) {
#pragma unroll
                for (int v = 0; v < QPL; ++v) {
                    // 4 table words of this quad: cell | sign << 31 (u = 0 where the quad is absent)
                    uint32_t h[4];
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]) : "r"(haddr[v] + (uint32_t)(i * bx) * 4u));
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        addr[4 * v + e] = col_addr + (h[e] << 7);     // the shift drops the sign bit
                        val[4 * v + e] = flip(u[4 * v + e], h[e] & 0x80000000u);
                    }
                }
            };
            if (ROWS > 0) {
#pragma unroll
                for (int i = 0; i < ROWS; ++i) {
                    uint32_t addr[NB];
                    float val[NB];
                    row_updates(i, addr, val);
                    apply_updates<NB>(addr, val);
                }
            } else {
                for (int i = 0; i < rows; ++i) {
                    uint32_t addr[NB];
                    float val[NB];
                    row_updates(i, addr, val);
                    apply_updates<NB>(addr, val);
                }
            }
        }
        acc_n += (double)tile_n;
        if (LINEAR) acc_p += (double)tile_p;
    };

    bool dead = false;
    if (warp == 0) {
        // ---- producer: keep the ring full ----
        for (int64_t n = 0; n < my_tiles; ++n) {
            const int st = (int)(n % S);
            const int64_t use = n / S;
            const uint32_t mbar = smem_base + 8u * st;
            if (use > 0) {                      // wait until the consumers released the previous use
                const uint32_t parity = (uint32_t)((use - 1) & 1);
                uint32_t polls = 0;
                while (!mbar_try_wait(smem_base + 32u + 8u * st, parity)) {
                    if (++polls > kWaitLimit) { dead = true; atomicExch(p.err_flag, 1u); break; }
                }
                dead = __any_sync(0xffffffffu, dead);
                if (dead) break;
            }
            if (lane == 0) {
                const int64_t j0 = (c + n * cpg) * (int64_t)tile;
                const uint32_t base = stage0 + (uint32_t)st * stage_bytes;
                mbar_expect_tx(mbar, tx_bytes);
                for (int b = 0; b < nb; ++b) {
                    const int x = (int)(j0 + (int64_t)b * bx);
                    tma_load_2d(base + (uint32_t)b * p.wbox_bytes, &tm_w, x, g * p.Kg, mbar);
                    tma_load_2d(base + w0_off + (uint32_t)b * p.vbox_bytes, &tm_w0, x, 0, mbar);
                    if (LINEAR) tma_load_2d(base + xi_off + (uint32_t)b * p.vbox_bytes, &tm_xi, x, 0, mbar);
                    tma_load_2d(base + h_off + (uint32_t)b * p.hbox_bytes, &tm_tab, x, row0, mbar);
                }
            }
            __syncwarp();
        }
    } else {
        // ---- consumers ----
        for (int64_t n = 0; n < my_tiles; ++n) {
            const int st = (int)(n % S);
            const uint32_t parity = (uint32_t)((n / S) & 1);
            uint32_t polls = 0;
            while (!mbar_try_wait(smem_base + 8u * st, parity)) {
                if (++polls > kWaitLimit) { dead = true; atomicExch(p.err_flag, 1u); break; }
            }
            dead = __any_sync(0xffffffffu, dead);
            if (dead) break;
            process(stage0 + (uint32_t)st * stage_bytes, (c + n * cpg) * (int64_t)tile);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_base + 32u + 8u * st);       // release the stage
        }
    }

    // ---- flush: bins -> this block's partial (sum of the columns of each worker) ----
    __syncthreads();
    {
        float *out = p.part_sk + (size_t)blockIdx.x * p.part_pitch;
        const int reps = 32 / LWK;
        const int cells = rows * p.m;
        for (int idx = tid; idx < cells * LWK; idx += blockDim.x) {
            const int cell = idx / LWK, w_in = idx % LWK;
            float v = 0.f;
            for (int r = 0; r < reps; ++r) v += bins[cell * 32 + r * LWK + w_in];
            out[idx] = v;
        }
        __syncthreads();
    }
    // ---- block partial of (||u||^2, <xi,u>) per worker ----
#pragma unroll
    for (int off = LWK; off < 32; off <<= 1) {
        acc_n += __shfl_xor_sync(0xffffffffu, acc_n, off);
        acc_p += __shfl_xor_sync(0xffffffffu, acc_p, off);
    }
    double *red = reinterpret_cast<double *>(smem_raw + 128);       // [nwarps][LWK][2], reuses the bins
    if (lane < LWK) {
        red[(warp * LWK + lane) * 2 + 0] = acc_n;
        red[(warp * LWK + lane) * 2 + 1] = acc_p;
    }
    __syncthreads();
    if (tid < LWK * 2) {
        double t = 0.0;
        for (int wv = 0; wv < nwarps; ++wv) t += red[wv * LWK * 2 + tid];
        p.part_np[(size_t)blockIdx.x * LWK * 2 + tid] = t;
    }
}

// states[k][.] = sum of the partials of worker k's blocks, in block order, in fp64.
template <int LWK>
__global__ void k_finalize_staged(const StagedParams p, uint32_t flags, float *__restrict__ states)
{
    const int lm = p.l * p.m, slen = 2 + lm;
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    const int64_t per_group = (int64_t)(lm + 2) * LWK;
    const int64_t total = per_group * p.groups;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(t / per_group);
        const int r = (int)(t % per_group);
        const int e = r / LWK, kl = r % LWK;
        const int k = g * p.Kg + kl;
        if (kl >= p.Kg || k >= p.K) continue;
        double acc = 0.0;
        if (e < 2) {
            const bool on = (e == 0) ? (flags & FDA_STATE_NORM) != 0
                                     : ((flags & FDA_STATE_LINEAR) != 0 && p.have_xi);
            if (on) {
                const int b0 = p.unit_first_block[g], b1 = p.unit_first_block[g + 1];   // role 0
                for (int b = b0; b < b1; ++b) acc += p.part_np[((size_t)b * LWK + kl) * 2 + e];
            }
        } else if (sketch) {
            const int cell = e - 2;
            const int role = (cell / p.m) / p.rows_per_role;
            const int local = cell - role * p.rows_per_role * p.m;
            const int unit = role * p.groups + g;
            const int b0 = p.unit_first_block[unit], b1 = p.unit_first_block[unit + 1];
            const float *src = p.part_sk + (size_t)b0 * p.part_pitch + (size_t)local * LWK + kl;
            int b = b0;
            for (; b + 4 <= b1; b += 4) {
                const float v0 = src[0], v1 = src[p.part_pitch], v2 = src[2 * p.part_pitch], v3 = src[3 * p.part_pitch];
                acc += (double)v0; acc += (double)v1; acc += (double)v2; acc += (double)v3;
                src += 4 * p.part_pitch;
            }
            for (; b < b1; ++b, src += p.part_pitch) acc += (double)src[0];
        }
        states[(size_t)k * slen + e] = (float)acc;
    }
}

int pow2_ceil(int v) { int r = 1; while (r < v) r <<= 1; return r; }
size_t align128(size_t v) { return (v + 127) / 128 * 128; }

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            sym = nullptr;
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

// rank-2 tensor [dim1][dim0] with row pitch `pitch_bytes`, box [box1][box0], zero fill outside
bool make_map(CUtensorMap *map, CUtensorMapDataType type, const void *base, uint64_t dim0, uint64_t dim1,
              uint64_t pitch_bytes, uint32_t box0, uint32_t box1)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {dim0, dim1};
    const cuuint64_t gstride[1] = {pitch_bytes};
    const cuuint32_t box[2] = {box0, box1};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, type, 2, const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int LWK>
cudaError_t launch(fda_ctx *ctx, const StagedParams &p, const CUtensorMap *maps, bool linear, int blocks,
                   int threads, size_t smem, uint32_t flags, float *states, cudaStream_t s)
{
    // the usual sketch depths get their row loop unrolled
    auto kern = linear ? k_local_state_staged<LWK, true, 0> : k_local_state_staged<LWK, false, 0>;
    if (p.roles == 1 && p.l == 5) kern = linear ? k_local_state_staged<LWK, true, 5> : k_local_state_staged<LWK, false, 5>;
    if (p.roles == 1 && p.l == 7) kern = linear ? k_local_state_staged<LWK, true, 7> : k_local_state_staged<LWK, false, 7>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, threads, smem, s>>>(p, maps[0], maps[1], maps[2], maps[3]);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)p.groups * (2 + p.l * p.m) * LWK;
    int fb = (int)((total + 255) / 256);
    if (fb > ctx->n_sm * 8) fb = ctx->n_sm * 8;
    k_finalize_staged<LWK><<<fb, 256, 0, s>>>(p, flags, states);
    return cudaGetLastError();
}

}  // namespace

// Returns cudaErrorNotSupported when the request does not fit this path (the caller then
// uses the plain-load kernels); any other value is the result of the launches.
cudaError_t fda_launch_local_state_staged(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s)
{
    if (!(flags & FDA_STATE_SKETCH) || ctx->l == 0 || !ctx->tab32) return cudaErrorNotSupported;
    if (d + 1024 > ctx->tab32_stride) return cudaErrorNotSupported;      // the table covers smaller jobs only
    const float *xi_used = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
    const bool aligned = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) &&
                         (row_stride % 4 == 0);
    if (!aligned || !encode_fn()) return cudaErrorNotSupported;

    StagedParams p{};
    p.K = K; p.d = d; p.have_xi = xi_used != nullptr;
    p.l = ctx->l; p.m = ctx->m;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np; p.err_flag = ctx->err_flag;

    const int lwk = pow2_ceil(K < 32 ? K : 32);      // worker lanes per index slot
    p.groups = (K + lwk - 1) / lwk;
    p.Kg = (K + p.groups - 1) / p.groups;

    // Ring geometry: the widest box bx = 4 (mod 32) and the most boxes per tile that fit
    // `stages` stages beside the bins of `rows` sketch rows.
    const size_t budget = (size_t)ctx->smem_optin - 128;
    const size_t row_bins = (size_t)ctx->m * 32 * sizeof(float);
    auto stage_size = [&](int rows, int bx, int nb) -> size_t {
        return (size_t)nb * (align128((size_t)p.Kg * bx * 4) + 2 * align128((size_t)bx * 4) +
                             align128((size_t)rows * bx * 4));
    };
    // Among the (box width, boxes per tile) pairs that fit: first as many consumer warps as the
    // tile can keep busy (counted up to 28: beyond that a larger tile pays more), then the
    // largest tile.  One quad per lane and pass; box width / 4 odd keeps the box rows on
    // different banks.
    const int js_sel = 32 / lwk;
    auto warps_for = [&](int tile_indices) -> int {
        const int q = tile_indices / 4, cap = kMaxThreads / 32 - 1;
        const int passes = (q + cap * js_sel - 1) / (cap * js_sel);
        return (q + passes * js_sel - 1) / (passes * js_sel);
    };
    auto best_tile = [&](int rows, int stages, int *bx_out, int *nb_out) -> int {
        int best = 0, best_w = 0;
        if (budget <= (size_t)rows * row_bins) return 0;
        const size_t room = (budget - (size_t)rows * row_bins) / stages;
        for (int bx = 252; bx >= 36; bx -= 8)
            for (int nb = kMaxBoxes; nb >= 1; --nb) {
                if (stage_size(rows, bx, nb) > room) continue;
                const int t = bx * nb, wv = std::min(warps_for(t), 28);
                if (wv > best_w || (wv == best_w && t > best)) { best = t; best_w = wv; *bx_out = bx; *nb_out = nb; }
            }
        return best;
    };
    int rows_cap = 0, bx = 0, nb = 0;
    for (int rows = ctx->l; rows >= 1; --rows)
        if (best_tile(rows, 2, &bx, &nb) >= 64) { rows_cap = rows; break; }
    if (rows_cap == 0) return cudaErrorNotSupported;
    // Splitting the rows over several blocks was measured slower than the plain-load kernel
    // with fewer bin columns (every role re-stages the tile and amortises it over fewer rows),
    // so this path only takes sketches whose l*m bins fit with 32 columns beside the ring.
    // (measured again with 372-index tiles and two rows per role at 7 x 500, K = 60: 8.4 ms
    // against 6.9 ms.)
    if (rows_cap < ctx->l) return cudaErrorNotSupported;
    p.roles = 1;
    p.rows_per_role = ctx->l;
    p.stages = 2;      // deeper rings were measured slower (smaller tiles, same latency cover)
    const int tile = best_tile(p.rows_per_role, p.stages, &bx, &nb);
    p.bx = bx; p.nb = nb;
    p.tiles = (d + tile - 1) / tile;
    p.wbox_bytes = (uint32_t)align128((size_t)p.Kg * bx * 4);
    p.vbox_bytes = (uint32_t)align128((size_t)bx * 4);
    p.hbox_bytes = (uint32_t)align128((size_t)p.rows_per_role * bx * 4);
    const int units = p.roles * p.groups;
    if (units > kMaxUnits || units > ctx->n_sm) return cudaErrorNotSupported;

    int ncons = warps_for(tile);
    if (ncons < 4) ncons = 4;
    const int threads = (ncons + 1) * 32;

    // blocks per unit in proportion to the rows the unit scatters
    int total_rows = 0;
    for (int r = 0; r < p.roles; ++r)
        total_rows += std::min(p.rows_per_role, ctx->l - r * p.rows_per_role) * p.groups;
    int first = 0;
    for (int u = 0; u < units; ++u) {
        const int rows = std::min(p.rows_per_role, ctx->l - (u / p.groups) * p.rows_per_role);
        int64_t nblk = (int64_t)ctx->n_sm * rows / total_rows;
        if (nblk < 1) nblk = 1;
        if (nblk > p.tiles) nblk = p.tiles;
        p.unit_first_block[u] = first;
        first += (int)nblk;
    }
    p.unit_first_block[units] = first;
    const int blocks = first;
    p.part_pitch = (size_t)p.rows_per_role * ctx->m * lwk;
    if ((size_t)blocks * p.part_pitch > ctx->part_sk_floats || blocks > ctx->max_blocks)
        return cudaErrorNotSupported;

    // tensor maps: w [K][d], w_t0 / xi [1][d], hash table [l][tab_stride]; reused from the last
    // call when pointers and shapes are the same
    static_assert(sizeof(CUtensorMap) <= 128, "tensor map does not fit its cache slot");
    CUtensorMap *maps = reinterpret_cast<CUtensorMap *>(ctx->tmap_cache);
    auto &key = ctx->tmap_key;
    const void *xi_key = xi_used ? (const void *)xi_used : (const void *)w_t0;
    if (!(key.w == w && key.w_t0 == w_t0 && key.xi == xi_key && key.row_stride == row_stride && key.d == d &&
          key.K == K && key.bx == bx && key.Kg == p.Kg)) {
        key.w = nullptr;
        const uint64_t vec_pitch = (uint64_t)align128((size_t)d * 4);
        bool ok = make_map(&maps[0], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, w, (uint64_t)d, (uint64_t)K,
                           (uint64_t)row_stride * 4, (uint32_t)bx, (uint32_t)p.Kg);
        ok = ok && make_map(&maps[1], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, w_t0, (uint64_t)d, 1, vec_pitch, (uint32_t)bx, 1);
        ok = ok && make_map(&maps[2], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, xi_key, (uint64_t)d, 1, vec_pitch, (uint32_t)bx, 1);
        ok = ok && make_map(&maps[3], CU_TENSOR_MAP_DATA_TYPE_UINT32, ctx->tab32, (uint64_t)ctx->tab32_stride,
                            (uint64_t)ctx->l, (uint64_t)ctx->tab32_stride * 4, (uint32_t)bx, (uint32_t)p.rows_per_role);
        if (!ok) return cudaErrorNotSupported;
        key.w = w; key.w_t0 = w_t0; key.xi = xi_key; key.row_stride = row_stride; key.d = d;
        key.K = K; key.bx = bx; key.Kg = p.Kg;
    }

    size_t smem = 128 + (size_t)p.rows_per_role * row_bins + (size_t)p.stages * stage_size(p.rows_per_role, bx, nb);
    const size_t smem_min = 128 + (size_t)(ncons + 1) * lwk * 2 * sizeof(double);     // reduction scratch
    if (smem < smem_min) smem = smem_min;
    const bool linear = xi_used != nullptr;
    switch (lwk) {
        case 1:  return launch<1>(ctx, p, maps, linear, blocks, threads, smem, flags, states, s);
        case 2:  return launch<2>(ctx, p, maps, linear, blocks, threads, smem, flags, states, s);
        case 4:  return launch<4>(ctx, p, maps, linear, blocks, threads, smem, flags, states, s);
        case 8:  return launch<8>(ctx, p, maps, linear, blocks, threads, smem, flags, states, s);
        case 16: return launch<16>(ctx, p, maps, linear, blocks, threads, smem, flags, states, s);
        default: return launch<32>(ctx, p, maps, linear, blocks, threads, smem, flags, states, s);
    }
}
