// Local-state pass (Section 3: drift, ||u||^2; Section 3.1: AMS sketch; Section 3.2: <xi,u>).
//
// One streaming pass over the K x d model tensor.  A thread block serves one group of at
// most LWK workers and a strided set of index tiles.  Inside a warp the lanes are
// (index slot s, worker kl) pairs, lane = s*LWK + kl, so the LWK workers of a group at the
// same index share one hash-table entry (one broadcast load) and one w_t0 / xi value.
//
// Sketch bins live in shared memory as bins[cell][column], column = lane mod C with C a
// power of two >= LWK: every lane of a warp adds into its own bank, so a warp-wide update
// is free of bank conflicts, and the C/LWK columns that belong to one worker are summed
// when the block flushes.  Each block writes its partial sketch and its partial
// (norm, projection) sums once; a second small kernel adds the partials of all blocks in a
// fixed order in fp64 and writes the K states.
#include "fda_internal.h"

namespace {

struct LsParams {
    const float *w;
    int64_t row_stride;
    int K;
    int64_t d;
    const float *w_t0;
    const float *xi;         // may be null
    const uint16_t *tab;     // l planes
    int64_t tab_stride;
    int l, m, lm;
    int Kg;                  // workers per group (last group may hold fewer)
    int cpg;                 // blocks per group
    int cshift;              // log2(columns)
    int64_t tiles;           // index tiles of TJ indices each
    float *part_sk;          // [block][cell][LWK]
    double *part_np;         // [block][LWK][2]
};

constexpr int kQuadsPerLane = 2;   // float4 loads per lane and tile
constexpr int kFastThreads = 640;  // block size of the fast sketch kernel
constexpr int kFastQuads = 1;      // index quads per lane and tile in the fast sketch kernel (4 updates in flight)

__device__ __forceinline__ float flip(float v, uint32_t signbit)   // signbit: 0 or 0x80000000
{
    return __uint_as_float(__float_as_uint(v) ^ signbit);
}

template <int LWK, bool SKETCH, bool LINEAR, bool VEC>
__global__ void __launch_bounds__(1024, 1) k_local_state(const LsParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *bins = reinterpret_cast<float *>(smem_raw);

    constexpr int JS = 32 / LWK;                 // index slots per warp
    constexpr int TW = JS * kQuadsPerLane * 4;   // indices per warp and tile
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int kl = lane % LWK, s = lane / LWK;
    const int g = blockIdx.x / p.cpg, c = blockIdx.x % p.cpg;
    const int k = g * p.Kg + kl;
    const int kg_here = min(p.Kg, p.K - g * p.Kg);
    const bool active = kl < kg_here;
    const int columns = 1 << p.cshift;

    if (SKETCH) {
        for (int i = tid; i < p.lm * columns; i += blockDim.x) bins[i] = 0.f;
        __syncthreads();
    }

    double acc_n = 0.0, acc_p = 0.0;
    if (active) {
        const float *__restrict__ wk = p.w + (size_t)k * (size_t)p.row_stride;
        const float *__restrict__ w0 = p.w_t0;
        const float *__restrict__ xi = p.xi;
        const int col = lane & (columns - 1);
        const int64_t TJ = (int64_t)nwarps * TW;
        for (int64_t tile = c; tile < p.tiles; tile += p.cpg) {
            const int64_t base = tile * TJ + (int64_t)warp * TW;
            float u[kQuadsPerLane][4];
            float x[kQuadsPerLane][4];
            int64_t jq[kQuadsPerLane];
#pragma unroll
            for (int v = 0; v < kQuadsPerLane; ++v) {
                jq[v] = base + (int64_t)(v * JS + s) * 4;
                if (VEC && jq[v] + 3 < p.d) {
                    const float4 a = __ldg(reinterpret_cast<const float4 *>(wk + jq[v]));
                    const float4 b = __ldg(reinterpret_cast<const float4 *>(w0 + jq[v]));
                    u[v][0] = a.x - b.x; u[v][1] = a.y - b.y; u[v][2] = a.z - b.z; u[v][3] = a.w - b.w;
                    if (LINEAR) {
                        const float4 q = __ldg(reinterpret_cast<const float4 *>(xi + jq[v]));
                        x[v][0] = q.x; x[v][1] = q.y; x[v][2] = q.z; x[v][3] = q.w;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int64_t j = jq[v] + e;
                        const bool in = j < p.d;
                        u[v][e] = in ? __ldg(wk + j) - __ldg(w0 + j) : 0.f;
                        if (LINEAR) x[v][e] = in ? __ldg(xi + j) : 0.f;
                    }
                }
            }
            float pn = 0.f, pp = 0.f;
#pragma unroll
            for (int v = 0; v < kQuadsPerLane; ++v)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    pn = fmaf(u[v][e], u[v][e], pn);
                    if (LINEAR) pp = fmaf(x[v][e], u[v][e], pp);
                }
            acc_n += (double)pn;
            if (LINEAR) acc_p += (double)pp;

            if (SKETCH) {
#pragma unroll
                for (int v = 0; v < kQuadsPerLane; ++v) {
                    if (jq[v] >= p.d) continue;      // whole quad past the end: u is all zero
                    for (int i = 0; i < p.l; ++i) {
                        // 4 consecutive 16-bit entries; the table is padded past d_max
                        const uint2 h = __ldg(reinterpret_cast<const uint2 *>(
                            p.tab + (size_t)i * (size_t)p.tab_stride + jq[v]));
                        const int rowbase = i * p.m;
                        const uint32_t e0 = h.x & 0xffffu, e1 = h.x >> 16, e2 = h.y & 0xffffu, e3 = h.y >> 16;
                        atomicAdd(&bins[((rowbase + (int)(e0 & 0x7fffu)) << p.cshift) + col],
                                  flip(u[v][0], (e0 & FDA_TAB_SIGN_BIT) << 16));
                        atomicAdd(&bins[((rowbase + (int)(e1 & 0x7fffu)) << p.cshift) + col],
                                  flip(u[v][1], (e1 & FDA_TAB_SIGN_BIT) << 16));
                        atomicAdd(&bins[((rowbase + (int)(e2 & 0x7fffu)) << p.cshift) + col],
                                  flip(u[v][2], (e2 & FDA_TAB_SIGN_BIT) << 16));
                        atomicAdd(&bins[((rowbase + (int)(e3 & 0x7fffu)) << p.cshift) + col],
                                  flip(u[v][3], (e3 & FDA_TAB_SIGN_BIT) << 16));
                    }
                }
            }
        }
    }

    // ---- flush the block's sketch partial: sum the columns of each worker ----------------
    if (SKETCH) {
        __syncthreads();
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)p.lm * LWK;
        const int reps = columns / LWK;
        for (int idx = tid; idx < p.lm * LWK; idx += blockDim.x) {
            const int cell = idx / LWK, w_in = idx % LWK;
            float v = 0.f;
            for (int r = 0; r < reps; ++r) v += bins[(cell << p.cshift) + r * LWK + w_in];
            out[idx] = v;
        }
        __syncthreads();     // bins are reused below
    }

    // ---- block partial of (||u||^2, <xi,u>) per worker -----------------------------------
    // lanes with the same kl inside a warp first, then across warps through shared memory
#pragma unroll
    for (int off = LWK; off < 32; off <<= 1) {
        acc_n += __shfl_xor_sync(0xffffffffu, acc_n, off);
        acc_p += __shfl_xor_sync(0xffffffffu, acc_p, off);
    }
    double *red = reinterpret_cast<double *>(smem_raw);      // [nwarps][LWK][2]
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


// ---------------------------------------------------------------------------------------
// Fast path of the sketch pass (16-byte aligned inputs, L known at compile time).
//
// Same lane mapping and bin layout as k_local_state, but (a) every global load of a tile -
// w, w_t0, xi and the L hash-table words - is issued up front and the next tile's loads are
// in flight while the current tile is scattered, and (b) the shared-memory updates of one
// sketch row are done eight at a time: eight loads, eight adds, eight compare-and-swaps, and
// only an update whose compare-and-swap lost a race (another warp hit the same cell and
// column in between, or two of the eight share a cell) is redone with an atomic add.  The
// hardware has no native fp32 add on shared memory, so this keeps eight updates per thread
// in flight where the library atomicAdd loop keeps one.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
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

template <int L, bool LINEAR>
struct TileRegs {
    float4 a[kFastQuads], b[kFastQuads], q[kFastQuads];
    uint2 h[L][kFastQuads];
};

template <int LWK, int L, bool LINEAR>
__global__ void __launch_bounds__(kFastThreads, 1) k_local_state_fast(const LsParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *bins = reinterpret_cast<float *>(smem_raw);

    constexpr int JS = 32 / LWK;
    constexpr int TW = JS * kFastQuads * 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int kl = lane % LWK, s = lane / LWK;
    const int g = blockIdx.x / p.cpg, c = blockIdx.x % p.cpg;
    const int k = g * p.Kg + kl;
    const int kg_here = min(p.Kg, p.K - g * p.Kg);
    const bool active = kl < kg_here;
    const int columns = 1 << p.cshift;

    for (int i = tid; i < p.lm * columns; i += blockDim.x) bins[i] = 0.f;
    __syncthreads();

    double acc_n = 0.0, acc_p = 0.0;
    if (active) {
        const float *__restrict__ wk = p.w + (size_t)k * (size_t)p.row_stride;
        const float *__restrict__ w0 = p.w_t0;
        const float *__restrict__ xi = p.xi;
        const uint16_t *__restrict__ tab = p.tab;
        const int64_t TJ = (int64_t)nwarps * TW;
        const int64_t lane_off = (int64_t)warp * TW + (int64_t)s * 4;
        const uint32_t col_addr = (uint32_t)__cvta_generic_to_shared(bins) + (uint32_t)(lane & (columns - 1)) * 4u;
        const uint32_t row_bytes = (uint32_t)p.m << (p.cshift + 2);
        const int bshift = p.cshift + 2;

        auto load_tile = [&](TileRegs<L, LINEAR> &r, int64_t tile) {
#pragma unroll
            for (int v = 0; v < kFastQuads; ++v) {
                const int64_t jq = tile * TJ + lane_off + (int64_t)v * (JS * 4);
                if (jq + 3 < p.d) {
                    r.a[v] = __ldg(reinterpret_cast<const float4 *>(wk + jq));
                    r.b[v] = __ldg(reinterpret_cast<const float4 *>(w0 + jq));
                    if (LINEAR) r.q[v] = __ldg(reinterpret_cast<const float4 *>(xi + jq));
#pragma unroll
                    for (int i = 0; i < L; ++i)
                        r.h[i][v] = __ldg(reinterpret_cast<const uint2 *>(tab + (size_t)i * (size_t)p.tab_stride + jq));
                } else {
                    // ragged end: scalar, bounds-checked; indices past d contribute u = 0 to cell 0
                    float a[4], b[4], q[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const bool in = jq + e < p.d;
                        a[e] = in ? __ldg(wk + jq + e) : 0.f;
                        b[e] = in ? __ldg(w0 + jq + e) : 0.f;
                        q[e] = (LINEAR && in) ? __ldg(xi + jq + e) : 0.f;
                    }
                    r.a[v] = make_float4(a[0], a[1], a[2], a[3]);
                    r.b[v] = make_float4(b[0], b[1], b[2], b[3]);
                    if (LINEAR) r.q[v] = make_float4(q[0], q[1], q[2], q[3]);
#pragma unroll
                    for (int i = 0; i < L; ++i)
                        r.h[i][v] = (jq < p.d)
                            ? __ldg(reinterpret_cast<const uint2 *>(tab + (size_t)i * (size_t)p.tab_stride + jq))
                            : make_uint2(0u, 0u);
                }
            }
        };

        TileRegs<L, LINEAR> cur, nxt;
        int64_t tile = c;
        if (tile < p.tiles) load_tile(cur, tile);
        for (; tile < p.tiles; tile += p.cpg) {
            const bool more = tile + p.cpg < p.tiles;
            if (more) load_tile(nxt, tile + p.cpg);

            float u[kFastQuads * 4];
            float pn = 0.f, pp = 0.f;
#pragma unroll
            for (int v = 0; v < kFastQuads; ++v) {
                u[4 * v + 0] = cur.a[v].x - cur.b[v].x; u[4 * v + 1] = cur.a[v].y - cur.b[v].y;
                u[4 * v + 2] = cur.a[v].z - cur.b[v].z; u[4 * v + 3] = cur.a[v].w - cur.b[v].w;
                if (LINEAR) {
                    pp = fmaf(cur.q[v].x, u[4 * v + 0], pp); pp = fmaf(cur.q[v].y, u[4 * v + 1], pp);
                    pp = fmaf(cur.q[v].z, u[4 * v + 2], pp); pp = fmaf(cur.q[v].w, u[4 * v + 3], pp);
                }
            }
#pragma unroll
            for (int e = 0; e < kFastQuads * 4; ++e) pn = fmaf(u[e], u[e], pn);
            acc_n += (double)pn;
            if (LINEAR) acc_p += (double)pp;

#pragma unroll
            for (int i = 0; i < L; ++i) {
                constexpr int NB = kFastQuads * 4;
                uint32_t addr[NB];
                float val[NB], old[NB];
                const uint32_t rowaddr = col_addr + (uint32_t)i * row_bytes;
#pragma unroll
                for (int v = 0; v < kFastQuads; ++v) {
                    const uint32_t hx = cur.h[i][v].x, hy = cur.h[i][v].y;
                    addr[4 * v + 0] = rowaddr + ((hx & 0x7fffu) << bshift);
                    addr[4 * v + 1] = rowaddr + (((hx >> 16) & 0x7fffu) << bshift);
                    addr[4 * v + 2] = rowaddr + ((hy & 0x7fffu) << bshift);
                    addr[4 * v + 3] = rowaddr + (((hy >> 16) & 0x7fffu) << bshift);
                    val[4 * v + 0] = flip(u[4 * v + 0], (hx << 16) & 0x80000000u);
                    val[4 * v + 1] = flip(u[4 * v + 1], hx & 0x80000000u);
                    val[4 * v + 2] = flip(u[4 * v + 2], (hy << 16) & 0x80000000u);
                    val[4 * v + 3] = flip(u[4 * v + 3], hy & 0x80000000u);
                }
#pragma unroll
                for (int e = 0; e < NB; ++e) old[e] = lds_f32(addr[e]);
                uint32_t got[NB];
#pragma unroll
                for (int e = 0; e < NB; ++e)
                    got[e] = cas_shared(addr[e], __float_as_uint(old[e]), __float_as_uint(old[e] + val[e]));
#pragma unroll
                for (int e = 0; e < NB; ++e)
                    if (got[e] != __float_as_uint(old[e])) red_shared_add(addr[e], val[e]);
            }
            if (more) cur = nxt;
        }
    }

    __syncthreads();
    {
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)p.lm * LWK;
        const int reps = columns / LWK;
        for (int idx = tid; idx < p.lm * LWK; idx += blockDim.x) {
            const int cell = idx / LWK, w_in = idx % LWK;
            float v = 0.f;
            for (int r = 0; r < reps; ++r) v += bins[(cell << p.cshift) + r * LWK + w_in];
            out[idx] = v;
        }
        __syncthreads();
    }
#pragma unroll
    for (int off = LWK; off < 32; off <<= 1) {
        acc_n += __shfl_xor_sync(0xffffffffu, acc_n, off);
        acc_p += __shfl_xor_sync(0xffffffffu, acc_p, off);
    }
    double *red = reinterpret_cast<double *>(smem_raw);
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

// states[k][.] = sum over the blocks of worker k's group, in block order, in fp64.
// Threads run over (group, cell, worker-in-group) with the worker fastest, which is the order
// of the partial buffers, so the reads of every block's partial are contiguous.
template <int LWK>
__global__ void k_finalize_states(const float *__restrict__ part_sk, const double *__restrict__ part_np,
                                  int K, int Kg, int groups, int cpg, int lm, uint32_t flags,
                                  bool have_xi, float *__restrict__ states)
{
    const int slen = 2 + lm;
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    const int64_t per_group = (int64_t)(lm + 2) * LWK;
    const int64_t total = per_group * groups;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(t / per_group);
        const int r = (int)(t % per_group);
        const int e = r / LWK, kl = r % LWK;       // e: 0 norm, 1 projection, 2.. sketch cells
        const int k = g * Kg + kl;
        if (kl >= Kg || k >= K) continue;
        double acc = 0.0;
        if (e < 2) {
            const bool on = (e == 0) ? (flags & FDA_STATE_NORM) != 0
                                     : ((flags & FDA_STATE_LINEAR) != 0 && have_xi);
            if (on)
                for (int b = 0; b < cpg; ++b)
                    acc += part_np[((size_t)(g * cpg + b) * LWK + kl) * 2 + e];
        } else if (sketch) {
            const float *src = part_sk + ((size_t)g * cpg * lm + (e - 2)) * LWK + kl;
            const size_t step = (size_t)lm * LWK;
            int b = 0;
            for (; b + 4 <= cpg; b += 4) {          // four loads in flight, added in block order
                const float v0 = src[(size_t)b * step], v1 = src[(size_t)(b + 1) * step];
                const float v2 = src[(size_t)(b + 2) * step], v3 = src[(size_t)(b + 3) * step];
                acc += (double)v0; acc += (double)v1; acc += (double)v2; acc += (double)v3;
            }
            for (; b < cpg; ++b) acc += (double)src[(size_t)b * step];
        }
        states[(size_t)k * slen + e] = (float)acc;
    }
}

int ilog2(int v) { int r = 0; while ((1 << (r + 1)) <= v) ++r; return r; }
int pow2_ceil(int v) { int r = 1; while (r < v) r <<= 1; return r; }

template <int LWK, int L>
cudaError_t launch_fast(fda_ctx *ctx, const LsParams &p, bool linear, int blocks, size_t smem,
                        cudaStream_t s)
{
    auto kern = linear ? k_local_state_fast<LWK, L, true> : k_local_state_fast<LWK, L, false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, kFastThreads, smem, s>>>(p);
    return cudaGetLastError();
}

template <int LWK>
cudaError_t launch_for_lwk(fda_ctx *ctx, LsParams &p, uint32_t flags, bool vec, bool fast, int groups,
                           int blocks, int threads, size_t smem, float *states, cudaStream_t s)
{
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    const bool linear = (flags & FDA_STATE_LINEAR) != 0 && p.xi != nullptr;
    if (fast) {
        if constexpr (LWK >= 8) {
            cudaError_t e = p.l == 5 ? launch_fast<LWK, 5>(ctx, p, linear, blocks, smem, s)
                                     : launch_fast<LWK, 7>(ctx, p, linear, blocks, smem, s);
            if (e != cudaSuccess) return e;
        } else {
            return cudaErrorInvalidValue;     // the fast path is never selected for fewer than 8 worker lanes
        }
    } else {
#define FDA_LS_LAUNCH(SK, LI, VE)                                                              \
    do {                                                                                       \
        auto kern = k_local_state<LWK, SK, LI, VE>;                                            \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                             ctx->smem_optin);                                 \
        if (e != cudaSuccess) return e;                                                        \
        kern<<<blocks, threads, smem, s>>>(p);                                                 \
    } while (0)
    if (sketch) {
        if (linear) { if (vec) FDA_LS_LAUNCH(true, true, true); else FDA_LS_LAUNCH(true, true, false); }
        else        { if (vec) FDA_LS_LAUNCH(true, false, true); else FDA_LS_LAUNCH(true, false, false); }
    } else {
        if (linear) { if (vec) FDA_LS_LAUNCH(false, true, true); else FDA_LS_LAUNCH(false, true, false); }
        else        { if (vec) FDA_LS_LAUNCH(false, false, true); else FDA_LS_LAUNCH(false, false, false); }
    }
#undef FDA_LS_LAUNCH
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)groups * (2 + p.lm) * LWK;
    int fb = (int)((total + 255) / 256);
    if (fb > ctx->n_sm * 8) fb = ctx->n_sm * 8;
    k_finalize_states<LWK><<<fb, 256, 0, s>>>(p.part_sk, p.part_np, p.K, p.Kg, groups, p.cpg, p.lm, flags,
                                             p.xi != nullptr, states);
    return cudaGetLastError();
}

}  // namespace

cudaError_t fda_setup_local_state(fda_ctx *ctx)
{
    // columns: the largest power of two (<= 32) of lane-private copies of the l*m bins that
    // fits the opt-in shared memory.
    if (ctx->l == 0) { ctx->columns = 0; return cudaSuccess; }
    const size_t per_col = (size_t)ctx->lm * sizeof(float);
    int cap = (int)((size_t)ctx->smem_optin / per_col);
    if (cap < 1) { ctx->columns = 0; return cudaSuccess; }       // caller reports UNSUPPORTED
    ctx->columns = cap >= 32 ? 32 : (1 << ilog2(cap));
    return cudaSuccess;
}

cudaError_t fda_launch_local_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                   int64_t d, const float *w_t0, const float *xi, uint32_t flags,
                                   float *states, cudaStream_t s)
{
    {   // sketch requests: the list kernel when the context holds its schedule; requests without a
        // sketch: the streaming kernel; everything else: the plain-load kernels below
        cudaError_t e = fda_launch_local_state_gather(ctx, w, row_stride, K, d, w_t0, xi, flags, states, s);
        if (e != cudaErrorNotSupported) { ctx->last_ls_kernel = "k_local_state_gather"; return e; }   // (counts its launches itself)
        e = fda_launch_local_state_linear(ctx, w, row_stride, K, d, w_t0, xi, flags, states, s);
        if (e != cudaErrorNotSupported) { ctx->last_ls_kernel = "k_local_state_linear"; ctx->last_ls_launches = 2; return e; }
    }
    if (flags & FDA_STATE_SKETCH) {
        const cudaError_t e = fda_ensure_table(ctx, s);
        if (e != cudaSuccess) return e;
    }
    ctx->last_ls_kernel = "k_local_state";
    ctx->last_ls_launches = 2;
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    LsParams p{};
    p.w = w; p.row_stride = row_stride; p.K = K; p.d = d; p.w_t0 = w_t0;
    p.xi = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
    p.tab = ctx->tab; p.tab_stride = ctx->tab_stride;
    p.l = ctx->l; p.m = ctx->m; p.lm = ctx->lm;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np;

    // workers per group: a power of two lane count LWK, limited by the bin columns
    const int lane_cap = sketch ? ctx->columns : 32;
    int lwk = pow2_ceil(K < 32 ? K : 32);
    if (lwk > lane_cap) lwk = lane_cap;
    if (lwk < 8) lwk = 8 <= lane_cap ? 8 : lane_cap;
    const int groups = (K + lwk - 1) / lwk;
    p.Kg = (K + groups - 1) / groups;
    const int columns = sketch ? ctx->columns : lwk;
    p.cshift = ilog2(columns);

    const bool vec = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(p.xi ? p.xi : w)) & 15u) == 0) &&
                     (row_stride % 4 == 0);
    const bool fast = sketch && vec && lwk >= 8 && (ctx->l == 5 || ctx->l == 7);
    const int threads = fast ? kFastThreads : (sketch ? 1024 : 512);
    const int blocks_per_sm = sketch ? 1 : 2;
    const int js = 32 / lwk;
    const int64_t tile_j = (int64_t)(threads / 32) * js * (fast ? kFastQuads : kQuadsPerLane) * 4;
    p.tiles = (d + tile_j - 1) / tile_j;
    int64_t cpg = (int64_t)ctx->n_sm * blocks_per_sm / groups;
    if (cpg < 1) cpg = 1;
    if (cpg > p.tiles) cpg = p.tiles;
    if ((int64_t)groups * cpg > ctx->max_blocks) cpg = ctx->max_blocks / groups;
    p.cpg = (int)cpg;
    const int blocks = groups * p.cpg;
    // the partial sums of a launch must fit the context's scratch (sized for n_sm blocks of 32
    // worker lanes and 4 * n_sm blocks of K_max workers): more worker groups than that is refused
    if (blocks < 1 || (sketch && (size_t)blocks * p.lm * lwk > ctx->part_sk_floats) ||
        (size_t)blocks * lwk * 2 > ctx->part_np_doubles)
        return cudaErrorNotSupported;
    ctx->last_ls_kernel = fast ? "k_local_state_fast" : "k_local_state";

    size_t smem = (size_t)(threads / 32) * lwk * 2 * sizeof(double);
    if (sketch) {
        const size_t b = (size_t)p.lm * columns * sizeof(float);
        if (b > smem) smem = b;
    }
    switch (lwk) {
        case 1:  return launch_for_lwk<1>(ctx, p, flags, vec, fast, groups, blocks, threads, smem, states, s);
        case 2:  return launch_for_lwk<2>(ctx, p, flags, vec, fast, groups, blocks, threads, smem, states, s);
        case 4:  return launch_for_lwk<4>(ctx, p, flags, vec, fast, groups, blocks, threads, smem, states, s);
        case 8:  return launch_for_lwk<8>(ctx, p, flags, vec, fast, groups, blocks, threads, smem, states, s);
        case 16: return launch_for_lwk<16>(ctx, p, flags, vec, fast, groups, blocks, threads, smem, states, s);
        default: return launch_for_lwk<32>(ctx, p, flags, vec, fast, groups, blocks, threads, smem, states, s);
    }
}
