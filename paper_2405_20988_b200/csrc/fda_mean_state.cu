// Averaged state in one pass: S-bar = (mean_k ||u^(k)||^2, mean_k <xi,u^(k)>, sk(u-bar)).
//
// The sketch is linear (Section 3.1, property (a)), so the average of the K worker sketches
// that Algorithm 1 obtains with AllReduce equals the sketch of the average drift
// u-bar = (1/K) sum_k u^(k); the proof of Theorem 1 uses exactly this step.  When all K
// workers sit in one GPU's memory the per-worker sketches need not exist: summing the K
// drifts of an index in registers first leaves l shared-memory updates per index instead of
// K*l, which takes the pass from the shared-memory update ceiling to the HBM roofline.
// The result feeds fda_combine_estimate with K = 1 (a state that is already averaged).
//
// Lanes take consecutive index quads (coalesced 128-bit loads, 8 rows in flight), the bins
// are bins[cell][C] with column = lane mod C, updated eight at a time with compare-and-swap
// and an atomic-add retry for lost races, as in the per-worker pass.
#include <algorithm>

#include "fda_internal.h"

namespace {

constexpr int kThreads = 768;
constexpr int kBatch = 8;          // worker rows loaded before they are consumed

__device__ __forceinline__ float flip(float v, uint32_t signbit)
{
    return __uint_as_float(__float_as_uint(v) ^ signbit);
}
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

struct MeanParams {
    const float *w;
    int64_t row_stride;
    int K;
    int64_t d;
    const float *w_t0;
    const float *xi;
    const uint16_t *tab;
    int64_t tab_stride;
    int l, m, lm;
    int cshift;              // log2(columns)
    int64_t tiles;           // tiles of kThreads*8 indices
    float *part_sk;          // [block][cell]
    double *part_np;         // [block][2]
};

template <bool SKETCH, bool LINEAR, bool VEC>
__global__ void __launch_bounds__(kThreads, 1) k_mean_state(const MeanParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *bins = reinterpret_cast<float *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int columns = 1 << p.cshift;
    if (SKETCH) {
        for (int i = tid; i < p.lm * columns; i += blockDim.x) bins[i] = 0.f;
        __syncthreads();
    }
    const uint32_t col_addr = (uint32_t)__cvta_generic_to_shared(bins) + (uint32_t)(lane & (columns - 1)) * 4u;
    const int bshift = p.cshift + 2;
    const uint32_t row_bytes = (uint32_t)p.m << bshift;
    const float inv_k = 1.0f / (float)p.K;
    double acc_n = 0.0, acc_p = 0.0;

    for (int64_t tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        float s[8];                      // sum over workers of the drift, two quads
        int64_t jq[2];
        float pn = 0.f, pp = 0.f;
#pragma unroll
        for (int v = 0; v < 2; ++v) {
            jq[v] = (tile * 2 + v) * (int64_t)(kThreads * 4) + (int64_t)tid * 4;
            float b[4] = {0.f, 0.f, 0.f, 0.f}, x[4] = {0.f, 0.f, 0.f, 0.f};
            const bool full = VEC && jq[v] + 3 < p.d;
            if (full) {
                const float4 t = __ldg(reinterpret_cast<const float4 *>(p.w_t0 + jq[v]));
                b[0] = t.x; b[1] = t.y; b[2] = t.z; b[3] = t.w;
                if (LINEAR) {
                    const float4 q = __ldg(reinterpret_cast<const float4 *>(p.xi + jq[v]));
                    x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (jq[v] + e < p.d) { b[e] = __ldg(p.w_t0 + jq[v] + e); if (LINEAR) x[e] = __ldg(p.xi + jq[v] + e); }
            }
            float sv[4] = {0.f, 0.f, 0.f, 0.f};
            for (int k0 = 0; k0 < p.K; k0 += kBatch) {
                float a[kBatch][4];
#pragma unroll
                for (int t = 0; t < kBatch; ++t) {
                    const int k = k0 + t;
                    if (k < p.K) {
                        const float *wk = p.w + (size_t)k * (size_t)p.row_stride + jq[v];
                        if (full) {
                            const float4 q = __ldcs(reinterpret_cast<const float4 *>(wk));
                            a[t][0] = q.x; a[t][1] = q.y; a[t][2] = q.z; a[t][3] = q.w;
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) a[t][e] = jq[v] + e < p.d ? __ldg(wk + e) : 0.f;
                        }
                    }
                }
#pragma unroll
                for (int t = 0; t < kBatch; ++t)
                    if (k0 + t < p.K) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float u = a[t][e] - b[e];
                            pn = fmaf(u, u, pn);
                            sv[e] += u;
                        }
                    }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (LINEAR) pp = fmaf(x[e], sv[e], pp);
                s[4 * v + e] = sv[e] * inv_k;                  // u-bar at this index
            }
        }
        acc_n += (double)pn;
        if (LINEAR) acc_p += (double)pp;

        if (SKETCH) {
            for (int i = 0; i < p.l; ++i) {
                uint32_t addr[8];
                float val[8], old[8];
                const uint32_t rowaddr = col_addr + (uint32_t)i * row_bytes;
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    uint2 h = make_uint2(0u, 0u);              // indices past d: u-bar = 0 goes to cell 0
                    if (jq[v] < p.d)
                        h = __ldg(reinterpret_cast<const uint2 *>(p.tab + (size_t)i * (size_t)p.tab_stride + jq[v]));
                    addr[4 * v + 0] = rowaddr + ((h.x & 0x7fffu) << bshift);
                    addr[4 * v + 1] = rowaddr + (((h.x >> 16) & 0x7fffu) << bshift);
                    addr[4 * v + 2] = rowaddr + ((h.y & 0x7fffu) << bshift);
                    addr[4 * v + 3] = rowaddr + (((h.y >> 16) & 0x7fffu) << bshift);
                    val[4 * v + 0] = flip(s[4 * v + 0], (h.x << 16) & 0x80000000u);
                    val[4 * v + 1] = flip(s[4 * v + 1], h.x & 0x80000000u);
                    val[4 * v + 2] = flip(s[4 * v + 2], (h.y << 16) & 0x80000000u);
                    val[4 * v + 3] = flip(s[4 * v + 3], h.y & 0x80000000u);
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) old[e] = lds_f32(addr[e]);
                uint32_t lost = 0;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint32_t got = cas_shared(addr[e], __float_as_uint(old[e]), __float_as_uint(old[e] + val[e]));
                    lost |= (got != __float_as_uint(old[e])) ? (1u << e) : 0u;
                }
                while (lost) {
                    uint32_t a = addr[0];
                    float v = val[0];
#pragma unroll
                    for (int e = 1; e < 8; ++e)
                        if ((lost & ((1u << e) - 1u)) == 0 && (lost & (1u << e))) { a = addr[e]; v = val[e]; }
                    red_shared_add(a, v);
                    lost &= lost - 1u;
                }
            }
        }
    }

    if (SKETCH) {
        __syncthreads();
        float *out = p.part_sk + (size_t)blockIdx.x * (size_t)p.lm;
        for (int cell = tid; cell < p.lm; cell += blockDim.x) {
            float v = 0.f;
            for (int c = 0; c < columns; ++c) v += bins[(cell << p.cshift) + ((c + tid) & (columns - 1))];
            out[cell] = v;
        }
        __syncthreads();
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc_n += __shfl_xor_sync(0xffffffffu, acc_n, off);
        acc_p += __shfl_xor_sync(0xffffffffu, acc_p, off);
    }
    double *red = reinterpret_cast<double *>(smem_raw);
    if (lane == 0) { red[warp * 2] = acc_n; red[warp * 2 + 1] = acc_p; }
    __syncthreads();
    if (tid < 2) {
        double t = 0.0;
        for (int wv = 0; wv < nwarps; ++wv) t += red[wv * 2 + tid];
        p.part_np[(size_t)blockIdx.x * 2 + tid] = t;
    }
}

// mean_state[e] = (sum over blocks, block order, fp64) [/ K for the two scalars]
__global__ void k_finalize_mean(const float *__restrict__ part_sk, const double *__restrict__ part_np, int blocks,
                                int lm, int K, uint32_t flags, bool have_xi, float *__restrict__ mean_state)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= 2 + lm) return;
    double acc = 0.0;
    if (e < 2) {
        const bool on = e == 0 ? (flags & FDA_STATE_NORM) != 0 : ((flags & FDA_STATE_LINEAR) != 0 && have_xi);
        if (on) {
            for (int b = 0; b < blocks; ++b) acc += part_np[(size_t)b * 2 + e];
            acc /= (double)K;
        }
    } else if (flags & FDA_STATE_SKETCH) {
        for (int b = 0; b < blocks; ++b) acc += (double)part_sk[(size_t)b * lm + (e - 2)];
    }
    mean_state[e] = (float)acc;
}

int ilog2(int v) { int r = 0; while ((1 << (r + 1)) <= v) ++r; return r; }

}  // namespace

cudaError_t fda_launch_mean_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                                  const float *w_t0, const float *xi, uint32_t flags, float *mean_state,
                                  cudaStream_t s)
{
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    MeanParams p{};
    p.w = w; p.row_stride = row_stride; p.K = K; p.d = d; p.w_t0 = w_t0;
    p.xi = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
    p.tab = ctx->tab; p.tab_stride = ctx->tab_stride;
    p.l = ctx->l; p.m = ctx->m; p.lm = ctx->lm;
    p.cshift = sketch ? ilog2(ctx->columns) : 0;
    p.part_sk = ctx->part_sk; p.part_np = ctx->part_np;
    const int64_t per_tile = (int64_t)kThreads * 8;
    p.tiles = (d + per_tile - 1) / per_tile;
    int64_t blocks = sketch ? ctx->n_sm : (int64_t)ctx->n_sm * 2;
    if (blocks > p.tiles) blocks = p.tiles;
    size_t smem = (size_t)(kThreads / 32) * 2 * sizeof(double);
    if (sketch) smem = std::max(smem, (size_t)ctx->lm * ctx->columns * sizeof(float));
    const bool vec = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(p.xi ? p.xi : w)) & 15u) == 0) &&
                     (row_stride % 4 == 0);
    const bool linear = p.xi != nullptr;
#define FDA_MEAN(SK, LI, VE)                                                                             \
    do {                                                                                                 \
        auto kern = k_mean_state<SK, LI, VE>;                                                            \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin); \
        if (e != cudaSuccess) return e;                                                                  \
        kern<<<(unsigned)blocks, kThreads, smem, s>>>(p);                                                \
    } while (0)
    if (sketch) {
        if (linear) { if (vec) FDA_MEAN(true, true, true); else FDA_MEAN(true, true, false); }
        else        { if (vec) FDA_MEAN(true, false, true); else FDA_MEAN(true, false, false); }
    } else {
        if (linear) { if (vec) FDA_MEAN(false, true, true); else FDA_MEAN(false, true, false); }
        else        { if (vec) FDA_MEAN(false, false, true); else FDA_MEAN(false, false, false); }
    }
#undef FDA_MEAN
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int n = 2 + ctx->lm;
    k_finalize_mean<<<(n + 255) / 256, 256, 0, s>>>(ctx->part_sk, ctx->part_np, (int)blocks, ctx->lm, K, flags,
                                                   linear, mean_state);
    return cudaGetLastError();
}
