// Averaged state without per-worker sketches:
//   S-bar = (mean_k ||u^(k)||^2, mean_k <xi,u^(k)>, sk(u-bar)).
//
// The sketch is linear (Section 3.1, property (a)), so the average of the K worker sketches
// that Algorithm 1 obtains with AllReduce equals the sketch of the average drift
// u-bar = (1/K) sum_k u^(k); the proof of Theorem 1 uses exactly this step.  When all K
// workers sit in one GPU's memory the per-worker sketches need not exist: l shared-memory
// updates per index instead of K*l.  The result feeds fda_combine_estimate with K = 1 (a
// state that is already averaged).
//
// Two kernels.  k_mean_model streams the K rows once at HBM speed (many loads in flight, no
// shared memory): it writes the average drift u-bar to context scratch (summing the K drifts
// of an index, not the K models, keeps the fp32 rounding relative to the drift) and
// accumulates the two scalars.  Then u-bar, one vector, is sketched.  Measured on B200: a
// warp-wide shared-memory atomic whose 32 lanes fall into 32 different 128-byte rows runs at
// ~1.1 updates/clk/SM against 6.8 when they share a row, so the per-worker trick (all lanes on
// one cell) has no analogue for a single vector.  k_sketch_vector_rows therefore uses no
// atomics: warp r owns sketch row r and the 32 lane-private columns of its bins outright,
// streams the whole vector itself (the other warps' loads of the same bytes hit L1) and
// updates with plain load-add-store, four indices per lane at a time; equal cells among the
// four are folded so that every store to such a cell carries the whole sum.  k_sketch_vector (compare-and-swap on bins[cell][C]) is
// kept for sketches whose bins do not fit with 32 columns.
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
    asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
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

constexpr int kModelThreads = 256;

// ubar[j] = (1/K) sum_k (w_k[j] - w_t0[j]);  partial sums of sum_k ||u_k||^2 and sum_k <xi,u_k>
template <bool LINEAR, bool VEC>
__global__ void __launch_bounds__(kModelThreads)
k_mean_model(const float *__restrict__ w, int64_t row_stride, int K, int64_t d, const float *__restrict__ w_t0,
             const float *__restrict__ xi, float *__restrict__ ubar, double *__restrict__ part_np)
{
    const float inv_k = 1.0f / (float)K;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    double acc_n = 0.0, acc_p = 0.0;
    if (VEC) {
        const int64_t nq = d / 4;
        for (int64_t q = t0; q < nq; q += nthreads) {
            const float4 b = __ldg(reinterpret_cast<const float4 *>(w_t0 + q * 4));
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (LINEAR) x = __ldg(reinterpret_cast<const float4 *>(xi + q * 4));
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            float pn = 0.f;
            for (int k0 = 0; k0 < K; k0 += kBatch) {
                float4 a[kBatch];
#pragma unroll
                for (int t = 0; t < kBatch; ++t)
                    if (k0 + t < K)
                        a[t] = __ldcs(reinterpret_cast<const float4 *>(w + (size_t)(k0 + t) * row_stride + q * 4));
#pragma unroll
                for (int t = 0; t < kBatch; ++t)
                    if (k0 + t < K) {
                        const float ux = a[t].x - b.x, uy = a[t].y - b.y, uz = a[t].z - b.z, uw = a[t].w - b.w;
                        pn = fmaf(ux, ux, pn); pn = fmaf(uy, uy, pn); pn = fmaf(uz, uz, pn); pn = fmaf(uw, uw, pn);
                        sum.x += ux; sum.y += uy; sum.z += uz; sum.w += uw;
                    }
            }
            acc_n += (double)pn;
            if (LINEAR)   // sum_k <xi,u_k> = <xi, sum_k u_k>
                acc_p += (double)(x.x * sum.x + x.y * sum.y + x.z * sum.z + x.w * sum.w);
            *reinterpret_cast<float4 *>(ubar + q * 4) = make_float4(sum.x * inv_k, sum.y * inv_k, sum.z * inv_k, sum.w * inv_k);
        }
    }
    const int64_t begin = VEC ? (d / 4) * 4 : 0;
    for (int64_t j = begin + t0; j < d; j += nthreads) {
        const float b = __ldg(w_t0 + j);
        float sum = 0.f, pn = 0.f;
        for (int k = 0; k < K; ++k) {
            const float a = __ldg(w + (size_t)k * row_stride + j);
            pn = fmaf(a - b, a - b, pn);
            sum += a - b;
        }
        acc_n += (double)pn;
        if (LINEAR) acc_p += (double)(__ldg(xi + j) * sum);
        ubar[j] = sum * inv_k;
    }
    // block partial (fixed order)
    __shared__ double red[kModelThreads / 32][2];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc_n += __shfl_xor_sync(0xffffffffu, acc_n, off);
        acc_p += __shfl_xor_sync(0xffffffffu, acc_p, off);
    }
    if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5][0] = acc_n; red[threadIdx.x >> 5][1] = acc_p; }
    __syncthreads();
    if (threadIdx.x < 2) {
        double t = 0.0;
        for (int wv = 0; wv < kModelThreads / 32; ++wv) t += red[wv][threadIdx.x];
        part_np[(size_t)blockIdx.x * 2 + threadIdx.x] = t;
    }
}

struct SketchVecParams {
    const float *v;          // the vector that is sketched (u-bar, 16-byte aligned context scratch)
    int64_t d;
    const uint16_t *tab;
    int64_t tab_stride;
    int l, m, lm;
    int cshift;              // log2(columns)
    int64_t tiles;           // tiles of kThreads*8 indices
    float *part_sk;          // [block][cell]
};

// L > 0: number of sketch rows known at compile time (table words kept in registers);
// L == 0: any number of rows, table words loaded row by row.
template <int L>
__global__ void __launch_bounds__(kThreads, 1) k_sketch_vector(const SketchVecParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *bins = reinterpret_cast<float *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31;
    const int columns = 1 << p.cshift;
    for (int i = tid; i < p.lm * columns; i += blockDim.x) bins[i] = 0.f;
    __syncthreads();
    const uint32_t col_addr = (uint32_t)__cvta_generic_to_shared(bins) + (uint32_t)(lane & (columns - 1)) * 4u;
    const int bshift = p.cshift + 2;
    const uint32_t row_bytes = (uint32_t)p.m << bshift;
    constexpr int LR = L > 0 ? L : 1;

    for (int64_t tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        // a lane takes 8 consecutive indices: two 16-byte loads of the vector, one per table row
        float u[8];
        uint4 h[LR];
        const int64_t j8 = tile * (int64_t)(kThreads * 8) + (int64_t)tid * 8;
        if (j8 + 7 < p.d) {
            const float4 a = __ldcs(reinterpret_cast<const float4 *>(p.v + j8));
            const float4 b = __ldcs(reinterpret_cast<const float4 *>(p.v + j8 + 4));
            u[0] = a.x; u[1] = a.y; u[2] = a.z; u[3] = a.w; u[4] = b.x; u[5] = b.y; u[6] = b.z; u[7] = b.w;
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) u[e] = j8 + e < p.d ? __ldg(p.v + j8 + e) : 0.f;
        }
        // the table planes are padded to a multiple of 64 entries past d_max: whole 16-byte reads stay inside
        const bool any = j8 < p.d;
        if (L > 0) {
#pragma unroll
            for (int i = 0; i < LR; ++i)
                h[i] = any ? __ldg(reinterpret_cast<const uint4 *>(p.tab + (size_t)i * (size_t)p.tab_stride + j8))
                           : make_uint4(0u, 0u, 0u, 0u);
        }
        const int rows = L > 0 ? L : p.l;
#pragma unroll
        for (int i = 0; i < rows; ++i) {
            uint32_t addr[8], got[8];
            float val[8], old[8];
            const uint32_t rowaddr = col_addr + (uint32_t)i * row_bytes;
            uint4 hw;
            if (L > 0) hw = h[L > 0 ? i : 0];
            else hw = any ? __ldg(reinterpret_cast<const uint4 *>(p.tab + (size_t)i * (size_t)p.tab_stride + j8))
                          : make_uint4(0u, 0u, 0u, 0u);          // indices past d: u = 0 goes to cell 0
            const uint32_t hv[4] = {hw.x, hw.y, hw.z, hw.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                addr[2 * q + 0] = rowaddr + ((hv[q] & 0x7fffu) << bshift);
                addr[2 * q + 1] = rowaddr + (((hv[q] >> 16) & 0x7fffu) << bshift);
                val[2 * q + 0] = flip(u[2 * q + 0], (hv[q] << 16) & 0x80000000u);
                val[2 * q + 1] = flip(u[2 * q + 1], hv[q] & 0x80000000u);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) old[e] = lds_f32(addr[e]);
            uint32_t diff = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                got[e] = cas_shared(addr[e], __float_as_uint(old[e]), __float_as_uint(old[e] + val[e]));
                diff |= got[e] ^ __float_as_uint(old[e]);
            }
            if (diff) {
                uint32_t lost = 0;
#pragma unroll
                for (int e = 0; e < 8; ++e) lost |= (got[e] != __float_as_uint(old[e])) ? (1u << e) : 0u;
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
    __syncthreads();
    float *out = p.part_sk + (size_t)blockIdx.x * (size_t)p.lm;
    for (int cell = tid; cell < p.lm; cell += blockDim.x) {
        float v = 0.f;
        for (int c = 0; c < columns; ++c) v += bins[(cell << p.cshift) + ((c + tid) & (columns - 1))];
        out[cell] = v;
    }
}

// One warp per sketch row, plain read-modify-write on bins[row][cell][32] (column = lane).
// Lanes own their column and the warp owns the row, so no other thread touches a lane's cells.
__global__ void __launch_bounds__(32 * FDA_MAX_ROWS, 1) k_sketch_vector_rows(const SketchVecParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *bins = reinterpret_cast<float *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, row = tid >> 5;      // blockDim = 32 * l
    for (int i = tid; i < p.lm * 32; i += blockDim.x) bins[i] = 0.f;
    __syncthreads();
    const uint32_t rowaddr = (uint32_t)__cvta_generic_to_shared(bins) + (uint32_t)row * ((uint32_t)p.m << 7) +
                             (uint32_t)lane * 4u;
    const uint16_t *__restrict__ plane = p.tab + (size_t)row * (size_t)p.tab_stride;
    constexpr int kStep = 128;                       // indices per warp step: 4 per lane
    const int64_t steps = (p.d + kStep - 1) / kStep;

    auto load = [&](int64_t st, float4 &a, uint2 &h) {
        const int64_t j = st * kStep + lane * 4;
        a = make_float4(0.f, 0.f, 0.f, 0.f);
        h = make_uint2(0u, 0u);                      // past d: u = 0 goes to cell 0
        if (j + 3 < p.d) a = __ldg(reinterpret_cast<const float4 *>(p.v + j));
        else {
            if (j + 0 < p.d) a.x = __ldg(p.v + j + 0);
            if (j + 1 < p.d) a.y = __ldg(p.v + j + 1);
            if (j + 2 < p.d) a.z = __ldg(p.v + j + 2);
        }
        if (j < p.d) h = __ldg(reinterpret_cast<const uint2 *>(plane + j));      // plane padded past d_max
    };

    auto update = [&](const float4 &a, const uint2 &h) {
        const uint32_t a0 = rowaddr + ((h.x & 0x7fffu) << 7), a1 = rowaddr + (((h.x >> 16) & 0x7fffu) << 7);
        const uint32_t a2 = rowaddr + ((h.y & 0x7fffu) << 7), a3 = rowaddr + (((h.y >> 16) & 0x7fffu) << 7);
        const float v0 = flip(a.x, (h.x << 16) & 0x80000000u), v1 = flip(a.y, h.x & 0x80000000u);
        const float v2 = flip(a.z, (h.y << 16) & 0x80000000u), v3 = flip(a.w, h.y & 0x80000000u);
        const float o0 = lds_f32(a0), o1 = lds_f32(a1), o2 = lds_f32(a2), o3 = lds_f32(a3);
        // equal cells among the four: the four loads above are issued before the four stores below,
        // so two updates of one cell would both start from the old value and one would be lost
        // whatever the order of the stores; every store to such a cell carries the sum of all of them
        const bool e01 = a0 == a1, e02 = a0 == a2, e03 = a0 == a3, e12 = a1 == a2, e13 = a1 == a3, e23 = a2 == a3;
        const float t0 = v0 + (e01 ? v1 : 0.f) + (e02 ? v2 : 0.f) + (e03 ? v3 : 0.f);
        const float t1 = v1 + (e01 ? v0 : 0.f) + (e12 ? v2 : 0.f) + (e13 ? v3 : 0.f);
        const float t2 = v2 + (e02 ? v0 : 0.f) + (e12 ? v1 : 0.f) + (e23 ? v3 : 0.f);
        const float t3 = v3 + (e03 ? v0 : 0.f) + (e13 ? v1 : 0.f) + (e23 ? v2 : 0.f);
        asm volatile("st.volatile.shared.f32 [%0], %1;" ::"r"(a0), "f"(o0 + t0) : "memory");
        asm volatile("st.volatile.shared.f32 [%0], %1;" ::"r"(a1), "f"(o1 + t1) : "memory");
        asm volatile("st.volatile.shared.f32 [%0], %1;" ::"r"(a2), "f"(o2 + t2) : "memory");
        asm volatile("st.volatile.shared.f32 [%0], %1;" ::"r"(a3), "f"(o3 + t3) : "memory");
    };

    // groups of kGroup steps: the loads of the next group are in flight while this one is applied
    constexpr int kGroup = 8;
    float4 a[kGroup], an[kGroup];
    uint2 h[kGroup], hn[kGroup];
    const int64_t groups = (steps + kGroup - 1) / kGroup;
    int64_t g = blockIdx.x;
    if (g < groups) {
#pragma unroll
        for (int t = 0; t < kGroup; ++t) load(g * kGroup + t, a[t], h[t]);       // steps past the end load nothing
    }
    for (; g < groups; g += gridDim.x) {
        const int64_t gn = g + gridDim.x;
        if (gn < groups) {
#pragma unroll
            for (int t = 0; t < kGroup; ++t) load(gn * kGroup + t, an[t], hn[t]);
        }
#pragma unroll
        for (int t = 0; t < kGroup; ++t) update(a[t], h[t]);
#pragma unroll
        for (int t = 0; t < kGroup; ++t) { a[t] = an[t]; h[t] = hn[t]; }
    }
    __syncthreads();
    float *out = p.part_sk + (size_t)blockIdx.x * (size_t)p.lm;
    for (int cell = tid; cell < p.lm; cell += blockDim.x) {
        float v = 0.f;
        for (int c = 0; c < 32; ++c) v += bins[cell * 32 + ((c + tid) & 31)];
        out[cell] = v;
    }
}

// mean_state[e] = sum over blocks in fp64 [/ K for the two scalars].  Warp 0 and 1 of block 0
// reduce the scalar partials (lanes stride the blocks, fixed shuffle tree); the cells are summed
// in block order by one thread each.
__global__ void k_finalize_mean(const float *__restrict__ part_sk, const double *__restrict__ part_np,
                                int np_blocks, int sk_blocks, int lm, int K, uint32_t flags, bool have_xi,
                                float *__restrict__ mean_state)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && warp < 2) {
        const int e = warp;
        const bool on = e == 0 ? (flags & FDA_STATE_NORM) != 0 : ((flags & FDA_STATE_LINEAR) != 0 && have_xi);
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
    if (flags & FDA_STATE_SKETCH)
        for (int b = 0; b < sk_blocks; ++b) acc += (double)part_sk[(size_t)b * lm + cell];
    mean_state[2 + cell] = (float)acc;
}

int ilog2(int v) { int r = 0; while ((1 << (r + 1)) <= v) ++r; return r; }

template <int L>
cudaError_t launch_sketch_vector(fda_ctx *ctx, const SketchVecParams &p, int blocks, size_t smem, cudaStream_t s)
{
    auto kern = k_sketch_vector<L>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin);
    if (e != cudaSuccess) return e;
    kern<<<blocks, kThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t fda_launch_mean_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                                  const float *w_t0, const float *xi, uint32_t flags, float *mean_state,
                                  cudaStream_t s)
{
    const bool sketch = (flags & FDA_STATE_SKETCH) != 0;
    const float *xi_used = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
    // With a list schedule in the context the cells can come from the list kernel.  In one pass over
    // the K rows when there are few of them and the vector is long: 1.50 against 2.58 ms at 5 x 250,
    // K = 8, d = 198M, but no gain at d = 7M, where the averaged drifts and the 16-bit table of the
    // two-kernel route stay in L2.  From the averaged drifts that phase 1 below leaves in memory when
    // the sketch is too large for the lane-private bins of k_sketch_vector_rows: 0.93 against 1.42 ms
    // at 7 x 500, K = 60, d = 20M (at 5 x 250 that kernel is the faster one: 0.22 against 0.25 ms at
    // K = 30, d = 7M).
    const bool lists = sketch && ctx->sched != nullptr;
    const int64_t tiles = lists ? (d + ctx->sched_T - 1) / ctx->sched_T : 0;
    if (lists && K <= 2 * ctx->l && tiles >= 8 * (int64_t)ctx->n_sm) {
        const cudaError_t e = fda_launch_mean_state_gather(ctx, w, row_stride, K, d, w_t0, xi, flags, mean_state, s);
        if (e != cudaErrorNotSupported) {
            if (e == cudaSuccess) ctx->last_ls_kernel = "k_mean_state_gather";
            return e;
        }
    }
    if (!ctx->mean_model) {      // first use: d_max floats of scratch for the average drift
        cudaError_t e = cudaMalloc(&ctx->mean_model, sizeof(float) * (size_t)((ctx->d_max + 3) / 4 * 4));
        if (e != cudaSuccess) return e;
    }
    // phase 1: one pass over the K rows
    const bool vec = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) &&
                     (row_stride % 4 == 0);
    const bool linear = xi_used != nullptr;
    int64_t work = vec ? (d + 3) / 4 : d;
    int64_t nblk = (work + kModelThreads - 1) / kModelThreads;
    if (nblk > (int64_t)ctx->n_sm * 8) nblk = (int64_t)ctx->n_sm * 8;
    if (nblk > ctx->max_blocks * 2) nblk = ctx->max_blocks * 2;      // part_np holds >= max_blocks*64 doubles
    if (linear) {
        if (vec) k_mean_model<true, true><<<(unsigned)nblk, kModelThreads, 0, s>>>(w, row_stride, K, d, w_t0, xi_used, ctx->mean_model, ctx->part_np);
        else     k_mean_model<true, false><<<(unsigned)nblk, kModelThreads, 0, s>>>(w, row_stride, K, d, w_t0, xi_used, ctx->mean_model, ctx->part_np);
    } else {
        if (vec) k_mean_model<false, true><<<(unsigned)nblk, kModelThreads, 0, s>>>(w, row_stride, K, d, w_t0, xi_used, ctx->mean_model, ctx->part_np);
        else     k_mean_model<false, false><<<(unsigned)nblk, kModelThreads, 0, s>>>(w, row_stride, K, d, w_t0, xi_used, ctx->mean_model, ctx->part_np);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    // phase 2: sketch of u-bar
    if (lists && ctx->columns != 32) {
        e = fda_launch_mean_sketch_gather(ctx, ctx->mean_model, K, d, linear, flags, (int)nblk, mean_state, s);
        if (e != cudaErrorNotSupported) {
            if (e == cudaSuccess) ctx->last_ls_kernel = "k_mean_model + k_mean_state_gather";
            return e;
        }
    }
    ctx->last_ls_kernel = sketch ? "k_mean_model + k_sketch_vector" : "k_mean_model";
    int sk_blocks = 0;
    if (sketch) {
        e = fda_ensure_table(ctx, s);        // first use: the 16-bit hash table
        if (e != cudaSuccess) return e;
        SketchVecParams p{};
        p.v = ctx->mean_model; p.d = d; p.tab = ctx->tab; p.tab_stride = ctx->tab_stride;
        p.l = ctx->l; p.m = ctx->m; p.lm = ctx->lm; p.cshift = ilog2(ctx->columns); p.part_sk = ctx->part_sk;
        const int64_t per_tile = (int64_t)kThreads * 8;
        p.tiles = (d + per_tile - 1) / per_tile;
        int64_t blocks = ctx->n_sm;
        if (blocks > p.tiles) blocks = p.tiles;
        sk_blocks = (int)blocks;
        const size_t smem = (size_t)ctx->lm * ctx->columns * sizeof(float);
        if (ctx->columns == 32) {
            const int64_t ngroups = (d + 1023) / 1024;            // 8 steps of 128 indices
            int64_t rb = (int64_t)ctx->n_sm;
            if (rb > ngroups) rb = ngroups;
            sk_blocks = (int)rb;
            e = cudaFuncSetAttribute(k_sketch_vector_rows, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin);
            if (e != cudaSuccess) return e;
            k_sketch_vector_rows<<<sk_blocks, 32 * ctx->l, smem, s>>>(p);
            e = cudaGetLastError();
        } else
        switch (ctx->l) {
            case 1: e = launch_sketch_vector<1>(ctx, p, sk_blocks, smem, s); break;
            case 2: e = launch_sketch_vector<2>(ctx, p, sk_blocks, smem, s); break;
            case 3: e = launch_sketch_vector<3>(ctx, p, sk_blocks, smem, s); break;
            case 4: e = launch_sketch_vector<4>(ctx, p, sk_blocks, smem, s); break;
            case 5: e = launch_sketch_vector<5>(ctx, p, sk_blocks, smem, s); break;
            case 6: e = launch_sketch_vector<6>(ctx, p, sk_blocks, smem, s); break;
            case 7: e = launch_sketch_vector<7>(ctx, p, sk_blocks, smem, s); break;
            default: e = launch_sketch_vector<0>(ctx, p, sk_blocks, smem, s); break;
        }
        if (e != cudaSuccess) return e;
    }
    const int n = ctx->lm > 64 ? ctx->lm : 64;        // at least two warps for the scalars
    k_finalize_mean<<<(n + 255) / 256, 256, 0, s>>>(ctx->part_sk, ctx->part_np, (int)nblk, sk_blocks, ctx->lm, K,
                                                   flags, linear, mean_state);
    return cudaGetLastError();
}
