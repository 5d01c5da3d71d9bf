// Local-state pass without the sketch: ||u^(k)||^2 and <xi,u^(k)> only (Section 3, local
// state; Section 3.2, LinearFDA).  Pure streaming: K*d + 2*d floats are read once.
//
// A block walks index tiles; w_t0 and xi of a tile are parked in shared memory once (the next
// tile's copy runs asynchronously under the current tile's row streaming) and every
// warp then streams the rows of "its" workers (k = warp, warp + NW, ...) with coalesced
// 128-bit loads, several in flight per lane.  With fewer workers than warps, several warps
// share a worker and split the tile's chunks between them.  fp32 partial sums cover one tile (at most 64
// elements per lane), the running sums are fp64; each block writes one partial per worker and
// a small second kernel adds the partials in block order.
#include "fda_internal.h"

namespace {

constexpr int kTile = 4096;           // indices per tile
constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kChunks = kTile / 128;  // 128 indices = one float4 per lane

__device__ __forceinline__ void cp_async16(float *dst_shared, const float *src)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(dst_shared);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(a), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.wait_all;" ::: "memory");
}

template <int KPW, bool LINEAR, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_local_state_linear(const float *__restrict__ w, int64_t row_stride, int K, int64_t d,
                     const float *__restrict__ w_t0, const float *__restrict__ xi, int64_t tiles,
                     double *__restrict__ part_np /* [block][K][2] */)
{
    // two buffers: the next tile's w_t0 / xi arrive while the rows of this tile stream
    extern __shared__ __align__(16) float tile_smem[];
    float (*w0buf)[kTile] = reinterpret_cast<float (*)[kTile]>(tile_smem);
    float (*xibuf)[kTile] = reinterpret_cast<float (*)[kTile]>(tile_smem + 2 * kTile);   // LINEAR only
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // K < kWarps: warp -> (worker warp % K, share warp / K of nsub); otherwise one warp per worker slot
    const int kc = K < kWarps ? K : kWarps;
    const int nsub = kWarps / kc;
    const int wslot = warp % kc, sub = warp / kc;
    const bool idle = sub >= nsub;
    double acc_n[KPW], acc_p[KPW];
#pragma unroll
    for (int kk = 0; kk < KPW; ++kk) { acc_n[kk] = 0.0; acc_p[kk] = 0.0; }

    // park w_t0 / xi of one tile (zeros past the end); asynchronous copies where aligned
    auto fill = [&](int buf, int64_t tile) {
        const int64_t j0 = tile * kTile;
        float *w0s = w0buf[buf], *xis = xibuf[buf];
        for (int i = tid * 4; i < kTile; i += kThreads * 4) {
            const int64_t j = j0 + i;
            if (VEC && j + 3 < d) {
                cp_async16(w0s + i, w_t0 + j);
                if (LINEAR) cp_async16(xis + i, xi + j);
            } else {
                float4 b = make_float4(0.f, 0.f, 0.f, 0.f), x = b;
                if (j + 0 < d) { b.x = __ldg(w_t0 + j + 0); if (LINEAR) x.x = __ldg(xi + j + 0); }
                if (j + 1 < d) { b.y = __ldg(w_t0 + j + 1); if (LINEAR) x.y = __ldg(xi + j + 1); }
                if (j + 2 < d) { b.z = __ldg(w_t0 + j + 2); if (LINEAR) x.z = __ldg(xi + j + 2); }
                if (j + 3 < d) { b.w = __ldg(w_t0 + j + 3); if (LINEAR) x.w = __ldg(xi + j + 3); }
                *reinterpret_cast<float4 *>(w0s + i) = b;
                if (LINEAR) *reinterpret_cast<float4 *>(xis + i) = x;
            }
        }
    };

    int buf = 0;
    if ((int64_t)blockIdx.x < tiles) fill(0, blockIdx.x);
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x, buf ^= 1) {
        const int64_t j0 = tile * kTile;
        cp_async_wait_all();
        __syncthreads();           // this tile's buffer is complete; the other one is no longer read
        if (tile + gridDim.x < tiles) fill(buf ^ 1, tile + gridDim.x);
        const float *w0s = w0buf[buf], *xis = xibuf[buf];
#pragma unroll
        for (int kk = 0; kk < KPW; ++kk) {
            const int k = wslot + kk * kWarps;
            if (k >= K || idle) continue;
            const float *__restrict__ wk = w + (size_t)k * (size_t)row_stride;
            float pn = 0.f, pp = 0.f;
            constexpr int B = VEC ? 8 : 2;                 // row loads in flight per lane
#pragma unroll 1
            for (int c0 = sub * B; c0 < kChunks; c0 += B * nsub) {
                float4 a[B];
#pragma unroll
                for (int c = 0; c < B; ++c) {
                    const int64_t j = j0 + (c0 + c) * 128 + lane * 4;
                    if (VEC && j + 3 < d) {
                        a[c] = __ldcs(reinterpret_cast<const float4 *>(wk + j));
                    } else {
                        // past the end u must be 0: w_t0 is 0 there, so load 0 for w as well
                        a[c].x = j + 0 < d ? __ldg(wk + j + 0) : 0.f;
                        a[c].y = j + 1 < d ? __ldg(wk + j + 1) : 0.f;
                        a[c].z = j + 2 < d ? __ldg(wk + j + 2) : 0.f;
                        a[c].w = j + 3 < d ? __ldg(wk + j + 3) : 0.f;
                    }
                }
#pragma unroll
                for (int c = 0; c < B; ++c) {
                    const int i = (c0 + c) * 128 + lane * 4;
                    const float4 b = *reinterpret_cast<const float4 *>(w0s + i);
                    const float ux = a[c].x - b.x, uy = a[c].y - b.y, uz = a[c].z - b.z, uw = a[c].w - b.w;
                    pn = fmaf(ux, ux, pn); pn = fmaf(uy, uy, pn); pn = fmaf(uz, uz, pn); pn = fmaf(uw, uw, pn);
                    if (LINEAR) {
                        const float4 x = *reinterpret_cast<const float4 *>(xis + i);
                        pp = fmaf(x.x, ux, pp); pp = fmaf(x.y, uy, pp); pp = fmaf(x.z, uz, pp); pp = fmaf(x.w, uw, pp);
                    }
                }
            }
            acc_n[kk] += (double)pn;
            if (LINEAR) acc_p[kk] += (double)pp;
        }
    }
#pragma unroll
    for (int kk = 0; kk < KPW; ++kk) {
        double n = acc_n[kk], pr = acc_p[kk];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            n += __shfl_xor_sync(0xffffffffu, n, off);
            pr += __shfl_xor_sync(0xffffffffu, pr, off);
        }
        // warps that share a worker add up through shared memory (fixed order)
        __syncthreads();
        double *red = reinterpret_cast<double *>(w0buf[0]);      // [kWarps][2]
        if (lane == 0) { red[warp * 2] = n; red[warp * 2 + 1] = pr; }
        __syncthreads();
        const int k = wslot + kk * kWarps;
        if (lane == 0 && sub == 0 && k < K) {
            double tn = 0.0, tp = 0.0;
            for (int q = 0; q < nsub; ++q) { tn += red[(wslot + q * kc) * 2]; tp += red[(wslot + q * kc) * 2 + 1]; }
            part_np[((size_t)blockIdx.x * K + k) * 2 + 0] = tn;
            part_np[((size_t)blockIdx.x * K + k) * 2 + 1] = tp;
        }
    }
}

// states[k][0..1] = sum over blocks in fp64 (one warp per value: lanes take blocks b = lane,
// lane + 32, ..., then a fixed shuffle tree, so the result is reproducible); every sketch slot
// is written as 0.
__global__ void k_finalize_linear(const double *__restrict__ part_np, int K, int blocks, int slen,
                                  uint32_t flags, bool have_xi, float *__restrict__ states)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t v = warp; v < (int64_t)K * 2; v += nwarps) {
        const int k = (int)(v / 2), e = (int)(v % 2);
        const bool on = e == 0 ? (flags & FDA_STATE_NORM) != 0 : ((flags & FDA_STATE_LINEAR) != 0 && have_xi);
        double acc = 0.0;
        if (on)
            for (int b = lane; b < blocks; b += 32) acc += part_np[((size_t)b * K + k) * 2 + e];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) states[(size_t)k * slen + e] = (float)acc;
    }
    const int64_t cells = (int64_t)K * (slen - 2);
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < cells; t += (int64_t)gridDim.x * blockDim.x)
        states[(t / (slen - 2)) * slen + 2 + t % (slen - 2)] = 0.f;
}

template <int KPW>
cudaError_t launch_kpw(int blocks, bool linear, bool vec, const float *w, int64_t row_stride, int K, int64_t d,
                       const float *w_t0, const float *xi, int64_t tiles, double *part, cudaStream_t s)
{
#define FDA_LIN(LI, VE)                                                                            \
    do {                                                                                           \
        const int smem = (LI ? 4 : 2) * kTile * (int)sizeof(float);                                \
        cudaError_t ea = cudaFuncSetAttribute(k_local_state_linear<KPW, LI, VE>,                   \
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, smem);  \
        if (ea != cudaSuccess) return ea;                                                          \
        k_local_state_linear<KPW, LI, VE><<<blocks, kThreads, smem, s>>>(w, row_stride, K, d, w_t0, \
                                                                         xi, tiles, part);         \
    } while (0)
    if (linear) { if (vec) FDA_LIN(true, true); else FDA_LIN(true, false); }
    else        { if (vec) FDA_LIN(false, true); else FDA_LIN(false, false); }
#undef FDA_LIN
    return cudaGetLastError();
}

}  // namespace

// Returns cudaErrorNotSupported for requests this kernel does not take (sketch asked for, or
// more workers than 8 per warp).
cudaError_t fda_launch_local_state_linear(fda_ctx *ctx, const float *w, int64_t row_stride, int K,
                                          int64_t d, const float *w_t0, const float *xi,
                                          uint32_t flags, float *states, cudaStream_t s)
{
    if (flags & FDA_STATE_SKETCH) return cudaErrorNotSupported;
    if (K > kWarps * 8) return cudaErrorNotSupported;
    const float *xi_used = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
    const bool vec = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)(xi_used ? xi_used : w)) & 15u) == 0) &&
                     (row_stride % 4 == 0);
    const int64_t tiles = (d + kTile - 1) / kTile;
    int64_t blocks = (int64_t)ctx->n_sm * 3;
    if (blocks > tiles) blocks = tiles;
    if (blocks > ctx->max_blocks) blocks = ctx->max_blocks;
    if ((size_t)blocks * K * 2 > ctx->part_np_doubles) return cudaErrorNotSupported;
    const int kpw = (K + kWarps - 1) / kWarps;
    const bool linear = xi_used != nullptr;
    cudaError_t e;
    if (kpw <= 1)      e = launch_kpw<1>((int)blocks, linear, vec, w, row_stride, K, d, w_t0, xi_used, tiles, ctx->part_np, s);
    else if (kpw <= 2) e = launch_kpw<2>((int)blocks, linear, vec, w, row_stride, K, d, w_t0, xi_used, tiles, ctx->part_np, s);
    else if (kpw <= 4) e = launch_kpw<4>((int)blocks, linear, vec, w, row_stride, K, d, w_t0, xi_used, tiles, ctx->part_np, s);
    else               e = launch_kpw<8>((int)blocks, linear, vec, w, row_stride, K, d, w_t0, xi_used, tiles, ctx->part_np, s);
    if (e != cudaSuccess) return e;
    const int slen = 2 + ctx->lm;
    const int64_t total = (int64_t)K * slen;
    int fb = (int)((total + 255) / 256);
    if (fb > ctx->n_sm * 8) fb = ctx->n_sm * 8;
    k_finalize_linear<<<fb, 256, 0, s>>>(ctx->part_np, K, (int)blocks, slen, flags, linear, states);
    return cudaGetLastError();
}
