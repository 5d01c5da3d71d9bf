// Bare read-only probe: streams a float array once and returns its sum.  It measures what a
// kernel that does nothing but read reaches on this device, the yardstick beside the
// bandwidth-bound kernels of the path.  The method itself has no such step.
#include "fda_internal.h"

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeBatch = 8;

__global__ void __launch_bounds__(kProbeThreads)
k_read_probe(const float *__restrict__ src, int64_t n, double *__restrict__ part)
{
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    // peel to a 16-byte boundary, then float4 loads, then the tail
    const int64_t head = min(n, (int64_t)((16 - ((uintptr_t)src & 15)) & 15) / 4);
    const int64_t nq = (n - head) / 4;
    const float4 *q = reinterpret_cast<const float4 *>(src + head);
    float acc = 0.f;
    // each block reads one contiguous run of kProbeBatch * blockDim float4 per iteration
    const int64_t run = (int64_t)kProbeBatch * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * run; base < nq; base += (int64_t)gridDim.x * run) {
        float4 v[kProbeBatch];
#pragma unroll
        for (int b = 0; b < kProbeBatch; ++b) {
            const int64_t i = base + (int64_t)b * blockDim.x + threadIdx.x;
            v[b] = (i < nq) ? __ldcs(q + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int b = 0; b < kProbeBatch; ++b) acc += (v[b].x + v[b].y) + (v[b].z + v[b].w);
    }
    for (int64_t j = t0; j < head; j += nthreads) acc += src[j];
    for (int64_t j = head + nq * 4 + t0; j < n; j += nthreads) acc += src[j];
    double a = (double)acc;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) a += __shfl_down_sync(0xffffffffu, a, off);
    __shared__ double red[kProbeThreads / 32];
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < kProbeThreads / 32; ++w) s += red[w];
        part[blockIdx.x] = s;
    }
}

__global__ void k_read_probe_finalize(const double *__restrict__ part, int nblocks, float *__restrict__ out)
{
    double s = 0.0;
    for (int b = threadIdx.x; b < nblocks; b += 32) s += part[b];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xffffffffu, s, off);
    if (threadIdx.x == 0) *out = (float)s;
}

}  // namespace

cudaError_t fda_launch_read_probe(const fda_ctx *ctx, const float *src, int64_t n, float *sum_out, cudaStream_t s)
{
    int blocks = ctx->n_sm * 8;
    if ((size_t)blocks > ctx->part_np_doubles) blocks = (int)ctx->part_np_doubles;
    k_read_probe<<<blocks, kProbeThreads, 0, s>>>(src, n, ctx->part_np);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_read_probe_finalize<<<1, 32, 0, s>>>(ctx->part_np, blocks, sum_out);
    return cudaGetLastError();
}
