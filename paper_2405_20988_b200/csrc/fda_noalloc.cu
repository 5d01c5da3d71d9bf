// fda_local_state_linear_noalloc: the sketch-free local state for callers that may not
// allocate.  Same arithmetic as the streaming kernel in fda_local_state_linear.cu, but the
// per-block partial sums live in a fixed array that is part of the library image, so the
// call needs no context and never calls cudaMalloc / cudaFree.
#include <mutex>

#include "fda_internal.h"

#define FDA_NOALLOC_MAX_BLOCKS 1024

namespace {

constexpr int kTile = 2048;
constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kChunks = kTile / 128;
constexpr int kKpw = FDA_NOALLOC_MAX_WORKERS / kWarps;      // worker slots per warp

// [block][K][2] partial sums.  Lives on every device that loads the library, until exit
// (FDA_NOALLOC_MAX_BLOCKS * FDA_NOALLOC_MAX_WORKERS * 16 bytes = 1 MiB).  In host code this
// name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) double g_noalloc_partials[FDA_NOALLOC_MAX_BLOCKS * FDA_NOALLOC_MAX_WORKERS * 2];

__global__ void __launch_bounds__(kThreads)
k_noalloc_local_state(const float *__restrict__ w, int64_t row_stride, int K, int64_t d,
                      const float *__restrict__ w_t0, const float *__restrict__ xi, int64_t tiles,
                      double *__restrict__ part /* device address of g_noalloc_partials */)
{
    __shared__ float w0s[kTile];
    __shared__ float xis[kTile];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double acc_n[kKpw], acc_p[kKpw];
#pragma unroll
    for (int kk = 0; kk < kKpw; ++kk) { acc_n[kk] = 0.0; acc_p[kk] = 0.0; }

    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int64_t j0 = tile * kTile;
        __syncthreads();
        for (int i = tid; i < kTile; i += kThreads) {          // scalar loads: any alignment
            const int64_t j = j0 + i;
            w0s[i] = j < d ? __ldg(w_t0 + j) : 0.f;
            xis[i] = (xi != nullptr && j < d) ? __ldg(xi + j) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kKpw; ++kk) {
            const int k = warp + kk * kWarps;
            if (k >= K) continue;
            const float *__restrict__ wk = w + (size_t)k * (size_t)row_stride;
            float pn = 0.f, pp = 0.f;
#pragma unroll 4
            for (int c = 0; c < kChunks * 4; ++c) {            // 32 consecutive indices per step
                const int i = c * 32 + lane;
                const int64_t j = j0 + i;
                const float u = (j < d ? __ldg(wk + j) : 0.f) - w0s[i];
                pn = fmaf(u, u, pn);
                pp = fmaf(xis[i], u, pp);
            }
            acc_n[kk] += (double)pn;
            acc_p[kk] += (double)pp;
        }
    }
#pragma unroll
    for (int kk = 0; kk < kKpw; ++kk) {
        double n = acc_n[kk], pr = acc_p[kk];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            n += __shfl_xor_sync(0xffffffffu, n, off);
            pr += __shfl_xor_sync(0xffffffffu, pr, off);
        }
        const int k = warp + kk * kWarps;
        if (lane == 0 && k < K) {              // every slot that the second kernel reads is written here
            part[((size_t)blockIdx.x * K + k) * 2 + 0] = n;
            part[((size_t)blockIdx.x * K + k) * 2 + 1] = pr;
        }
    }
}

__global__ void k_noalloc_finalize(const double *__restrict__ part, int K, int blocks, uint32_t flags,
                                   bool have_xi, float *__restrict__ states /* K x 2 */)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= K * 2) return;
    const int k = t / 2, e = t % 2;
    const bool on = e == 0 ? (flags & FDA_STATE_NORM) != 0 : ((flags & FDA_STATE_LINEAR) != 0 && have_xi);
    double acc = 0.0;
    if (on)
        for (int b = 0; b < blocks; ++b) acc += part[((size_t)b * K + k) * 2 + e];
    states[t] = (float)acc;
}

struct DeviceSetup {
    bool ready = false;
    double *partials = nullptr;     // device address of g_noalloc_partials on this device
    int n_sm = 0;
};
constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

}  // namespace

extern "C" fda_status fda_local_state_linear_noalloc(int device, const float *w, int64_t row_stride, int K,
                                                     int64_t d, const float *w_t0, const float *xi,
                                                     uint32_t flags, float *states, void *stream)
{
    if (!w || !w_t0 || !states) return FDA_ERR_INVALID_ARG;
    if (K < 1 || d < 1 || row_stride < d || device < 0 || device >= kMaxDevices) return FDA_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(FDA_STATE_NORM | FDA_STATE_LINEAR)) return FDA_ERR_INVALID_ARG;
    if (K > FDA_NOALLOC_MAX_WORKERS) return FDA_ERR_UNSUPPORTED;      // beyond the fixed scratch

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) { cudaGetLastError(); return FDA_ERR_CUDA; }
    if (device >= ndev) return FDA_ERR_INVALID_ARG;                   // no such device
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return FDA_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return FDA_ERR_CUDA; }
    fda_status st = FDA_OK;
    DeviceSetup setup;
    {
        // first call on this device: resolve the device address of the scratch array (the
        // device is current here); no memory is allocated by this
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        DeviceSetup &slot = g_setup[device];
        if (!slot.ready) {
            void *ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_partials);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&slot.n_sm, cudaDevAttrMultiProcessorCount, device);
            if (e != cudaSuccess || ptr == nullptr) { cudaGetLastError(); st = FDA_ERR_CUDA; }
            else { slot.partials = static_cast<double *>(ptr); slot.ready = true; }
        }
        setup = slot;
    }
    if (st == FDA_OK) {
        const int64_t tiles = (d + kTile - 1) / kTile;
        int64_t blocks = (int64_t)setup.n_sm * 3;
        if (blocks > tiles) blocks = tiles;
        if (blocks > FDA_NOALLOC_MAX_BLOCKS) blocks = FDA_NOALLOC_MAX_BLOCKS;
        cudaStream_t s = (cudaStream_t)stream;
        const float *xi_used = (flags & FDA_STATE_LINEAR) ? xi : nullptr;
        k_noalloc_local_state<<<(unsigned)blocks, kThreads, 0, s>>>(w, row_stride, K, d, w_t0, xi_used, tiles,
                                                                   setup.partials);
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess) {
            k_noalloc_finalize<<<(K * 2 + 127) / 128, 128, 0, s>>>(setup.partials, K, (int)blocks, flags,
                                                                  xi_used != nullptr, states);
            e = cudaGetLastError();
        }
        if (e != cudaSuccess) st = FDA_ERR_CUDA;
    }
    if (prev != device) cudaSetDevice(prev);
    return st;
}
