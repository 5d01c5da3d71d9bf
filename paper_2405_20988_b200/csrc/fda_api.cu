// C ABI of libfda: context management, argument validation, stream plumbing.
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "fda_internal.h"

namespace {

constexpr uint64_t kP61 = (1ull << 61) - 1;

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

fda_status fail(fda_ctx *ctx, fda_status st, const char *what)
{
    if (ctx) ctx->err = what;
    return st;
}

fda_status fail_cuda(fda_ctx *ctx, cudaError_t e, const char *where)
{
    if (ctx) {
        ctx->err = std::string(where) + ": " + cudaGetErrorString(e);
    }
    if (e == cudaErrorNotSupported) return FDA_ERR_UNSUPPORTED;      // a launcher refused the shape
    return e == cudaErrorMemoryAllocation ? FDA_ERR_NOMEM : FDA_ERR_CUDA;
}

void free_device(fda_ctx *ctx)
{
    cudaFree(ctx->coeffs_dev);
    cudaFree(ctx->tab);
    cudaFree(ctx->sched);
    cudaFree(ctx->sched_off);
    cudaFree(ctx->part_sk);
    cudaFree(ctx->part_np);
    cudaFree(ctx->combine_scratch);
    cudaFree(ctx->combine_ticket);
    cudaFree(ctx->mean_model);
    cudaFree(ctx->stage_w);
    cudaFree(ctx->stage_w_t0);
    cudaFree(ctx->stage_xi);
    cudaFree(ctx->stage_states);
    cudaFree(ctx->stage_est);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
}

bool finite_f(float v) { return std::isfinite(v); }

}  // namespace

extern "C" {

fda_status fda_create(fda_ctx **out, int device, int l, int m, const uint64_t *hash_coeffs,
                      int64_t d_max, int K_max)
{
    return fda_create_limited(out, device, l, m, hash_coeffs, d_max, K_max, 0);
}

fda_status fda_create_limited(fda_ctx **out, int device, int l, int m, const uint64_t *hash_coeffs,
                              int64_t d_max, int K_max, int64_t schedule_limit_bytes)
{
    if (!out) return FDA_ERR_INVALID_ARG;
    *out = nullptr;
    if (l < 0 || l > FDA_MAX_ROWS) return FDA_ERR_INVALID_ARG;
    if (l > 0 && (m < 1 || m > 32768 || !hash_coeffs)) return FDA_ERR_INVALID_ARG;
    if (d_max < 1 || d_max >= (int64_t)1 << 31 || K_max < 1) return FDA_ERR_INVALID_ARG;
    for (int i = 0; i < 6 * l; ++i) {
        if (hash_coeffs[i] >= kP61) return FDA_ERR_INVALID_ARG;
        if ((i % 6 == 0 || i % 6 == 2) && hash_coeffs[i] == 0) return FDA_ERR_INVALID_ARG;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        cudaGetLastError();
        return FDA_ERR_CUDA;
    }
    fda_ctx *ctx = new (std::nothrow) fda_ctx();
    if (!ctx) return FDA_ERR_NOMEM;
    ctx->device = device;
    ctx->l = l;
    ctx->m = l > 0 ? m : 0;
    ctx->lm = ctx->l * ctx->m;
    ctx->d_max = d_max;
    ctx->K_max = K_max;
    for (int i = 0; i < 6 * l; ++i) ctx->coeffs_host[i] = hash_coeffs[i];

    DeviceGuard guard(device);
    cudaError_t e = guard.ok ? cudaSuccess : cudaErrorInvalidDevice;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&ctx->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) { delete ctx; return FDA_ERR_CUDA; }

    fda_setup_local_state(ctx);
    if (l > 0 && ctx->columns < 1) { delete ctx; return FDA_ERR_UNSUPPORTED; }

    ctx->max_blocks = ctx->n_sm * 4;
    ctx->sched_limit_bytes = schedule_limit_bytes;
    // padded by more than the widest tile of the plain-load kernels, so that a tile that starts below
    // d_max never reads past the table (entries past d_max are valid hashes of those indices)
    ctx->tab_stride = (d_max + 1024 + 63) / 64 * 64;
    ctx->part_sk_floats = l > 0 ? (size_t)ctx->n_sm * ctx->lm * 32 : 0;
    if (l > 0) {
        e = cudaMalloc(&ctx->coeffs_dev, sizeof(uint64_t) * 6 * l);
        if (e == cudaSuccess)
            e = cudaMemcpy(ctx->coeffs_dev, ctx->coeffs_host, sizeof(uint64_t) * 6 * l, cudaMemcpyHostToDevice);
        if (e == cudaSuccess && schedule_limit_bytes >= 0) {
            const auto t0 = std::chrono::steady_clock::now();
            e = fda_build_list_schedule(ctx, nullptr);
            ctx->sched_build_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
        }
        if (e == cudaSuccess) e = cudaMalloc(&ctx->part_sk, sizeof(float) * ctx->part_sk_floats);
        if (e == cudaSuccess && ctx->sched) {
            e = cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
        }
    }
    ctx->part_np_doubles = (size_t)ctx->max_blocks * (size_t)(K_max > 32 ? K_max : 32) * 2;
    if (e == cudaSuccess) e = cudaMalloc(&ctx->part_np, sizeof(double) * ctx->part_np_doubles);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->combine_scratch, sizeof(double) * (2 + FDA_MAX_ROWS));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->combine_ticket, sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(ctx->combine_ticket, 0, sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        const fda_status st = e == cudaErrorMemoryAllocation ? FDA_ERR_NOMEM : FDA_ERR_CUDA;
        cudaGetLastError();
        free_device(ctx);
        delete ctx;
        return st;
    }
    *out = ctx;
    return FDA_OK;
}

fda_status fda_destroy(fda_ctx *ctx)
{
    if (!ctx) return FDA_OK;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    free_device(ctx);
    delete ctx;
    return FDA_OK;
}

size_t fda_state_len(const fda_ctx *ctx) { return ctx ? 2 + (size_t)ctx->lm : 0; }

const char *fda_last_error(const fda_ctx *ctx) { return ctx ? ctx->err.c_str() : ""; }

const char *fda_debug_last_kernel(const fda_ctx *ctx) { return ctx ? ctx->last_ls_kernel : ""; }

int fda_debug_last_launches(const fda_ctx *ctx) { return ctx ? ctx->last_ls_launches : 0; }

fda_status fda_local_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                           const float *w_t0, const float *xi, uint32_t flags, float *states,
                           void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!w || !w_t0 || !states) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_local_state: null pointer");
    if (K < 1 || K > ctx->K_max) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_local_state: K out of range");
    if (d < 1 || d > ctx->d_max) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_local_state: d out of range");
    if (row_stride < d) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_local_state: row_stride < d");
    if (flags & ~(uint32_t)(FDA_STATE_NORM | FDA_STATE_LINEAR | FDA_STATE_SKETCH))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_local_state: unknown flag");
    if ((flags & FDA_STATE_SKETCH) && ctx->l == 0)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_local_state: context has no sketch");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_local_state: cannot select device");
    cudaError_t e = fda_launch_local_state(ctx, w, row_stride, K, d, w_t0, xi, flags, states,
                                           (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_local_state");
    return FDA_OK;
}

fda_status fda_mean_state(fda_ctx *ctx, const float *w, int64_t row_stride, int K, int64_t d,
                          const float *w_t0, const float *xi, uint32_t flags, float *mean_state,
                          void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!w || !w_t0 || !mean_state) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_mean_state: null pointer");
    if (K < 1 || K > ctx->K_max) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_mean_state: K out of range");
    if (d < 1 || d > ctx->d_max) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_mean_state: d out of range");
    if (row_stride < d) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_mean_state: row_stride < d");
    if (flags & ~(uint32_t)(FDA_STATE_NORM | FDA_STATE_LINEAR | FDA_STATE_SKETCH))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_mean_state: unknown flag");
    if ((flags & FDA_STATE_SKETCH) && ctx->l == 0)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_mean_state: context has no sketch");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_mean_state: cannot select device");
    cudaError_t e = fda_launch_mean_state(ctx, w, row_stride, K, d, w_t0, xi, flags, mean_state,
                                          (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_mean_state");
    return FDA_OK;
}

fda_status fda_combine_estimate(fda_ctx *ctx, const float *states, int K, int variant,
                                float epsilon, float theta, fda_estimate *est_dev,
                                fda_estimate *est_host, void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!states || !est_dev) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_combine_estimate: null pointer");
    if (K < 1 || K > ctx->K_max) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_combine_estimate: K out of range");
    if (variant != FDA_VARIANT_LINEAR && variant != FDA_VARIANT_SKETCH)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_combine_estimate: bad variant");
    if (variant == FDA_VARIANT_SKETCH && ctx->l == 0)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_combine_estimate: context has no sketch");
    if (!finite_f(epsilon) || epsilon <= -1.0f || !finite_f(theta))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_combine_estimate: epsilon or theta out of range");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_combine_estimate: cannot select device");
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = fda_launch_combine(ctx, states, K, variant, epsilon, theta, est_dev, s);
    if (e == cudaSuccess && est_host) {
        e = cudaMemcpyAsync(est_host, est_dev, sizeof(fda_estimate), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    }
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_combine_estimate");
    return FDA_OK;
}

fda_status fda_average_models(fda_ctx *ctx, float *w, int64_t row_stride, int K, int64_t d,
                              float *w_t0, const fda_estimate *est_dev, uint32_t flags,
                              void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!w || !w_t0) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_average_models: null pointer");
    if (K < 1 || d < 1 || row_stride < d)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_average_models: size out of range");
    if (flags & ~(uint32_t)(FDA_AVG_BROADCAST | FDA_AVG_UNCONDITIONAL))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_average_models: unknown flag");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_average_models: cannot select device");
    cudaError_t e = fda_launch_average(ctx, w, row_stride, K, d, w_t0, nullptr, est_dev, flags,
                                       (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_average_models");
    return FDA_OK;
}

fda_status fda_average_models_xi(fda_ctx *ctx, float *w, int64_t row_stride, int K, int64_t d,
                                 float *w_t0, float *xi_out, const fda_estimate *est_dev,
                                 uint32_t flags, void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!w || !w_t0 || !xi_out) return fail(ctx, FDA_ERR_INVALID_ARG, "fda_average_models_xi: null pointer");
    if (K < 1 || d < 1 || row_stride < d)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_average_models_xi: size out of range");
    if (flags & ~(uint32_t)(FDA_AVG_BROADCAST | FDA_AVG_UNCONDITIONAL))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_average_models_xi: unknown flag");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_average_models_xi: cannot select device");
    cudaError_t e = fda_launch_average(ctx, w, row_stride, K, d, w_t0, xi_out, est_dev, flags,
                                       (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_average_models_xi");
    return FDA_OK;
}

fda_status fda_round_host(fda_ctx *ctx, float *w_host, int64_t row_stride, int K, int64_t d,
                          float *w_t0_host, const float *xi_host, uint32_t state_flags,
                          int variant, float epsilon, float theta, uint32_t avg_flags,
                          float *states_host, fda_estimate *est_host, void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!w_host || !w_t0_host || !est_host)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_round_host: null pointer");
    if (K < 1 || K > ctx->K_max || d < 1 || d > ctx->d_max || row_stride < d)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_round_host: size out of range");
    if (avg_flags & ~(uint32_t)(FDA_AVG_BROADCAST | FDA_AVG_UNCONDITIONAL))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_round_host: unknown flag");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_round_host: cannot select device");
    cudaStream_t s = (cudaStream_t)stream;
    const size_t slen = fda_state_len(ctx);
    cudaError_t e = cudaSuccess;
    if (!ctx->stage_w) {
        ctx->stage_stride = (ctx->d_max + 31) / 32 * 32;
        e = cudaMalloc(&ctx->stage_w, sizeof(float) * (size_t)ctx->K_max * ctx->stage_stride);
        if (e == cudaSuccess) e = cudaMalloc(&ctx->stage_w_t0, sizeof(float) * ctx->stage_stride);
        if (e == cudaSuccess) e = cudaMalloc(&ctx->stage_xi, sizeof(float) * ctx->stage_stride);
        if (e == cudaSuccess) e = cudaMalloc(&ctx->stage_states, sizeof(float) * (size_t)ctx->K_max * slen);
        if (e == cudaSuccess) e = cudaMalloc(&ctx->stage_est, sizeof(fda_estimate));
        if (e != cudaSuccess) {
            cudaFree(ctx->stage_w); cudaFree(ctx->stage_w_t0); cudaFree(ctx->stage_xi);
            cudaFree(ctx->stage_states); cudaFree(ctx->stage_est);
            ctx->stage_w = ctx->stage_w_t0 = ctx->stage_xi = ctx->stage_states = nullptr;
            ctx->stage_est = nullptr;
            cudaGetLastError();
            return fail_cuda(ctx, e, "fda_round_host: staging allocation");
        }
    }
    const int64_t sst = ctx->stage_stride;
    e = cudaMemcpy2DAsync(ctx->stage_w, sizeof(float) * sst, w_host, sizeof(float) * row_stride,
                          sizeof(float) * d, (size_t)K, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(ctx->stage_w_t0, w_t0_host, sizeof(float) * d, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && xi_host)
        e = cudaMemcpyAsync(ctx->stage_xi, xi_host, sizeof(float) * d, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_round_host: host-to-device copy");

    fda_status st = fda_local_state(ctx, ctx->stage_w, sst, K, d, ctx->stage_w_t0,
                                    xi_host ? ctx->stage_xi : nullptr, state_flags,
                                    ctx->stage_states, stream);
    if (st != FDA_OK) return st;
    st = fda_combine_estimate(ctx, ctx->stage_states, K, variant, epsilon, theta, ctx->stage_est,
                              est_host, stream);          // synchronises: est_host is valid
    if (st != FDA_OK) return st;
    if (states_host) {
        e = cudaMemcpyAsync(states_host, ctx->stage_states, sizeof(float) * (size_t)K * slen,
                            cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_round_host: states copy");
    }
    const bool fire = (avg_flags & FDA_AVG_UNCONDITIONAL) || est_host->trigger != 0;
    if (fire) {
        st = fda_average_models(ctx, ctx->stage_w, sst, K, d, ctx->stage_w_t0, nullptr,
                                (avg_flags & FDA_AVG_BROADCAST) | FDA_AVG_UNCONDITIONAL, stream);
        if (st != FDA_OK) return st;
        e = cudaMemcpyAsync(w_t0_host, ctx->stage_w_t0, sizeof(float) * d, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess && (avg_flags & FDA_AVG_BROADCAST))
            e = cudaMemcpy2DAsync(w_host, sizeof(float) * row_stride, ctx->stage_w, sizeof(float) * sst,
                                  sizeof(float) * d, (size_t)K, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_round_host: device-to-host copy");
    }
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_round_host: synchronize");
    return FDA_OK;
}

fda_status fda_debug_hash(fda_ctx *ctx, int64_t j0, int64_t n, uint16_t *buckets, int8_t *signs,
                          void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!buckets || !signs || ctx->l == 0 || j0 < 0 || n < 1 || j0 + n > ((int64_t)1 << 31))
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_debug_hash: argument out of range");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_debug_hash: cannot select device");
    cudaError_t e = fda_launch_debug_hash(ctx, j0, n, buckets, signs, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_debug_hash");
    return FDA_OK;
}

fda_status fda_debug_schedule(const fda_ctx *ctx, int64_t tile, void *record_host, size_t capacity,
                              int64_t *info)
{
    if (!ctx || !record_host || !info) return FDA_ERR_INVALID_ARG;
    if (!ctx->sched) return FDA_ERR_UNSUPPORTED;
    if (tile < 0 || tile >= ctx->sched_tiles) return FDA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FDA_ERR_CUDA;
    uint64_t off[2] = {0, 0};
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(off, ctx->sched_off + tile, sizeof(off), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { cudaGetLastError(); return FDA_ERR_CUDA; }
    info[0] = ctx->sched_T;
    info[1] = kListSlots;
    info[2] = kListMaxLen;
    info[3] = (int64_t)(off[1] - off[0]);
    info[4] = ctx->sched_tiles;
    info[5] = kListPadRows;
    info[6] = kListOct;
    info[7] = (int64_t)ctx->sched_bytes;
    const size_t n = capacity < (size_t)info[3] ? capacity : (size_t)info[3];
    e = cudaMemcpy(record_host, ctx->sched + off[0], n, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { cudaGetLastError(); return FDA_ERR_CUDA; }
    return FDA_OK;
}

fda_status fda_context_info(const fda_ctx *ctx, int64_t *info)
{
    if (!ctx || !info) return FDA_ERR_INVALID_ARG;
    const int64_t table = ctx->tab ? (int64_t)(sizeof(uint16_t) * (size_t)ctx->l * ctx->tab_stride) : 0;
    const int64_t sched = ctx->sched ? (int64_t)(ctx->sched_bytes + sizeof(uint64_t) * (size_t)(ctx->sched_tiles + 1)) : 0;
    const int64_t partial = (int64_t)(sizeof(float) * ctx->part_sk_floats + sizeof(double) * ctx->part_np_doubles +
                                      sizeof(double) * (2 + FDA_MAX_ROWS) + sizeof(unsigned int)) +
                            (ctx->coeffs_dev ? (int64_t)sizeof(uint64_t) * 6 * ctx->l : 0);
    const int64_t mean = ctx->mean_model ? (int64_t)sizeof(float) * ((ctx->d_max + 3) / 4 * 4) : 0;
    int64_t stage = 0;
    if (ctx->stage_w)
        stage = (int64_t)sizeof(float) * ((int64_t)ctx->K_max * ctx->stage_stride + 2 * ctx->stage_stride +
                                          (int64_t)ctx->K_max * (2 + ctx->lm)) + (int64_t)sizeof(fda_estimate);
    info[0] = table + sched + partial + mean + stage;
    info[1] = sched;
    info[2] = ctx->sched ? 1 : 0;
    info[3] = ctx->sched_T;
    info[4] = (int64_t)ctx->sched_skipped_bytes;
    info[5] = table;
    info[6] = (int64_t)(ctx->sched_build_ms * 1000.0);
    info[7] = mean + stage;
    return FDA_OK;
}

fda_status fda_debug_read_probe(fda_ctx *ctx, const float *src, int64_t n, float *sum_out, void *stream)
{
    if (!ctx) return FDA_ERR_INVALID_ARG;
    if (!src || !sum_out || n < 1)
        return fail(ctx, FDA_ERR_INVALID_ARG, "fda_debug_read_probe: argument out of range");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, FDA_ERR_CUDA, "fda_debug_read_probe: cannot select device");
    cudaError_t e = fda_launch_read_probe(ctx, src, n, sum_out, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fda_debug_read_probe");
    return FDA_OK;
}

}  // extern "C"
