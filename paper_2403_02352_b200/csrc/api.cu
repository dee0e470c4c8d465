// Context management, argument validation, status handling and the Norm box of Fig. 3.
#include "common.cuh"
#include <new>
#include <string>
#include <string.h>
#include <stdio.h>

atp_status check_mat(const atp_mat *m, bool need_data)
{
    if (!m) return ATP_ERR_INVALID_ARG;
    if (need_data && !m->data) return ATP_ERR_INVALID_ARG;
    if (m->dtype != ATP_F32 && m->dtype != ATP_BF16) return ATP_ERR_UNSUPPORTED_DTYPE;
    if (m->rows < 0 || m->cols < 0 || m->ld < m->cols) return ATP_ERR_INVALID_ARG;
    if (m->rows > 0x7fffffff || m->cols > 0x7fffffff || m->ld > 0x7fffffff) return ATP_ERR_INVALID_ARG;
    if (m->dtype == ATP_BF16) {
        if (((uintptr_t)m->data & 15) || (m->ld & 7)) return ATP_ERR_INVALID_ARG;
    } else if ((uintptr_t)m->data & 3) {
        return ATP_ERR_INVALID_ARG;
    }
    return ATP_OK;
}

atp_status check_seqs(const atp_seqs *s, std::vector<SeqDims> &out, int64_t total_rows_expected)
{
    if (!s || s->batch < 0 || (s->batch > 0 && (!s->row_off || !s->rank || !s->rank_off))) return ATP_ERR_INVALID_ARG;
    out.clear();
    if (s->batch > 0 && (s->row_off[0] != 0 || s->rank_off[0] != 0)) return ATP_ERR_INVALID_ARG;
    for (int b = 0; b < s->batch; ++b) {
        SeqDims d;
        d.row0 = s->row_off[b];
        d.L = s->row_off[b + 1] - s->row_off[b];
        d.r = s->rank[b];
        d.rank0 = s->rank_off[b];
        if (d.L < 0) return ATP_ERR_INVALID_ARG;
        if (s->rank_off[b + 1] - s->rank_off[b] != d.r) return ATP_ERR_INVALID_ARG;
        if (d.L > 0 && (d.r < 1 || d.r > d.L)) return ATP_ERR_INVALID_RANK;
        if (d.L == 0 && d.r != 0) return ATP_ERR_INVALID_RANK;
        out.push_back(d);
    }
    if (total_rows_expected >= 0 && s->batch > 0 && s->row_off[s->batch] != total_rows_expected) return ATP_ERR_INVALID_ARG;
    return ATP_OK;
}

extern "C" {

atp_status atp_create(atp_ctx **out, int device)
{
    if (!out) return ATP_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return ATP_ERR_CUDA;
    atp_ctx *ctx = new (std::nothrow) atp_ctx();
    if (!ctx) return ATP_ERR_INVALID_ARG;
    ctx->device = device;
    if (cudaSetDevice(device) != cudaSuccess) { delete ctx; return ATP_ERR_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return ATP_ERR_CUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    // two words: [0] the sticky status, [1] the abort flag shared by the bounded waits of persistent kernels
    if (cudaMalloc(&ctx->dev_status, 2 * sizeof(int)) != cudaSuccess) { delete ctx; return ATP_ERR_CUDA; }
    if (cudaMemset(ctx->dev_status, 0, 2 * sizeof(int)) != cudaSuccess) { cudaFree(ctx->dev_status); delete ctx; return ATP_ERR_CUDA; }
    bool ok = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
        ok = cudaStreamCreateWithFlags(&ctx->aux[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&ctx->ev_join[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaHostAlloc((void **)&ctx->h_flags, 4 * sizeof(int), cudaHostAllocDefault) == cudaSuccess &&
         cudaMalloc((void **)&ctx->d_flags, 4 * sizeof(int)) == cudaSuccess;
    for (int i = 0; i < 4 && ok; ++i) ok = cudaEventCreateWithFlags(&ctx->ev_flag[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { atp_destroy(ctx); return ATP_ERR_CUDA; }
    *out = ctx;
    return ATP_OK;
}

atp_status atp_destroy(atp_ctx *ctx)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    for (int i = 0; i < 2; ++i) {
        if (ctx->aux[i]) cudaStreamDestroy(ctx->aux[i]);
        if (ctx->ev_join[i]) cudaEventDestroy(ctx->ev_join[i]);
    }
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    for (int i = 0; i < 4; ++i) if (ctx->ev_flag[i]) cudaEventDestroy(ctx->ev_flag[i]);
    if (ctx->h_flags) cudaFreeHost(ctx->h_flags);
    if (ctx->d_flags) cudaFree(ctx->d_flags);
    delete ctx;
    return ATP_OK;
}

atp_status atp_set_stream(atp_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    ctx->stream = (cudaStream_t)cuda_stream;
    return ATP_OK;
}

atp_status atp_set_workspace(atp_ctx *ctx, void *dev_ptr, size_t bytes)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    if (bytes > 0 && (!dev_ptr || ((uintptr_t)dev_ptr & 255))) return ATP_ERR_INVALID_ARG;
    ctx->workspace = dev_ptr;
    ctx->workspace_bytes = bytes;
    return ATP_OK;
}

atp_status atp_poll_device_status(atp_ctx *ctx)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    ATP_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));
    int st[2] = {0, 0};
    ATP_CUDA_OK(ctx, cudaMemcpy(st, ctx->dev_status, 2 * sizeof(int), cudaMemcpyDeviceToHost));
    if (st[0] != 0 || st[1] != 0) ATP_CUDA_OK(ctx, cudaMemset(ctx->dev_status, 0, 2 * sizeof(int)));
    return (atp_status)st[0];
}

int64_t atp_launch_count(const atp_ctx *ctx) { return ctx ? ctx->launches : -1; }

atp_status atp_profile_start(atp_ctx *ctx)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    ctx->profiling = true;
    return ATP_OK;
}

atp_status atp_profile_stop(atp_ctx *ctx, char *buf, size_t cap, size_t *needed)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    ctx->profiling = false;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    ATP_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));
    struct Agg { const char *name; long n; double ms, flops, bytes; };
    std::vector<Agg> agg;
    for (auto &r : ctx->recs) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, r.a, r.b);
        cudaEventDestroy(r.a); cudaEventDestroy(r.b);
        size_t i = 0;
        for (; i < agg.size(); ++i) if (!strcmp(agg[i].name, r.name)) break;
        if (i == agg.size()) agg.push_back(Agg{r.name, 0, 0, 0, 0});
        agg[i].n++; agg[i].ms += ms; agg[i].flops += r.flops; agg[i].bytes += r.bytes;
    }
    ctx->recs.clear();
    std::string out;
    char line[256];
    for (auto &a : agg) {
        snprintf(line, sizeof line, "%s %ld %.6f %.6e %.6e\n", a.name, a.n, a.ms, a.flops, a.bytes);
        out += line;
    }
    if (needed) *needed = out.size() + 1;
    if (buf && cap > 0) {
        size_t n = out.size() < cap - 1 ? out.size() : cap - 1;
        memcpy(buf, out.data(), n);
        buf[n] = 0;
    }
    return ATP_OK;
}

const char *atp_status_string(atp_status s)
{
    switch (s) {
        case ATP_OK: return "ok";
        case ATP_ERR_INVALID_ARG: return "invalid argument";
        case ATP_ERR_INVALID_RANK: return "invalid rank (need 1 <= r <= min(L, d))";
        case ATP_ERR_UNSUPPORTED_DTYPE: return "unsupported dtype";
        case ATP_ERR_WORKSPACE_TOO_SMALL: return "workspace too small (see atp_workspace_bytes)";
        case ATP_ERR_CUDA: return "CUDA runtime error";
        case ATP_ERR_NOT_CONVERGED: return "Jacobi iteration hit its sweep limit";
        case ATP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case ATP_ERR_RANGE: return "value outside the representable range";
        case ATP_ERR_STATIC_SCRATCH_LIMIT:
            return "problem exceeds the fixed scratch buffer of atp_lowrank_linear_static (sum(r) * d_out * 4 bytes > ATP_STATIC_SCRATCH_BYTES)";
    }
    return "unknown status";
}

}  // extern "C"

// ----------------------------------------------------------------------------------------------
// Norm box of Fig. 3: one warp per row, row statistics in fp32, two passes over the row (the
// second one hits L1/L2). HBM-bound: one read and one write of X.
// ----------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
norm_kernel(const T *X, const T *R, T *Y, int rows, int cols, int ldx, int ldr, int ldy, int kind, float eps)
{
    int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const T *x = X + (size_t)row * ldx;
    const T *r = R ? R + (size_t)row * ldr : nullptr;
    float s = 0.f, s2 = 0.f;
    for (int c = lane; c < cols; c += 32) {
        float v = to_f32(x[c]) + (r ? to_f32(r[c]) : 0.f);
        s += v;
        s2 += v * v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, o);
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    float mean = (kind == ATP_NORM_LAYER) ? s / cols : 0.f;
    float var = 0.f;
    if (kind == ATP_NORM_LAYER) {        // second moment about the mean, computed directly
        for (int c = lane; c < cols; c += 32) {
            float v = to_f32(x[c]) + (r ? to_f32(r[c]) : 0.f) - mean;
            var += v * v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) var += __shfl_xor_sync(0xffffffffu, var, o);
        var /= cols;
    } else {
        var = s2 / cols;
    }
    float inv = rsqrtf(var + eps);
    T *y = Y + (size_t)row * ldy;
    for (int c = lane; c < cols; c += 32) {
        float v = to_f32(x[c]) + (r ? to_f32(r[c]) : 0.f);
        y[c] = from_f32<T>((v - mean) * inv);
    }
}

extern "C" atp_status atp_input_norm(atp_ctx *ctx, const atp_mat *X, const atp_mat *residual, int kind, float eps,
                                     atp_mat *Y)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    atp_status st;
    if ((st = check_mat(X)) != ATP_OK) return st;
    if ((st = check_mat(Y)) != ATP_OK) return st;
    if (residual && (st = check_mat(residual)) != ATP_OK) return st;
    if (kind != ATP_NORM_RMS && kind != ATP_NORM_LAYER) return ATP_ERR_INVALID_ARG;
    if (Y->rows != X->rows || Y->cols != X->cols || Y->dtype != X->dtype) return ATP_ERR_INVALID_ARG;
    if (residual && (residual->rows != X->rows || residual->cols != X->cols || residual->dtype != X->dtype))
        return ATP_ERR_INVALID_ARG;
    if (!(eps >= 0.f)) return ATP_ERR_INVALID_ARG;
    if (X->rows == 0 || X->cols == 0) return ATP_OK;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    int rows = (int)X->rows, cols = (int)X->cols;
    dim3 grid(ceil_div(rows, 8));
    ATP_KERNEL(ctx, "norm", 0, (double)rows * cols * dtype_size(X->dtype) * (residual ? 3 : 2));
    if (X->dtype == ATP_F32)
        norm_kernel<float><<<grid, 256, 0, ctx->stream>>>((const float *)X->data, residual ? (const float *)residual->data : nullptr,
                                                          (float *)Y->data, rows, cols, (int)X->ld, residual ? (int)residual->ld : 0,
                                                          (int)Y->ld, kind, eps);
    else
        norm_kernel<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>((const __nv_bfloat16 *)X->data,
                                                                  residual ? (const __nv_bfloat16 *)residual->data : nullptr,
                                                                  (__nv_bfloat16 *)Y->data, rows, cols, (int)X->ld,
                                                                  residual ? (int)residual->ld : 0, (int)Y->ld, kind, eps);
    ATP_LAUNCHED(ctx);
    return ATP_OK;
}
