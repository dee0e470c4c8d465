// Shared declarations of libatp: context, launch helpers, dtype conversion, counter-based hash.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <vector>
#include <mutex>
#include "atp.h"

// One record per kernel launch while profiling is on (see atp_profile_start).
struct ProfRec { const char *name; cudaEvent_t a, b; double flops, bytes; };

struct atp_ctx {
    bool profiling = false;
    bool prof_open = false;
    std::vector<ProfRec> recs;
    int device = 0;
    cudaStream_t stream = nullptr;
    void *workspace = nullptr;
    size_t workspace_bytes = 0;
    int *dev_status = nullptr;       // one word, sticky: first non-zero atp_status raised on device
    int64_t launches = 0;
    cudaError_t last_cuda = cudaSuccess;
    int sm_count = 148;
    // two auxiliary streams: halves of a batch run their latency-bound kernel chains side by side
    cudaStream_t aux[2] = {nullptr, nullptr};
    cudaEvent_t ev_fork = nullptr, ev_join[2] = {nullptr, nullptr};
    // convergence feedback of iterative kernels: device word -> pinned host word, ring of 4 slots
    int *h_flags = nullptr;          // pinned host, 4 ints
    int *d_flags = nullptr;          // device, 4 ints
    cudaEvent_t ev_flag[4] = {nullptr, nullptr, nullptr, nullptr};
};

#define ATP_CUDA_OK(ctx, expr)                                   \
    do {                                                         \
        cudaError_t e__ = (expr);                                \
        if (e__ != cudaSuccess) { (ctx)->last_cuda = e__; return ATP_ERR_CUDA; } \
    } while (0)

// Before a kernel launch: name it and state its algorithmic work (used only while profiling).
static inline void prof_begin(atp_ctx *ctx, const char *name, double flops, double bytes)
{
    if (!ctx->profiling) return;
    ProfRec r{name, nullptr, nullptr, flops, bytes};
    if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
    cudaEventRecord(r.a, ctx->stream);
    ctx->recs.push_back(r);
    ctx->prof_open = true;
}
static inline void prof_end(atp_ctx *ctx)
{
    if (ctx->prof_open) { cudaEventRecord(ctx->recs.back().b, ctx->stream); ctx->prof_open = false; }
}
#define ATP_KERNEL(ctx, name, flops, bytes) prof_begin((ctx), (name), (double)(flops), (double)(bytes))

// After a kernel launch: count it and surface launch-configuration errors.
#define ATP_LAUNCHED(ctx)                                        \
    do {                                                         \
        (ctx)->launches++;                                       \
        prof_end(ctx);                                           \
        cudaError_t e__ = cudaGetLastError();                    \
        if (e__ != cudaSuccess) { (ctx)->last_cuda = e__; return ATP_ERR_CUDA; } \
    } while (0)

// Programmatic dependent launch: a kernel launched through launch_pdl may begin (run its prologue, which
// must touch no global data) while its predecessor in the stream is still draining; pdl_wait() then
// blocks until the predecessor has completed and its writes are visible. Every thread of such a kernel
// calls pdl_wait() before its first global access and before any exit, so "this kernel has completed"
// keeps implying "everything before it has completed". pdl_trigger() lets the successor start launching.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Runs a per-device set-up step (a kernel attribute, an address look-up) once for every device
// ordinal, whichever context or thread comes first; a failed step is retried by the next caller.
struct PerDeviceOnce {
    static constexpr int MAX_DEV = 64;
    std::mutex mu;
    bool done[MAX_DEV] = {};
    template <typename F> cudaError_t run(int device, F step)
    {
        std::lock_guard<std::mutex> lk(mu);
        if (device >= 0 && device < MAX_DEV && done[device]) return cudaSuccess;
        const cudaError_t e = step();
        if (e == cudaSuccess && device >= 0 && device < MAX_DEV) done[device] = true;
        return e;
    }
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Bump allocator over the caller's workspace (host-side bookkeeping only).
struct Arena {
    char *base; size_t cap; size_t off = 0; bool overflow = false;
    Arena(void *b, size_t c) : base((char *)b), cap(c) {}
    template <typename T> T *take(size_t n) {
        off = align_up(off, 256);
        size_t bytes = n * sizeof(T);
        T *p = (T *)(base ? base + off : nullptr);
        off += bytes;
        if (off > cap) overflow = true;
        return p;
    }
};

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// splitmix64 finaliser used as a counter-based generator: value = mix(seed, counter).
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t seed, uint64_t ctr) {
    uint64_t z = seed + 0x9E3779B97F4A7C15ull * (ctr + 1);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ float hash_uniform(uint64_t seed, uint64_t ctr) {   // in (-1, 1)
    return ((float)(mix64(seed, ctr) >> 40) + 0.5f) * (2.0f / 16777216.0f) - 1.0f;
}

__device__ __forceinline__ void raise_status(int *dev_status, int code) { atomicCAS(dev_status, 0, code); }

static inline size_t dtype_size(atp_dtype t) { return t == ATP_BF16 ? 2 : 4; }

// Per-sequence sizes of a packed batch, host side.
struct SeqDims { int row0, L, r, rank0; };
atp_status check_seqs(const atp_seqs *s, std::vector<SeqDims> &out, int64_t total_rows_expected);
atp_status check_mat(const atp_mat *m, bool need_data = true);
size_t alternating_workspace_bytes(const std::vector<SeqDims> &sd, int d);
