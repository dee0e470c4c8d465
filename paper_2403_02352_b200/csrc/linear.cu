// atp_lowrank_linear: Y = act(U_r (X_r W) + bias)  (Sec. 4.3: linear layers on the r-row representation).
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include <type_traits>

struct LinearPlan {
    float *T = nullptr, *Tg = nullptr, *Yg = nullptr;
    __nv_bfloat16 *Tb = nullptr, *Tgb = nullptr;     // tensor-core path: T and T_gate in bf16
};

static size_t plan_linear(Arena &ar, int64_t total_rank, int64_t total_rows, int64_t d_out, bool swiglu, bool bf16, LinearPlan &p)
{
    if (bf16) {
        const size_t ldt = align_up((size_t)d_out, 8);
        p.Tb = ar.take<__nv_bfloat16>((size_t)total_rank * ldt);
        if (swiglu) p.Tgb = ar.take<__nv_bfloat16>((size_t)total_rank * ldt);
    } else {
        p.T = ar.take<float>((size_t)total_rank * d_out);
        if (swiglu) p.Tg = ar.take<float>((size_t)total_rank * d_out);
    }
    if (swiglu) p.Yg = ar.take<float>((size_t)total_rows * d_out);
    return ar.off;
}

size_t linear_workspace_bytes(const std::vector<SeqDims> &seqs, int64_t d_out)
{
    int64_t tr = 0, tl = 0;
    for (auto &s : seqs) { tr += s.r; tl += s.L; }
    Arena ar(nullptr, (size_t)-1);
    LinearPlan p;
    return plan_linear(ar, tr, tl, d_out, true, false, p);      // sized for the fp32 SwiGLU case (the largest one)
}

template <typename T>
static atp_status linear_impl(atp_ctx *ctx, const atp_mat *U_r, const atp_mat *X_r, const atp_mat *W,
                              const std::vector<SeqDims> &seqs, int act, const float *bias, const atp_mat *Wg,
                              atp_mat *Y)
{
    const int d_in = (int)W->rows, d_out = (int)W->cols;
    int64_t tr = 0, tl = 0;
    for (auto &s : seqs) { tr += s.r; tl += s.L; }
    const bool swiglu = act == ATP_ACT_SWIGLU;
    Arena ar(ctx->workspace, ctx->workspace_bytes);
    LinearPlan pl;
    plan_linear(ar, tr, tl, d_out, swiglu, std::is_same<T, __nv_bfloat16>::value, pl);
    if (ar.overflow || (!ctx->workspace && ar.off > 0)) return ATP_ERR_WORKSPACE_TOO_SMALL;

    atp_status st;
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        // bf16: both GEMMs on the tensor cores; T is rounded to bf16 once (fp32 accumulation)
        const int ldt = (int)align_up((size_t)d_out, 8);
        std::vector<tc::HostProblem> p1;
        p1.push_back(tc::HostProblem{X_r->data, W->data, nullptr, pl.Tb, nullptr, nullptr, (int)tr, d_out, d_in,
                                     (int)X_r->ld, (int)W->ld, ldt, 0});
        if (swiglu)
            p1.push_back(tc::HostProblem{X_r->data, Wg->data, nullptr, pl.Tgb, nullptr, nullptr, (int)tr, d_out, d_in,
                                         (int)X_r->ld, (int)Wg->ld, ldt, 0});
        if ((st = tc::launch<false, false, tc::OUT_BF16>(ctx, p1, GemmEpi{EPI_STORE, nullptr})) != ATP_OK) return st;
        std::vector<tc::HostProblem> pg, pm;
        for (auto &s : seqs) {
            if (s.L == 0) continue;
            const T *u = (const T *)U_r->data + (size_t)s.row0 * U_r->ld;
            T *y = (T *)Y->data + (size_t)s.row0 * Y->ld;
            float *yg = swiglu ? pl.Yg + (size_t)s.row0 * d_out : nullptr;
            if (swiglu)
                pg.push_back(tc::HostProblem{u, pl.Tgb + (size_t)s.rank0 * ldt, nullptr, yg, nullptr, nullptr, s.L, d_out, s.r,
                                             (int)U_r->ld, ldt, d_out, 0});
            pm.push_back(tc::HostProblem{u, pl.Tb + (size_t)s.rank0 * ldt, nullptr, y, nullptr, yg, s.L, d_out, s.r,
                                         (int)U_r->ld, ldt, (int)Y->ld, d_out});
        }
        if (swiglu && (st = tc::launch<false, false, tc::OUT_F32>(ctx, pg, GemmEpi{EPI_STORE, nullptr})) != ATP_OK) return st;
        GemmEpi epi{swiglu ? EPI_SILU_D_MUL : (act == ATP_ACT_GELU ? EPI_BIAS_GELU : EPI_BIAS), bias};
        return tc::launch<false, false, tc::OUT_BF16>(ctx, pm, epi);
    }
    // T = X_r W for all sequences at once (rows of X_r are packed)
    {
        GemmBatch b; b.count = 1;
        b.p[0] = GemmProblem{X_r->data, W->data, pl.T, nullptr, (int)tr, d_out, d_in, (int)X_r->ld, (int)W->ld, d_out, 0};
        if ((st = launch_gemm_simt<T, T, float, false>(ctx, b, GemmEpi{EPI_STORE, nullptr})) != ATP_OK) return st;
        if (swiglu) {
            b.p[0].B = Wg->data; b.p[0].ldb = (int)Wg->ld; b.p[0].C = pl.Tg;
            if ((st = launch_gemm_simt<T, T, float, false>(ctx, b, GemmEpi{EPI_STORE, nullptr})) != ATP_OK) return st;
        }
    }
    // Y_b = U_r,b T_b with the epilogue
    std::vector<GemmProblem> gate, main_;
    for (auto &s : seqs) {
        if (s.L == 0) continue;
        const T *u = (const T *)U_r->data + (size_t)s.row0 * U_r->ld;
        T *y = (T *)Y->data + (size_t)s.row0 * Y->ld;
        const float *t = pl.T + (size_t)s.rank0 * d_out;
        if (swiglu) {
            float *yg = pl.Yg + (size_t)s.row0 * d_out;
            gate.push_back(GemmProblem{u, pl.Tg + (size_t)s.rank0 * d_out, yg, nullptr, s.L, d_out, s.r, (int)U_r->ld, d_out, d_out, 0});
            main_.push_back(GemmProblem{u, t, y, yg, s.L, d_out, s.r, (int)U_r->ld, d_out, (int)Y->ld, d_out});
        } else {
            main_.push_back(GemmProblem{u, t, y, nullptr, s.L, d_out, s.r, (int)U_r->ld, d_out, (int)Y->ld, 0});
        }
    }
    if (swiglu) {
        st = for_each_chunk(gate, [&](const GemmBatch &b) { return launch_gemm_simt<T, float, float, false>(ctx, b, GemmEpi{EPI_STORE, nullptr}); });
        if (st != ATP_OK) return st;
    }
    GemmEpi epi{swiglu ? EPI_SILU_D_MUL : (act == ATP_ACT_GELU ? EPI_BIAS_GELU : EPI_BIAS), bias};
    return for_each_chunk(main_, [&](const GemmBatch &b) { return launch_gemm_simt<T, float, T, false>(ctx, b, epi); });
}

extern "C" atp_status atp_lowrank_linear(atp_ctx *ctx, const atp_mat *U_r, const atp_mat *X_r, const atp_mat *W,
                                         const atp_seqs *seqs, const atp_linear_opts *opts, atp_mat *Y)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    atp_status st;
    if ((st = check_mat(U_r)) != ATP_OK || (st = check_mat(X_r)) != ATP_OK || (st = check_mat(W)) != ATP_OK ||
        (st = check_mat(Y)) != ATP_OK)
        return st;
    int act = ATP_ACT_NONE; const float *bias = nullptr; const atp_mat *Wg = nullptr;
    if (opts) {
        if (opts->struct_size < sizeof(atp_linear_opts)) return ATP_ERR_INVALID_ARG;
        act = opts->act; bias = opts->bias; Wg = opts->W_gate;
    }
    if (act != ATP_ACT_NONE && act != ATP_ACT_GELU && act != ATP_ACT_SWIGLU) return ATP_ERR_INVALID_ARG;
    if (act == ATP_ACT_SWIGLU) {
        if (!Wg || (st = check_mat(Wg)) != ATP_OK) return st != ATP_OK ? st : ATP_ERR_INVALID_ARG;
        if (Wg->rows != W->rows || Wg->cols != W->cols || Wg->dtype != W->dtype) return ATP_ERR_INVALID_ARG;
        if (bias) return ATP_ERR_INVALID_ARG;
    }
    if (U_r->dtype != X_r->dtype || W->dtype != X_r->dtype || Y->dtype != U_r->dtype) return ATP_ERR_UNSUPPORTED_DTYPE;
    std::vector<SeqDims> sd;
    if ((st = check_seqs(seqs, sd, U_r->rows)) != ATP_OK) return st;
    int64_t tr = 0; int maxr = 0;
    for (auto &s : sd) { tr += s.r; if (s.r > maxr) maxr = s.r; }
    if (X_r->rows != tr || X_r->cols != W->rows || U_r->cols < maxr || Y->rows != U_r->rows || Y->cols != W->cols)
        return ATP_ERR_INVALID_ARG;
    if (U_r->rows == 0) return ATP_OK;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    if (U_r->dtype == ATP_F32) return linear_impl<float>(ctx, U_r, X_r, W, sd, act, bias, Wg, Y);
    return linear_impl<__nv_bfloat16>(ctx, U_r, X_r, W, sd, act, bias, Wg, Y);
}

// ------------------------------------------------------------------------------------------------
// Low-rank linear layer for callers that cannot allocate device memory.
//
// The regular call keeps its intermediate T = X_r W (sum(r_b) x d_out, fp32) in the caller's
// workspace. Code that runs where cudaMalloc is off limits -- a plug-in inside a host process that
// owns the memory pool, a real-time loop that must not touch the allocator -- has no buffer to
// hand over and cannot create a context either (atp_create allocates its status word). For those
// callers the same kernels run here with T placed in a fixed array that is part of the library
// image: every GPU that loads libatp.so holds ATP_STATIC_SCRATCH_BYTES of it until the process
// exits, whether or not this entry point is ever called.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[ATP_STATIC_SCRATCH_BYTES];

#include <mutex>
static std::mutex g_static_mu;
static void *g_static_ptr[64];          // device address of g_static_scratch, per device ordinal

// The array's name is only a host-side handle; the device address a kernel can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static atp_status static_scratch_for_current_device(int *device, void **ptr)
{
    if (cudaGetDevice(device) != cudaSuccess) return ATP_ERR_CUDA;
    if (*device < 0 || *device >= 64) return ATP_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[*device]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ATP_ERR_CUDA;
        g_static_ptr[*device] = p;
    }
    *ptr = g_static_ptr[*device];
    return ATP_OK;
}

extern "C" atp_status atp_lowrank_linear_static(void *cuda_stream, const atp_mat *U_r, const atp_mat *X_r,
                                                const atp_mat *W, const atp_seqs *seqs, const atp_linear_opts *opts,
                                                atp_mat *Y)
{
    atp_status st;
    if ((st = check_mat(U_r)) != ATP_OK || (st = check_mat(X_r)) != ATP_OK || (st = check_mat(W)) != ATP_OK ||
        (st = check_mat(Y)) != ATP_OK)
        return st;
    int act = ATP_ACT_NONE; const float *bias = nullptr;
    if (opts) {
        if (opts->struct_size < sizeof(atp_linear_opts)) return ATP_ERR_INVALID_ARG;
        act = opts->act; bias = opts->bias;
    }
    if (act != ATP_ACT_NONE && act != ATP_ACT_GELU) return ATP_ERR_INVALID_ARG;     // no SwiGLU here: it needs L x d_out more
    if (U_r->dtype != X_r->dtype || W->dtype != X_r->dtype || Y->dtype != U_r->dtype) return ATP_ERR_UNSUPPORTED_DTYPE;
    std::vector<SeqDims> sd;
    if ((st = check_seqs(seqs, sd, U_r->rows)) != ATP_OK) return st;
    int64_t tr = 0; int maxr = 0;
    for (auto &s : sd) { tr += s.r; if (s.r > maxr) maxr = s.r; }
    if (X_r->rows != tr || X_r->cols != W->rows || U_r->cols < maxr || Y->rows != U_r->rows || Y->cols != W->cols)
        return ATP_ERR_INVALID_ARG;
    if (U_r->rows == 0) return ATP_OK;
    // T is the only scratch; it is written in full before it is read, so nothing has to be cleared.
    // (fp32: sum(r) x d_out floats; bf16: the same matrix in bf16 with its rows padded to 8 elements)
    const uint64_t need = U_r->dtype == ATP_F32 ? (uint64_t)tr * (uint64_t)W->cols * sizeof(float)
                                                 : (uint64_t)tr * (uint64_t)align_up((size_t)W->cols, 8) * sizeof(__nv_bfloat16);
    if (need > ATP_STATIC_SCRATCH_BYTES || (uint64_t)tr * (uint64_t)W->cols * sizeof(float) > ATP_STATIC_SCRATCH_BYTES)
        return ATP_ERR_STATIC_SCRATCH_LIMIT;
    atp_ctx local;                      // host-side bookkeeping only; owns nothing on the device
    void *scratch = nullptr;
    if ((st = static_scratch_for_current_device(&local.device, &scratch)) != ATP_OK) return st;
    local.stream = (cudaStream_t)cuda_stream;
    local.workspace = scratch;
    local.workspace_bytes = ATP_STATIC_SCRATCH_BYTES;
    if (U_r->dtype == ATP_F32) return linear_impl<float>(&local, U_r, X_r, W, sd, act, bias, nullptr, Y);
    return linear_impl<__nv_bfloat16>(&local, U_r, X_r, W, sd, act, bias, nullptr, Y);
}
