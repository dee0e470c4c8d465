// atp_alternating_basis: the paper's own approximate extraction (Algorithm 1, appendix B) - rank-1
// alternating fits with deflation - and atp_svd_entropy: Eq. 4 with the rank rule of Sec. 3.
//
// Algorithm 1 on the GPU. The method is a chain of matrix-vector products over the deflated matrix
// R (L x d, fp32, resident in the workspace): for every component, `inner` rounds of
//   u = R v / |v|^2,   v = R^T u / |u|^2,
// then R <- R - u v^T. Every product reads R once, so the path is bound by memory traffic
// ((2 inner + 2) L d 4 bytes per component; R stays in L2 when it fits). Dot products accumulate in
// fp64 so that the only rounding of a step is the fp32 storage of u, v and R.
#include "common.cuh"

constexpr int ALT_MAX = 32;        // sequences per launch
struct AltSeq {
    float *R, *u, *v;              // deflated copy (L x d), current u (L), current v (d)
    const float *v0;               // start vectors of this sequence (r x d, row stride ldv)
    void *U, *Xp;                  // outputs: U (L x r), X' (r x d)
    int L, r, ldu, ldx, ldv;
    int row0;                      // first row of the sequence in the packed input
};
struct AltBatch { AltSeq s[ALT_MAX]; int count; };

__device__ __forceinline__ double block_sum_256(double x, double *red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    const int w = threadIdx.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[w] = x;
    __syncthreads();
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += red[i];       // fixed order
    return s;
}

template <typename T>
__global__ void __launch_bounds__(256) alt_copy_kernel(const __grid_constant__ AltBatch batch, const T *X, int ldx_in, int d)
{
    const AltSeq &q = batch.s[blockIdx.y];
    const size_t n = (size_t)q.L * d;
    const T *src = X + (size_t)q.row0 * ldx_in;
    for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < n; e += (size_t)gridDim.x * 256) {
        const int l = (int)(e / d), k = (int)(e - (size_t)l * d);
        q.R[e] = to_f32(src[(size_t)l * ldx_in + k]);
    }
}

// u = R v / |v|^2; one warp per row. `first`: v is row `comp` of the start vectors.
__global__ void __launch_bounds__(256) alt_u_kernel(const __grid_constant__ AltBatch batch, int d, int comp, int first)
{
    pdl_trigger();
    pdl_wait();
    const AltSeq &q = batch.s[blockIdx.y];
    if (comp >= q.r) return;
    __shared__ double red[8];
    const float *v = first ? q.v0 + (size_t)comp * q.ldv : q.v;
    double part = 0.0;
    for (int k = threadIdx.x; k < d; k += 256) { const double x = v[k]; part += x * x; }
    const double vv = block_sum_256(part, red);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int l = blockIdx.x * 8 + warp;
    if (l >= q.L) return;
    const float *row = q.R + (size_t)l * d;
    double acc = 0.0;
    for (int k = lane; k < d; k += 32) acc = fma((double)row[k], (double)v[k], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) q.u[l] = vv > 0.0 ? (float)(acc / vv) : 0.f;
}

// v = R^T u / |u|^2; a CTA owns 64 columns, its four quarters split the rows.
__global__ void __launch_bounds__(256) alt_v_kernel(const __grid_constant__ AltBatch batch, int d, int comp)
{
    pdl_trigger();
    pdl_wait();
    const AltSeq &q = batch.s[blockIdx.y];
    if (comp >= q.r) return;
    __shared__ double red[8];
    __shared__ double quarter[3][64];
    double part = 0.0;
    for (int l = threadIdx.x; l < q.L; l += 256) { const double x = q.u[l]; part += x * x; }
    const double uu = block_sum_256(part, red);
    const int c = threadIdx.x & 63, h = threadIdx.x >> 6;
    const int k = blockIdx.x * 64 + c;
    double acc = 0.0;
    if (k < d) {
        int l = h;
        for (; l + 28 < q.L; l += 32) {            // eight loads in flight per thread
            float rv[8], uv[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) { rv[t] = q.R[(size_t)(l + 4 * t) * d + k]; uv[t] = q.u[l + 4 * t]; }
#pragma unroll
            for (int t = 0; t < 8; ++t) acc = fma((double)rv[t], (double)uv[t], acc);
        }
        for (; l < q.L; l += 4) acc = fma((double)q.R[(size_t)l * d + k], (double)q.u[l], acc);
    }
    if (h > 0) quarter[h - 1][c] = acc;
    __syncthreads();
    if (h == 0 && k < d) q.v[k] = uu > 0.0 ? (float)((acc + quarter[0][c] + quarter[1][c] + quarter[2][c]) / uu) : 0.f;
}

// R <- R - u v^T, and the finished component: U[:, comp] = u / |u|, X'[comp, :] = v |u|.
template <typename T>
__global__ void __launch_bounds__(256) alt_deflate_kernel(const __grid_constant__ AltBatch batch, int d, int comp)
{
    pdl_trigger();
    pdl_wait();
    const AltSeq &q = batch.s[blockIdx.y];
    if (comp >= q.r) return;
    __shared__ double red[8];
    double part = 0.0;
    for (int l = threadIdx.x; l < q.L; l += 256) { const double x = q.u[l]; part += x * x; }
    const double un = sqrt(block_sum_256(part, red));
    if (blockIdx.x == 0) {
        T *xp = (T *)q.Xp + (size_t)comp * q.ldx;
        for (int k = threadIdx.x; k < d; k += 256) xp[k] = from_f32<T>((float)((double)q.v[k] * un));
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int l = blockIdx.x * 8 + warp;
    if (l >= q.L) return;
    const float ul = q.u[l];
    float *row = q.R + (size_t)l * d;
    for (int k = lane; k < d; k += 32) row[k] = fmaf(-ul, q.v[k], row[k]);
    if (lane == 0) ((T *)q.U)[(size_t)l * q.ldu + comp] = from_f32<T>(un > 0.0 ? (float)((double)ul / un) : 0.f);
}

size_t alternating_workspace_bytes(const std::vector<SeqDims> &sd, int d)
{
    Arena ar(nullptr, (size_t)-1);
    for (auto &s : sd) { ar.take<float>((size_t)s.L * d); ar.take<float>(s.L); ar.take<float>(d); }
    return ar.off;
}

template <typename T>
static atp_status alternating_impl(atp_ctx *ctx, const atp_mat *X, const std::vector<SeqDims> &sd, const atp_mat *V0, int inner,
                                   atp_mat *U_r, atp_mat *X_r)
{
    const int d = (int)X->cols;
    Arena ar(ctx->workspace, ctx->workspace_bytes);
    std::vector<AltSeq> seqs(sd.size());
    for (size_t i = 0; i < sd.size(); ++i) {
        AltSeq &q = seqs[i];
        q.R = ar.take<float>((size_t)sd[i].L * d); q.u = ar.take<float>(sd[i].L); q.v = ar.take<float>(d);
        q.v0 = (const float *)V0->data + (size_t)sd[i].rank0 * V0->ld;
        q.U = (T *)U_r->data + (size_t)sd[i].row0 * U_r->ld;
        q.Xp = (T *)X_r->data + (size_t)sd[i].rank0 * X_r->ld;
        q.L = sd[i].L; q.r = sd[i].r; q.ldu = (int)U_r->ld; q.ldx = (int)X_r->ld; q.ldv = (int)V0->ld;
        q.row0 = sd[i].row0;
    }
    if (ar.overflow) return ATP_ERR_WORKSPACE_TOO_SMALL;
    for (size_t i0 = 0; i0 < sd.size(); i0 += ALT_MAX) {
        AltBatch b; b.count = (int)std::min<size_t>(ALT_MAX, sd.size() - i0);
        int maxL = 0, maxr = 0;
        for (int k = 0; k < b.count; ++k) { b.s[k] = seqs[i0 + k]; maxL = std::max(maxL, b.s[k].L); maxr = std::max(maxr, b.s[k].r); }
        if (maxL == 0) continue;
        const double mat_bytes = [&] { double s = 0; for (int k = 0; k < b.count; ++k) s += (double)b.s[k].L * d * 4; return s; }();
        ATP_KERNEL(ctx, "alt_copy", 0, mat_bytes * (1.0 + sizeof(T) / 4.0));
        alt_copy_kernel<T><<<dim3(std::min(1024, (int)(((size_t)maxL * d + 255) / 256)), b.count), 256, 0, ctx->stream>>>(
            b, (const T *)X->data, (int)X->ld, d);
        ATP_LAUNCHED(ctx);
        const dim3 grows((maxL + 7) / 8, b.count), gcols((d + 63) / 64, b.count);
        for (int comp = 0; comp < maxr; ++comp) {
            for (int j = 0; j < inner; ++j) {
                ATP_KERNEL(ctx, "alt_u", 0, mat_bytes);
                launch_pdl(alt_u_kernel, grows, dim3(256), 0, ctx->stream, b, d, comp, (int)(j == 0));
                ATP_LAUNCHED(ctx);
                ATP_KERNEL(ctx, "alt_v", 0, mat_bytes);
                launch_pdl(alt_v_kernel, gcols, dim3(256), 0, ctx->stream, b, d, comp);
                ATP_LAUNCHED(ctx);
            }
            ATP_KERNEL(ctx, "alt_deflate", 0, 2.0 * mat_bytes);
            launch_pdl(alt_deflate_kernel<T>, grows, dim3(256), 0, ctx->stream, b, d, comp);
            ATP_LAUNCHED(ctx);
        }
    }
    return ATP_OK;
}

extern "C" atp_status atp_alternating_basis(atp_ctx *ctx, const atp_mat *X, const atp_seqs *seqs, const atp_mat *V0, int inner,
                                            atp_mat *U_r, atp_mat *X_r)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    atp_status st;
    if ((st = check_mat(X)) != ATP_OK || (st = check_mat(U_r)) != ATP_OK || (st = check_mat(X_r)) != ATP_OK ||
        (st = check_mat(V0)) != ATP_OK) return st;
    if (V0->dtype != ATP_F32 || inner < 1 || inner > 64) return ATP_ERR_INVALID_ARG;
    if (U_r->dtype != X->dtype || X_r->dtype != X->dtype) return ATP_ERR_INVALID_ARG;
    std::vector<SeqDims> sd;
    if ((st = check_seqs(seqs, sd, X->rows)) != ATP_OK) return st;
    int maxr = 0, total_rank = 0;
    for (auto &s : sd) { maxr = std::max(maxr, s.r); total_rank += s.r; if (s.r > X->cols) return ATP_ERR_INVALID_RANK; }
    if (U_r->rows != X->rows || U_r->cols < maxr || X_r->rows != total_rank || X_r->cols != X->cols ||
        V0->rows != total_rank || V0->cols != X->cols) return ATP_ERR_INVALID_ARG;
    if (X->rows == 0 || X->cols == 0) return ATP_OK;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    if (X->dtype == ATP_F32) return alternating_impl<float>(ctx, X, sd, V0, inner, U_r, X_r);
    return alternating_impl<__nv_bfloat16>(ctx, X, sd, V0, inner, U_r, X_r);
}

// ------------------------------------------------------------------------------------------------
// Eq. 4: mu = -log2(sum_i sbar_i^2), sbar_i = sigma_i / sum_j sigma_j; rank rule ceil(2^mu).
struct EntBatch { int off[ALT_MAX + 1]; int count; };
__global__ void __launch_bounds__(256) svd_entropy_kernel(const __grid_constant__ EntBatch batch, const float *sigma, float *mu, int *rank)
{
    __shared__ double red[8];
    const int b = blockIdx.x;
    const int lo = batch.off[b], hi = batch.off[b + 1];
    double p = 0.0;
    for (int i = lo + threadIdx.x; i < hi; i += 256) p += (double)sigma[i];
    const double tot = block_sum_256(p, red);
    p = 0.0;
    for (int i = lo + threadIdx.x; i < hi; i += 256) { const double s = (double)sigma[i] / tot; p += s * s; }
    const double acc = block_sum_256(p, red);
    if (threadIdx.x == 0) {
        const double m = (tot > 0.0 && acc > 0.0) ? -log2(acc) : 0.0;
        mu[b] = (float)m;
        if (rank) rank[b] = (tot > 0.0) ? (int)ceil(exp2(m) - 1e-9) : 0;
    }
}

extern "C" atp_status atp_svd_entropy(atp_ctx *ctx, const float *sigma, const int32_t *offsets, int32_t batch, float *mu,
                                      int32_t *rank)
{
    if (!ctx || batch < 0 || (batch > 0 && (!sigma || !offsets || !mu))) return ATP_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (offsets[b + 1] < offsets[b] || offsets[0] != 0) return ATP_ERR_INVALID_ARG;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    for (int b0 = 0; b0 < batch; b0 += ALT_MAX) {
        EntBatch eb; eb.count = std::min(ALT_MAX, batch - b0);
        for (int k = 0; k <= eb.count; ++k) eb.off[k] = offsets[b0 + k];
        ATP_KERNEL(ctx, "svd_entropy", 0, (double)(eb.off[eb.count] - eb.off[0]) * 8);
        svd_entropy_kernel<<<eb.count, 256, 0, ctx->stream>>>(eb, sigma, mu + b0, rank ? rank + b0 : nullptr);
        ATP_LAUNCHED(ctx);
    }
    return ATP_OK;
}
