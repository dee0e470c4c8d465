// Batched SIMT GEMM with fp32 accumulation: C = epilogue(op(A) * B). 64 x 64 x 32 tiles, the next
// tile prefetched into registers during the multiply.
//   A: M x K row-major (TRANS_A = false) or K x M row-major (TRANS_A = true)
//   B: K x N row-major (TRANS_B = false) or N x K row-major (TRANS_B = true)
//   C: M x N row-major,  D (optional addend / gate): M x N fp32
// Used by the fp32 path everywhere and by the small projections of the bf16 path.
#pragma once
#include "common.cuh"

struct GemmProblem {
    const void *A; const void *B; void *C; const float *D;
    int M, N, K;
    int lda, ldb, ldc, ldd;
};
constexpr int GEMM_MAX_BATCH = 32;
struct GemmBatch {
    GemmProblem p[GEMM_MAX_BATCH];
    int count;
};

enum GemmEpiKind {
    EPI_STORE = 0,        // C = A B
    EPI_D_MINUS = 1,      // C = D - A B
    EPI_BIAS = 2,         // C = A B + bias
    EPI_BIAS_GELU = 3,    // C = gelu_erf(A B + bias)
    EPI_SILU_D_MUL = 4    // C = silu(D) * (A B)
};
struct GemmEpi {
    int kind;
    const float *bias;    // N floats or nullptr
};

__device__ __forceinline__ float gelu_erf_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

template <typename TA, typename TB, typename TC, bool TRANS_A, bool TRANS_B>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const __grid_constant__ GemmBatch batch, GemmEpi epi, int splits, float *part, size_t part_stride)
{
    pdl_trigger();
    pdl_wait();
    const int z = blockIdx.z;
    const int pidx = z / splits, split = z - pidx * splits;
    const GemmProblem &pr = batch.p[pidx];
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    if (m0 >= pr.M || n0 >= pr.N) return;
    int kchunk = (pr.K + splits - 1) / splits;
    kchunk = (kchunk + 31) / 32 * 32;
    const int kb = split * kchunk;
    const int ke = min(pr.K, kb + kchunk);

    constexpr int BK = 32;                              // K tile; 8 elements of A and of B per thread
    __shared__ __align__(16) float As[BK][68];
    __shared__ __align__(16) float Bs[BK][68];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const TA *A = (const TA *)pr.A;
    const TB *B = (const TB *)pr.B;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    // the next tile travels from global memory into registers while the current one is multiplied
    float ra[8], rb[8];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = tid + i * 256;
            float va = 0.f, vb = 0.f;
            if (!TRANS_A) {
                const int m = e >> 5, k = e & 31;
                if (m0 + m < pr.M && k0 + k < ke) va = to_f32(A[(size_t)(m0 + m) * pr.lda + k0 + k]);
            } else {
                const int k = e >> 6, m = e & 63;
                if (m0 + m < pr.M && k0 + k < ke) va = to_f32(A[(size_t)(k0 + k) * pr.lda + m0 + m]);
            }
            if (!TRANS_B) {
                const int k = e >> 6, n = e & 63;
                if (n0 + n < pr.N && k0 + k < ke) vb = to_f32(B[(size_t)(k0 + k) * pr.ldb + n0 + n]);
            } else {
                const int n = e >> 5, k = e & 31;
                if (n0 + n < pr.N && k0 + k < ke) vb = to_f32(B[(size_t)(n0 + n) * pr.ldb + k0 + k]);
            }
            ra[i] = va; rb[i] = vb;
        }
    };
    if (kb < ke) fetch(kb);
    for (int k0 = kb; k0 < ke; k0 += BK) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = tid + i * 256;
            if (!TRANS_A) As[e & 31][e >> 5] = ra[i]; else As[e >> 6][e & 63] = ra[i];
            if (!TRANS_B) Bs[e >> 6][e & 63] = rb[i]; else Bs[e & 31][e >> 5] = rb[i];
        }
        __syncthreads();
        if (k0 + BK < ke) fetch(k0 + BK);
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float4 a = *(const float4 *)&As[k][ty * 4];
            float4 b = *(const float4 *)&Bs[k][tx * 4];
            float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

    if (splits > 1) {
        float *dst = part + ((size_t)split * batch.count + pidx) * part_stride;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int m = m0 + ty * 4 + i;
            if (m >= pr.M) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int n = n0 + tx * 4 + j;
                if (n < pr.N) dst[(size_t)m * pr.N + n] = acc[i][j];
            }
        }
        return;
    }
    TC *C = (TC *)pr.C;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= pr.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx * 4 + j;
            if (n >= pr.N) continue;
            float v = acc[i][j];
            switch (epi.kind) {
                case EPI_D_MINUS: v = pr.D[(size_t)m * pr.ldd + n] - v; break;
                case EPI_BIAS: if (epi.bias) v += epi.bias[n]; break;
                case EPI_BIAS_GELU: if (epi.bias) v += epi.bias[n]; v = gelu_erf_f(v); break;
                case EPI_SILU_D_MUL: v = silu_f(pr.D[(size_t)m * pr.ldd + n]) * v; break;
                default: break;
            }
            C[(size_t)m * pr.ldc + n] = from_f32<TC>(v);
        }
    }
}

// Sums split-K partials in a fixed order (deterministic) and stores C.
template <typename TC>
__global__ void __launch_bounds__(256)
gemm_splitk_reduce_kernel(const __grid_constant__ GemmBatch batch, int splits, const float *part, size_t part_stride)
{
    pdl_trigger();
    pdl_wait();
    const int pidx = blockIdx.y;
    const GemmProblem &pr = batch.p[pidx];
    size_t total = (size_t)pr.M * pr.N;
    TC *C = (TC *)pr.C;
    for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < total; e += (size_t)gridDim.x * 256) {
        float v = 0.f;
        for (int s = 0; s < splits; ++s) v += part[((size_t)s * batch.count + pidx) * part_stride + e];
        int m = (int)(e / pr.N), n = (int)(e - (size_t)m * pr.N);
        C[(size_t)m * pr.ldc + n] = from_f32<TC>(v);
    }
}

// Host launcher. `part` is scratch for split-K (splits * count * part_stride floats) or nullptr.
template <typename TA, typename TB, typename TC, bool TRANS_A, bool TRANS_B = false>
static atp_status launch_gemm_simt(atp_ctx *ctx, const GemmBatch &batch, GemmEpi epi, int splits = 1,
                                   float *part = nullptr, size_t part_stride = 0, const char *name = "gemm_simt")
{
    int maxM = 0, maxN = 0;
    for (int i = 0; i < batch.count; ++i) {
        if (batch.p[i].M > maxM) maxM = batch.p[i].M;
        if (batch.p[i].N > maxN) maxN = batch.p[i].N;
    }
    if (maxM == 0 || maxN == 0 || batch.count == 0) return ATP_OK;
    if (splits < 1 || !part) splits = 1;
    double flops = 0, bytes = 0;
    for (int i = 0; i < batch.count; ++i) {
        const GemmProblem &q = batch.p[i];
        flops += 2.0 * q.M * q.N * q.K;
        bytes += (double)q.M * q.K * sizeof(TA) + (double)q.K * q.N * sizeof(TB) + (double)q.M * q.N * sizeof(TC);
    }
    dim3 grid(ceil_div(maxN, 64), ceil_div(maxM, 64), batch.count * splits);
    ATP_KERNEL(ctx, name, flops, bytes);
    launch_pdl(gemm_simt_kernel<TA, TB, TC, TRANS_A, TRANS_B>, grid, dim3(256), 0, ctx->stream, batch, epi, splits, part, part_stride);
    ATP_LAUNCHED(ctx);
    if (splits > 1) {
        int blocks = ceil_div(maxM * maxN, 256);
        if (blocks > 1024) blocks = 1024;
        ATP_KERNEL(ctx, "gemm_splitk_reduce", 0, 0);
        launch_pdl(gemm_splitk_reduce_kernel<TC>, dim3(blocks, batch.count), dim3(256), 0, ctx->stream, batch, splits, (const float *)part, part_stride);
        ATP_LAUNCHED(ctx);
    }
    return ATP_OK;
}

// Runs `fn(batch)` over problems in chunks of GEMM_MAX_BATCH.
template <typename F>
static atp_status for_each_chunk(const std::vector<GemmProblem> &probs, F fn)
{
    for (size_t i = 0; i < probs.size(); i += GEMM_MAX_BATCH) {
        GemmBatch b;
        b.count = (int)((probs.size() - i < GEMM_MAX_BATCH) ? probs.size() - i : GEMM_MAX_BATCH);
        for (int j = 0; j < b.count; ++j) b.p[j] = probs[i + j];
        atp_status st = fn(b);
        if (st != ATP_OK) return st;
    }
    return ATP_OK;
}
