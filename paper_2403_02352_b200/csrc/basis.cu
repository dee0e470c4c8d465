// atp_principal_basis: top-r left singular vectors U_r and X_r = U_r^T X (Eq. 3, Eq. 5, Sec. 4.2),
// i.e. the minimiser of Eq. 9, computed as
//   1. randomised range finder  Y = X Omega  (+-1 test matrix) with subspace (power) iterations
//      Z = X^T Y, Y = orth(X Z); every iterate is orthonormalised by one persistent block Gram-Schmidt
//      kernel (orth.cuh: Cholesky-QR of every 64-column panel, Gram matrix and factor in fp64);
//   2. projection  B^T = X^T Y  (d x r~) and its Gram matrix G = B B^T (r~ x r~);
//   3. two-sided block Jacobi on G in two passes, one persistent kernel each (jacobi3.cuh): the
//      accumulated rotation turns Y into singular vectors and the rows of B into sigma_i v_i^T
//      (opts->jacobi_block = 1: one-sided block Jacobi on the rows of B instead, a launch chain);
//   4. sort by sigma, fix signs, write U_r = Y W and X_r = W^T B.
// This file holds the host flow, the finishing kernels and the one-sided variant.
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "jacobi3.cuh"
#include "orth.cuh"
#include <type_traits>
#include <math.h>
#include <algorithm>

constexpr int BJ = 32;            // Jacobi block height (pairs are 64 rows)
constexpr int BMAX = 32;          // sequences per launch

// ------------------------------------------------------------------------------------------------
__global__ void fill_omega_bf16_kernel(__nv_bfloat16 *om, int rows, int cols, int ld, uint64_t seed)
{
    size_t n = (size_t)rows * cols;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        int r = (int)(i / cols), c = (int)(i - (size_t)r * cols);
        om[(size_t)r * ld + c] = __float2bfloat16_rn((mix64(seed, i) & 1) ? 1.f : -1.f);
    }
}

__global__ void fill_omega_kernel(float *om, size_t n, uint64_t seed)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        om[i] = (mix64(seed, i) & 1) ? 1.f : -1.f;
}

// fp32 -> bf16 hi/lo pair (hi = bf16(x), lo = bf16(x - hi)) for every sequence of a batch.
struct SplitSeq { const float *src; __nv_bfloat16 *hi, *lo; int lds, ldd, rows, cols; };
struct SplitBatch { SplitSeq s[BMAX]; int count; };
__global__ void __launch_bounds__(256) split_bf16_batch_kernel(const __grid_constant__ SplitBatch batch)
{
    pdl_trigger();
    pdl_wait();
    const SplitSeq &q = batch.s[blockIdx.y];
    const size_t n = (size_t)q.rows * q.cols;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(e / q.cols), c = (int)(e - (size_t)r * q.cols);
        const float x = q.src[(size_t)r * q.lds + c];
        const __nv_bfloat16 h = __float2bfloat16_rn(x);
        q.hi[(size_t)r * q.ldd + c] = h;
        q.lo[(size_t)r * q.ldd + c] = __float2bfloat16_rn(x - __bfloat162float(h));
    }
}

// ------------------------------------------------------------------------------------------------
// One-sided block Jacobi on the rows of BW = [B | Wt] (r~ x (d + r~)); only the first d columns
// enter the inner products, all d + r~ columns are rotated.
struct JacSeq { float *BW; int rt, d, ld, nb; unsigned *maxoff; int *conv; };
struct JacBatch { JacSeq s[BMAX]; int count; };

__global__ void init_w_kernel(const __grid_constant__ JacBatch batch)
{
    const JacSeq &sq = batch.s[blockIdx.y];
    size_t n = (size_t)sq.rt * sq.rt;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        int i = (int)(e / sq.rt), k = (int)(e - (size_t)i * sq.rt);
        sq.BW[(size_t)i * sq.ld + sq.d + k] = (i == k) ? 1.f : 0.f;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { *sq.maxoff = 0u; *sq.conv = 0; }
}

__device__ __forceinline__ void rr_pair(int nb, int step, int t, int &I, int &J)
{
    // round-robin tournament of nb (even) players, round `step` in [0, nb-1), table t in [0, nb/2)
    int m = nb - 1;
    if (t == 0) { I = m; J = step % m; }
    else { I = (step + t) % m; J = (step - t + m) % m; }
    if (I > J) { int x = I; I = J; J = x; }
}

__global__ void __launch_bounds__(256)
jacobi_pair_kernel(const __grid_constant__ JacBatch batch, int step, float tol_rot, float tol_skip)
{
    const JacSeq &sq = batch.s[blockIdx.y];
    if (*sq.conv) return;
    const int npairs = sq.nb / 2;
    if ((int)blockIdx.x >= npairs) return;
    int I, J;
    rr_pair(sq.nb, step % (sq.nb - 1), blockIdx.x, I, J);
    __shared__ float G[64][65];
    __shared__ float Vt[64][65];
    __shared__ __align__(16) float St[32][68];     // phase 1: transposed column tile; phase 3: reused as input tile
    float (*Tl)[65] = G;                           // phase 3 input tile (G is dead by then)
    __shared__ float cs[32], sn[32];
    __shared__ int pp[32], qq[32];
    __shared__ float red[8];
    __shared__ int rotated;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    auto grow = [&](int i) -> int {     // global row of local row i, or -1
        int g = (i < 32) ? I * BJ + i : J * BJ + (i - 32);
        return (g < sq.rt) ? g : -1;
    };
    // ---- phase 1: G = S S^T over the first d columns (tile sums in fp32, running sum in fp64)
    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
    for (int c0 = 0; c0 < sq.d; c0 += 32) {
        for (int e = tid; e < 64 * 32; e += 256) {
            int row = e >> 5, c = e & 31;
            int g = grow(row);
            float v = 0.f;
            if (g >= 0 && c0 + c < sq.d) v = sq.BW[(size_t)g * sq.ld + c0 + c];
            St[c][row] = v;
        }
        __syncthreads();
        float part[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) part[i][j] = 0.f;
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
            float4 a = *(const float4 *)&St[c][ty * 4];
            float4 b = *(const float4 *)&St[c][tx * 4];
            float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) part[i][j] = fmaf(av[i], bv[j], part[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] += (double)part[i][j];
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            G[ty * 4 + i][tx * 4 + j] = (float)acc[i][j];
            Vt[ty * 4 + i][tx * 4 + j] = (ty * 4 + i == tx * 4 + j) ? 1.f : 0.f;
        }
    __syncthreads();
    // largest scaled off-diagonal entry of this pair
    float mo = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int a = ty * 4 + i, b = tx * 4 + j;
            if (a != b) {
                float den = sqrtf(G[a][a] * G[b][b]);
                if (den > 0.f) mo = fmaxf(mo, fabsf(G[a][b]) / den);
            }
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mo = fmaxf(mo, __shfl_xor_sync(0xffffffffu, mo, o));
    if ((tid & 31) == 0) red[tid >> 5] = mo;
    __syncthreads();
    mo = red[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) mo = fmaxf(mo, red[w]);
    if (tid == 0) atomicMax(sq.maxoff, __float_as_uint(mo));
    if (mo <= tol_skip) return;

    // ---- phase 2: diagonalise G by cyclic two-sided Jacobi, accumulating the row operations in Vt
    for (int sweep = 0; sweep < 12; ++sweep) {
        if (tid == 0) rotated = 0;
        __syncthreads();
        for (int st = 0; st < 63; ++st) {
            if (tid < 32) {
                int p, q;
                rr_pair(64, st, tid, p, q);
                float gpp = G[p][p], gqq = G[q][q], gpq = G[p][q];
                float c = 1.f, s = 0.f;
                if (fabsf(gpq) > tol_rot * sqrtf(gpp * gqq) && gpq != 0.f) {
                    float zeta = (gqq - gpp) / (2.f * gpq);
                    float t = copysignf(1.f, zeta) / (fabsf(zeta) + sqrtf(1.f + zeta * zeta));
                    c = 1.f / sqrtf(1.f + t * t);
                    s = c * t;
                    rotated = 1;
                }
                cs[tid] = c; sn[tid] = s; pp[tid] = p; qq[tid] = q;
            }
            __syncthreads();
            // G <- J^T G J on 2x2 blocks (row pair a, column pair b); Vt rows rotate like G rows
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                int idx = tid + it * 256;
                int a = idx >> 5, b = idx & 31;
                int pa = pp[a], qa = qq[a], pb_ = pp[b], qb = qq[b];
                float ca = cs[a], sa = sn[a], cb = cs[b], sb = sn[b];
                float g00 = G[pa][pb_], g01 = G[pa][qb], g10 = G[qa][pb_], g11 = G[qa][qb];
                float r00 = ca * g00 - sa * g10, r01 = ca * g01 - sa * g11;
                float r10 = sa * g00 + ca * g10, r11 = sa * g01 + ca * g11;
                G[pa][pb_] = cb * r00 - sb * r01; G[pa][qb] = sb * r00 + cb * r01;
                G[qa][pb_] = cb * r10 - sb * r11; G[qa][qb] = sb * r10 + cb * r11;
            }
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                int idx = tid + it * 256;
                int a = idx >> 6, col = idx & 63;
                int pa = pp[a], qa = qq[a];
                float ca = cs[a], sa = sn[a];
                float x = Vt[pa][col], y = Vt[qa][col];
                Vt[pa][col] = ca * x - sa * y;
                Vt[qa][col] = sa * x + ca * y;
            }
            __syncthreads();
        }
        if (!rotated) break;
        __syncthreads();
    }
    // ---- phase 3: rows <- Vt * rows over all d + r~ columns
    const int ncols = sq.d + sq.rt;
    for (int c0 = 0; c0 < ncols; c0 += 64) {
        for (int e = tid; e < 64 * 64; e += 256) {
            int row = e >> 6, c = e & 63;
            int g = grow(row);
            float v = 0.f;
            if (g >= 0 && c0 + c < ncols) v = sq.BW[(size_t)g * sq.ld + c0 + c];
            Tl[row][c] = v;
        }
        __syncthreads();
        float out[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) out[i][j] = 0.f;
        for (int k = 0; k < 64; ++k) {
            float bv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Tl[k][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float a = Vt[ty * 4 + i][k];
#pragma unroll
                for (int j = 0; j < 4; ++j) out[i][j] = fmaf(a, bv[j], out[i][j]);
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int g = grow(ty * 4 + i);
            if (g < 0) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int c = c0 + tx + 16 * j;
                if (c < ncols) sq.BW[(size_t)g * sq.ld + c] = out[i][j];
            }
        }
    }
}

// One block of BMAX threads; *all_conv = 1 when every sequence of the launch has converged.
__global__ void jacobi_sweep_end_kernel(const __grid_constant__ JacBatch batch, float tol_conv, int last, int *dev_status, int *all_conv)
{
    const int b = threadIdx.x;
    int done = 1;
    if (b < batch.count) {
        const JacSeq &sq = batch.s[b];
        if (!*sq.conv) {
            float mo = __uint_as_float(*sq.maxoff);
            if (mo <= tol_conv) *sq.conv = 1;
            else { done = 0; if (last) raise_status(dev_status, ATP_ERR_NOT_CONVERGED); }
        }
        *sq.maxoff = 0u;
    }
    done = __syncthreads_and(done);
    if (threadIdx.x == 0 && all_conv) *all_conv = done;
}

// ------------------------------------------------------------------------------------------------
struct FinSeq {
    const float *BW; const float *Y; float *sig; int *ord; float *tsum; float *Wsel;
    void *Xr; float *sigma_out; int rt, r, d, ld, L, ldy, ldxr;
};
struct FinBatch { FinSeq s[BMAX]; int count; };

// Row norms of B (= singular values) and their descending order. One CTA per sequence.
__global__ void __launch_bounds__(1024) sigma_sort_kernel(const __grid_constant__ FinBatch batch)
{
    const FinSeq &sq = batch.s[blockIdx.x];
    extern __shared__ float sh[];
    int npow = 1;
    while (npow < sq.rt) npow <<= 1;
    float *key = sh;
    int *idx = (int *)(sh + npow);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = warp; i < npow; i += 32) {
        float s = -1.f;
        if (i < sq.rt) {
            double acc = 0.0;
            float part = 0.f;
            for (int c = lane; c < sq.d; c += 32) { float v = sq.BW[(size_t)i * sq.ld + c]; part = fmaf(v, v, part); }
            acc = part;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            s = (float)sqrt(acc);
        }
        if (lane == 0) { key[i] = s; idx[i] = i; }
    }
    __syncthreads();
    for (int k = 2; k <= npow; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < npow; i += 1024) {
                int l = i ^ j;
                if (l > i) {
                    bool desc = ((i & k) == 0);
                    float ki = key[i], kl = key[l];
                    int ii = idx[i], il = idx[l];
                    bool i_first = (ki > kl) || (ki == kl && ii < il);   // order wanted in a descending run
                    if (desc ? !i_first : i_first) { key[i] = kl; key[l] = ki; idx[i] = il; idx[l] = ii; }
                }
            }
            __syncthreads();
        }
    for (int i = tid; i < sq.rt; i += 1024) { sq.sig[i] = key[i]; sq.ord[i] = idx[i]; }
}

// Column sums of Y (L x r~): t[k] = sum_l Y[l][k].
__global__ void colsum_kernel(const __grid_constant__ FinBatch batch)
{
    const FinSeq &sq = batch.s[blockIdx.y];
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= sq.rt) return;
    float s = 0.f;
    for (int l = 0; l < sq.L; ++l) s += sq.Y[(size_t)l * sq.ldy + k];
    sq.tsum[k] = s;
}

// One CTA per kept component: sign rule, then X_r row, Wsel column and sigma.
template <typename T>
__global__ void __launch_bounds__(256) select_kernel(const __grid_constant__ FinBatch batch)
{
    const FinSeq &sq = batch.s[blockIdx.y];
    const int a = blockIdx.x;
    if (a >= sq.r) return;
    const int i = sq.ord[a];
    const float *row = sq.BW + (size_t)i * sq.ld;
    __shared__ float redf[8];
    __shared__ int redi[8];
    __shared__ float sgn_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float s = 0.f;
    for (int k = tid; k < sq.rt; k += 256) s = fmaf(sq.tsum[k], row[sq.d + k], s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) redf[warp] = s;
    __syncthreads();
    if (tid == 0) {
        float tot = 0.f;
        for (int w = 0; w < 8; ++w) tot += redf[w];
        sgn_s = tot;
    }
    __syncthreads();
    float colsum = sgn_s;
    __syncthreads();
    float sgn;
    if (fabsf(colsum) >= 1e-6f * sqrtf((float)sq.L)) {
        sgn = colsum < 0.f ? -1.f : 1.f;
    } else {      // fall back to the largest-magnitude entry of the row (first one on ties)
        float best = -1.f; int bi = 0x7fffffff;
        for (int c = tid; c < sq.d; c += 256) {
            float v = fabsf(row[c]);
            if (v > best) { best = v; bi = c; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ob = __shfl_xor_sync(0xffffffffu, best, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
        }
        if (lane == 0) { redf[warp] = best; redi[warp] = bi; }
        __syncthreads();
        if (tid == 0) {
            float b = redf[0]; int bi2 = redi[0];
            for (int w = 1; w < 8; ++w)
                if (redf[w] > b || (redf[w] == b && redi[w] < bi2)) { b = redf[w]; bi2 = redi[w]; }
            sgn_s = (bi2 < sq.d && row[bi2] < 0.f) ? -1.f : 1.f;
        }
        __syncthreads();
        sgn = sgn_s;
    }
    T *xr = (T *)sq.Xr + (size_t)a * sq.ldxr;
    for (int c = tid; c < sq.d; c += 256) xr[c] = from_f32<T>(sgn * row[c]);
    for (int k = tid; k < sq.rt; k += 256) sq.Wsel[(size_t)k * sq.r + a] = sgn * row[sq.d + k];
    if (tid == 0 && sq.sigma_out) sq.sigma_out[a] = sq.sig[a];
}

// ---- finalisation of the two-sided path ----------------------------------------------------------
constexpr int COLSUM_SLABS = 16;
struct Fin2Seq {
    const float *G; const float *Wt; const float *Y; float *sig; int *ord; float *tsum; float *Wsel; int *needfix;
    void *Xr; void *U; float *sigma_out; int rt, r, d, L, ldy, ldxr, ldu, ldg;
    // bf16 inputs: Y is held as a hi/lo pair (leading dimension ldy), and Wsel is written as one (ldws)
    const __nv_bfloat16 *Yh, *Yl; __nv_bfloat16 *Wselh, *Wsell; int ldws;
    float *tpart;                 // COLSUM_SLABS x rt partial column sums
};
struct Fin2Batch { Fin2Seq s[BMAX]; int count; };

// sigma_i = sqrt(G_ii) and their descending order. One CTA per sequence.
__global__ void __launch_bounds__(1024) sigma_sort2_kernel(const __grid_constant__ Fin2Batch batch)
{
    const Fin2Seq &sq = batch.s[blockIdx.x];
    extern __shared__ float sh[];
    int npow = 1;
    while (npow < sq.rt) npow <<= 1;
    float *key = sh;
    int *idx = (int *)(sh + npow);
    const int tid = threadIdx.x;
    for (int k = tid; k < sq.rt; k += 1024) {       // column sums of Y from the slab sums, fixed order
        float t = 0.f;
        for (int sl = 0; sl < COLSUM_SLABS; ++sl) t += sq.tpart[(size_t)sl * sq.rt + k];
        sq.tsum[k] = t;
    }
    for (int i = tid; i < npow; i += 1024) {
        key[i] = (i < sq.rt) ? sqrtf(fmaxf(sq.G[(size_t)i * sq.ldg + i], 0.f)) : -1.f;
        idx[i] = i;
    }
    __syncthreads();
    for (int k = 2; k <= npow; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < npow; i += 1024) {
                int l = i ^ j;
                if (l > i) {
                    bool desc = ((i & k) == 0);
                    float ki = key[i], kl = key[l];
                    int ii = idx[i], il = idx[l];
                    bool i_first = (ki > kl) || (ki == kl && ii < il);
                    if (desc ? !i_first : i_first) { key[i] = kl; key[l] = ki; idx[i] = il; idx[l] = ii; }
                }
            }
            __syncthreads();
        }
    for (int i = tid; i < sq.rt; i += 1024) { sq.sig[i] = key[i]; sq.ord[i] = idx[i]; }
}

// Column sums of Y (L x r~): t[k] = sum_l Y[l][k]. grid (column chunks of 32, row slabs, batch); 8 warps of a
// CTA take interleaved rows of the slab, lanes take columns; the slab sums go to tpart and are added up in a
// fixed order by sigma_sort2_kernel (same result on every run).
__global__ void __launch_bounds__(256) colsum2_kernel(const __grid_constant__ Fin2Batch batch)
{
    const Fin2Seq &sq = batch.s[blockIdx.z];
    const int k = blockIdx.x * 32 + (threadIdx.x & 31), w = threadIdx.x >> 5;
    const int rows = (sq.L + COLSUM_SLABS - 1) / COLSUM_SLABS, l0 = blockIdx.y * rows, l1 = min(sq.L, l0 + rows);
    float s = 0.f;
    if (k < sq.rt) {
        if (sq.Yh) for (int l = l0 + w; l < l1; l += 8) s += __bfloat162float(sq.Yh[(size_t)l * sq.ldy + k]) + __bfloat162float(sq.Yl[(size_t)l * sq.ldy + k]);
        else for (int l = l0 + w; l < l1; l += 8) s += sq.Y[(size_t)l * sq.ldy + k];
    }
    __shared__ float part[8][33];
    part[w][threadIdx.x & 31] = s;
    __syncthreads();
    if (w == 0 && k < sq.rt) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) t += part[i][threadIdx.x];
        sq.tpart[(size_t)blockIdx.y * sq.rt + k] = t;
    }
}

// One CTA per kept component: sign from the column sum of U (= tsum . w), Wsel column, sigma.
__global__ void __launch_bounds__(128) select2_kernel(const __grid_constant__ Fin2Batch batch)
{
    const Fin2Seq &sq = batch.s[blockIdx.y];
    const int a = blockIdx.x;
    if (a >= sq.r) return;
    const int i = sq.ord[a];
    const float *w = sq.Wt + (size_t)i * sq.ldg;
    __shared__ float redf[4];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float s = 0.f;
    for (int k = tid; k < sq.rt; k += 128) s = fmaf(sq.tsum[k], w[k], s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) redf[warp] = s;
    __syncthreads();
    float colsum = redf[0] + redf[1] + redf[2] + redf[3];
    float sgn = colsum < 0.f ? -1.f : 1.f;
    if (sq.Wselh) {
        for (int k = tid; k < sq.rt; k += 128) {
            const float v = sgn * w[k];
            const __nv_bfloat16 h = __float2bfloat16_rn(v);
            sq.Wselh[(size_t)k * sq.ldws + a] = h;
            sq.Wsell[(size_t)k * sq.ldws + a] = __float2bfloat16_rn(v - __bfloat162float(h));
        }
    } else {
        for (int k = tid; k < sq.rt; k += 128) sq.Wsel[(size_t)k * sq.r + a] = sgn * w[k];
    }
    if (tid == 0) {
        sq.needfix[a] = fabsf(colsum) < 1e-6f * sqrtf((float)sq.L);
        if (sq.sigma_out) sq.sigma_out[a] = sq.sig[a];
    }
}

// Components whose column sum is ~0 take their sign from the largest-magnitude entry of the X_r row.
template <typename T>
__global__ void __launch_bounds__(256) signfix_kernel(const __grid_constant__ Fin2Batch batch)
{
    const Fin2Seq &sq = batch.s[blockIdx.y];
    const int a = blockIdx.x;
    if (a >= sq.r || !sq.needfix[a]) return;
    T *row = (T *)sq.Xr + (size_t)a * sq.ldxr;
    __shared__ float redf[8];
    __shared__ int redi[8];
    __shared__ int flip;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float best = -1.f; int bi = 0x7fffffff;
    for (int c = tid; c < sq.d; c += 256) {
        float v = fabsf(to_f32(row[c]));
        if (v > best) { best = v; bi = c; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ob = __shfl_xor_sync(0xffffffffu, best, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    if (lane == 0) { redf[warp] = best; redi[warp] = bi; }
    __syncthreads();
    if (tid == 0) {
        float b = redf[0]; int b2 = redi[0];
        for (int w = 1; w < 8; ++w)
            if (redf[w] > b || (redf[w] == b && redi[w] < b2)) { b = redf[w]; b2 = redi[w]; }
        flip = (b2 < sq.d && to_f32(row[b2]) < 0.f);
    }
    __syncthreads();
    if (!flip) return;
    for (int c = tid; c < sq.d; c += 256) row[c] = from_f32<T>(-to_f32(row[c]));
    T *u = (T *)sq.U + a;
    for (int l = tid; l < sq.L; l += 256) u[(size_t)l * sq.ldu] = from_f32<T>(-to_f32(u[(size_t)l * sq.ldu]));
}

// ------------------------------------------------------------------------------------------------
struct SeqPlan {
    SeqDims dims; int rt, np, npanel_L, npanel_d; unsigned *jsync; float *tpart;
    __nv_bfloat16 *Bth, *Btl, *Y2h, *Y2l, *Wth, *Wtl, *Wsh, *Wsl;
    float *oCpart, *oC, *oDpart, *oW; double *ogpart, *ogpart2; unsigned *osync; int ocap;
    __nv_bfloat16 *Yb, *Yl, *Zb, *Zl; float *Y2; float *Y, *Z, *BW, *Wsel, *tsum, *sig, *Cc, *rinv, *G, *Wt, *Vbuf; double *gpart; int *ord, *flags, *conv, *vflag, *needfix; unsigned *maxoff;
};
struct BasisPlan {
    std::vector<SeqPlan> seqs; float *omega; __nv_bfloat16 *omega_b; float *part; size_t part_stride, part_group; int group = 0; int rtmax; int splits;
};

// Size of the Jacobi matrices: rt rounded up to a whole number of 64-row block pairs.
static int jacobi_padded(int rt) { return rt <= 0 ? 0 : (rt + 63) / 64 * 64; }

static void plan_basis(Arena &ar, const std::vector<SeqDims> &sd, int d, int oversample, int sm_count, BasisPlan &bp)
{
    bp.seqs.clear(); bp.rtmax = 0;
    int maxdim = d; size_t maxpart = 0;
    for (auto &s : sd) {
        SeqPlan p; p.dims = s;
        int m = std::min(s.L, d);
        p.rt = std::min(m, s.r + oversample);
        if (s.L == 0) p.rt = 0;
        bp.rtmax = std::max(bp.rtmax, p.rt);
        maxdim = std::max(maxdim, s.L);
        bp.seqs.push_back(p);
    }
    bp.omega = ar.take<float>((size_t)d * bp.rtmax);
    bp.omega_b = ar.take<__nv_bfloat16>((size_t)d * align_up((size_t)bp.rtmax, 8));
    for (auto &p : bp.seqs) {
        int L = p.dims.L, rt = p.rt;
        p.Y = ar.take<float>((size_t)L * rt);
        p.Z = ar.take<float>((size_t)d * rt);
        p.Yb = ar.take<__nv_bfloat16>((size_t)L * align_up((size_t)rt, 8));
        p.Yl = ar.take<__nv_bfloat16>((size_t)L * align_up((size_t)rt, 8));
        p.Zb = ar.take<__nv_bfloat16>((size_t)d * align_up((size_t)rt, 8));
        p.Zl = ar.take<__nv_bfloat16>((size_t)d * align_up((size_t)rt, 8));
        p.Y2 = ar.take<float>((size_t)L * rt);
        p.BW = ar.take<float>((size_t)rt * (d + rt));
        p.Wsel = ar.take<float>((size_t)rt * p.dims.r);
        p.tsum = ar.take<float>(rt);
        p.sig = ar.take<float>(rt);
        p.ord = ar.take<int>(rt);
        {   // tile scratch of the orthonormalisation kernel
            p.ocap = orth::max_ctas_per_seq(sm_count, (int)std::min<size_t>(sd.size(), BMAX));
            const orth::Scratch sc = orth::scratch_tiles(L, rt, p.ocap);
            p.oCpart = ar.take<float>(sc.cpart * 4096); p.oC = ar.take<float>(sc.c * 4096);
            p.oDpart = ar.take<float>(sc.dpart * 4096); p.oW = ar.take<float>(4096);
            p.ogpart = ar.take<double>(sc.gpart * 4096); p.ogpart2 = ar.take<double>((size_t)orth::NRED * 4096);
            p.flags = ar.take<int>(64); p.osync = ar.take<unsigned>(64 + (size_t)p.ocap);
        }
        p.np = jacobi_padded(rt);
        p.G = ar.take<float>((size_t)p.np * p.np);
        p.Wt = ar.take<float>((size_t)p.np * p.np);
        p.Vbuf = ar.take<float>((size_t)2 * (p.np / 64 + 1) * 4096);
        p.vflag = ar.take<int>(2 * (p.np / 64) + 4);
        p.tpart = ar.take<float>((size_t)COLSUM_SLABS * std::max(rt, 1));
        {   // bf16 hi/lo operands of the tensor-core products around the rotation (bf16 inputs only)
            const size_t ldr = align_up((size_t)std::max(rt, 1), 8), ldw = align_up((size_t)std::max(p.dims.r, 1), 8);
            p.Bth = ar.take<__nv_bfloat16>((size_t)d * ldr); p.Btl = ar.take<__nv_bfloat16>((size_t)d * ldr);
            p.Y2h = ar.take<__nv_bfloat16>((size_t)L * ldr); p.Y2l = ar.take<__nv_bfloat16>((size_t)L * ldr);
            p.Wth = ar.take<__nv_bfloat16>((size_t)p.np * p.np); p.Wtl = ar.take<__nv_bfloat16>((size_t)p.np * p.np);
            p.Wsh = ar.take<__nv_bfloat16>((size_t)std::max(rt, 1) * ldw); p.Wsl = ar.take<__nv_bfloat16>((size_t)std::max(rt, 1) * ldw);
        }
        p.jsync = ar.take<unsigned>(64);
        p.needfix = ar.take<int>(std::max(p.dims.r, 1));
        p.maxoff = ar.take<unsigned>(1);
        p.conv = ar.take<int>(1);
        maxpart = std::max(maxpart, (size_t)rt * PB);
    }
}

size_t basis_workspace_bytes(const std::vector<SeqDims> &sd, int d, int oversample, int sm_count)
{
    Arena ar(nullptr, (size_t)-1);
    BasisPlan bp;
    plan_basis(ar, sd, d, oversample, sm_count, bp);
    return ar.off;
}

// Orthonormalise the columns of Y_b (L_b x rt_b, ld = rt_b) for the sequences [i0, i1): one persistent kernel
// (orth.cuh). reps: Gram-Schmidt repetitions per panel; two give orthonormality to working precision and repair
// dependent columns. With TENSOR the finished columns also go out as the bf16 hi/lo pair (Yb, Yl).
template <bool TENSOR>
static atp_status orthonormalise(atp_ctx *ctx, BasisPlan &bp, size_t i0, size_t i1, uint64_t seed, int reps)
{
    orth::Batch ob; ob.count = (int)(i1 - i0);
    for (size_t i = i0; i < i1; ++i) {
        SeqPlan &p = bp.seqs[i];
        ob.s[i - i0] = orth::Seq{p.Y, p.dims.L, p.rt, p.rt, TENSOR ? p.Yb : nullptr, TENSOR ? p.Yl : nullptr,
                                 (int)align_up((size_t)std::max(p.rt, 1), 8), p.oCpart, p.oC, p.oDpart, p.oW, p.ogpart, p.ogpart2,
                                 p.flags, p.osync, 0, p.ocap, 0};
    }
    return orth::launch<TENSOR>(ctx, ob, reps, seed);
}

template <typename T>
static atp_status basis_impl(atp_ctx *ctx, const atp_mat *X, const std::vector<SeqDims> &sd, int oversample,
                             int power_iters, int max_sweeps, uint64_t seed, int jbj, int jinner, int groups, bool no_host_sync, atp_mat *U_r, atp_mat *X_r, float *sigma)
{
    const int d = (int)X->cols;
    Arena ar(ctx->workspace, ctx->workspace_bytes);
    BasisPlan bp;
    plan_basis(ar, sd, d, oversample, ctx->sm_count, bp);
    if (ar.overflow || !ctx->workspace) return ATP_ERR_WORKSPACE_TOO_SMALL;
    atp_status st;
    if (X->dtype == ATP_BF16) {
        ATP_KERNEL(ctx, "fill_omega", 0, 0);
        fill_omega_bf16_kernel<<<1024, 256, 0, ctx->stream>>>(bp.omega_b, d, bp.rtmax, (int)align_up((size_t)bp.rtmax, 8), seed);
        ATP_LAUNCHED(ctx);
    } else {
        size_t n = (size_t)d * bp.rtmax;
        ATP_KERNEL(ctx, "fill_omega", 0, 0);
        fill_omega_kernel<<<(unsigned)std::min<size_t>((n + 255) / 256, 4096), 256, 0, ctx->stream>>>(bp.omega, n, seed);
        ATP_LAUNCHED(ctx);
    }
    const float tol_conv = (X->dtype == ATP_F32) ? 1e-6f : 3e-4f;
    const float tol_rot = tol_conv * 0.25f;
    const bool two_sided = jbj != 1;    // jacobi_block = 1 selects the one-sided rotation of B itself
    GemmEpi store{EPI_STORE, nullptr};

    // The chains below are many small dependent launches (latency-bound). On request (groups = 2) the
    // batch is cut in two groups that run on the context's two auxiliary streams, forked from and
    // joined back into the caller's stream. Measured: no gain at batch 16 (the chain length, not the
    // occupancy, sets the time, and the launch count doubles), so it is off by default.
    const size_t nseq = bp.seqs.size();
    const bool forked = groups == 2 && nseq >= 2 && ctx->aux[0] && ctx->aux[1] && !ctx->profiling;
    const size_t gsz = forked ? std::min<size_t>(BMAX, (nseq + 1) / 2) : BMAX;
    // reading the convergence flags back lets the host stop enqueueing sweeps; without it (forked streams, or on
    // request: stream capture, callers that must never block) the whole sweep budget is enqueued and the kernels
    // of converged sequences return at once
    const bool hsync = !forked && !no_host_sync;
    struct StreamGuard {
        atp_ctx *c; cudaStream_t saved;
        ~StreamGuard() { c->stream = saved; }
    } guard{ctx, ctx->stream};
    const cudaStream_t main_stream = ctx->stream;
    if (forked) {
        ATP_CUDA_OK(ctx, cudaEventRecord(ctx->ev_fork, main_stream));
        for (int gq = 0; gq < 2; ++gq) ATP_CUDA_OK(ctx, cudaStreamWaitEvent(ctx->aux[gq], ctx->ev_fork, 0));
    }
    for (size_t i0 = 0; i0 < nseq; i0 += gsz) {
        const size_t i1 = std::min(nseq, i0 + gsz);
        const int cnt = (int)(i1 - i0);
        bp.group = forked ? (int)((i0 / gsz) & 1) : 0;
        if (forked) ctx->stream = ctx->aux[bp.group];
        auto Xb = [&](const SeqPlan &p) { return (const T *)X->data + (size_t)p.dims.row0 * X->ld; };
        GemmBatch g; g.count = cnt;
        if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            // bf16: every pass over X is a tensor-core GEMM with fp32 results; the iterates are
            // orthonormalised in fp32 and handed to the next pass as bf16 copies.
            const int ldo = (int)align_up((size_t)bp.rtmax, 8);
            // The orthonormal iterate goes to the next pass as a bf16 hi/lo pair (about 16 mantissa
            // bits, written by the orthonormalisation kernel): a single bf16 rounding of Y would leak
            // sigma_1 * 2^-9 / sqrt(L) of the leading direction into every column and bury directions
            // that are 10^3..10^4 times weaker.
            std::vector<tc::HostProblem> hp;
            for (size_t i = i0; i < i1; ++i) {
                SeqPlan &p = bp.seqs[i];
                hp.push_back(tc::HostProblem{Xb(p), bp.omega_b, nullptr, p.Y, nullptr, nullptr, p.dims.L, p.rt, d, (int)X->ld, ldo, p.rt, 0});
            }
            if ((st = tc::launch<false, false, tc::OUT_F32>(ctx, hp, store)) != ATP_OK) return st;
            if ((st = orthonormalise<std::is_same<T, __nv_bfloat16>::value>(ctx, bp, i0, i1, seed, 2)) != ATP_OK) return st;
            for (int it = 0; it < power_iters; ++it) {
                hp.clear();
                for (size_t i = i0; i < i1; ++i) {      // Z = X^T Y, kept as a bf16 hi/lo pair (only the next pass reads it)
                    SeqPlan &p = bp.seqs[i];
                    int ldb = (int)align_up((size_t)p.rt, 8);
                    hp.push_back(tc::HostProblem{Xb(p), p.Yb, p.Yl, p.Zb, p.Zl, nullptr, d, p.rt, p.dims.L, (int)X->ld, ldb, ldb, 0});
                }
                if ((st = tc::launch<true, true, tc::OUT_BF16_SPLIT>(ctx, hp, store)) != ATP_OK) return st;
                hp.clear();
                for (size_t i = i0; i < i1; ++i) {      // Y = X Z
                    SeqPlan &p = bp.seqs[i];
                    int ldb = (int)align_up((size_t)p.rt, 8);
                    hp.push_back(tc::HostProblem{Xb(p), p.Zb, p.Zl, p.Y, nullptr, nullptr, p.dims.L, p.rt, d, (int)X->ld, ldb, p.rt, 0});
                }
                if ((st = tc::launch<false, true, tc::OUT_F32>(ctx, hp, store)) != ATP_OK) return st;
                if ((st = orthonormalise<std::is_same<T, __nv_bfloat16>::value>(ctx, bp, i0, i1, seed + 2000003ull * (it + 1), 2)) != ATP_OK) return st;
                }
        } else {
            // Y = X Omega
            for (size_t i = i0; i < i1; ++i) {
                SeqPlan &p = bp.seqs[i];
                g.p[i - i0] = GemmProblem{Xb(p), bp.omega, p.Y, nullptr, p.dims.L, p.rt, d, (int)X->ld, bp.rtmax, p.rt, 0};
            }
            if ((st = launch_gemm_simt<T, float, float, false>(ctx, g, store)) != ATP_OK) return st;
            if ((st = orthonormalise<std::is_same<T, __nv_bfloat16>::value>(ctx, bp, i0, i1, seed, 2)) != ATP_OK) return st;
            for (int it = 0; it < power_iters; ++it) {
                // Z = X^T Y ; Y = X Z ; orth(Y).  Z is not orthonormalised: Y has orthonormal, QR-ordered
                // columns, so cond(Z) ~ sigma_1 / sigma_r~ and cond(X Z) is its square, which the fp64
                // panel factorisation of orth(Y) handles.
                for (size_t i = i0; i < i1; ++i) {
                    SeqPlan &p = bp.seqs[i];
                    g.p[i - i0] = GemmProblem{Xb(p), p.Y, p.Z, nullptr, p.rt > 0 ? d : 0, p.rt, p.dims.L, (int)X->ld, p.rt, p.rt, 0};
                }
                if ((st = launch_gemm_simt<T, float, float, true>(ctx, g, store)) != ATP_OK) return st;
                for (size_t i = i0; i < i1; ++i) {
                    SeqPlan &p = bp.seqs[i];
                    g.p[i - i0] = GemmProblem{Xb(p), p.Z, p.Y, nullptr, p.dims.L, p.rt, d, (int)X->ld, p.rt, p.rt, 0};
                }
                if ((st = launch_gemm_simt<T, float, float, false>(ctx, g, store)) != ATP_OK) return st;
                if ((st = orthonormalise<std::is_same<T, __nv_bfloat16>::value>(ctx, bp, i0, i1, seed + 2000003ull * (it + 1), 2)) != ATP_OK) return st;
            }
        }
        if (!two_sided) {
            // B = Y^T X into BW[:, :d]; Wt = I
            JacBatch jb; jb.count = cnt; FinBatch fb; fb.count = cnt;
            int maxnb = 2, maxrt = 0, maxr = 0;
            for (size_t i = i0; i < i1; ++i) {
                SeqPlan &p = bp.seqs[i];
                int k = (int)(i - i0);
                g.p[k] = GemmProblem{p.Y, Xb(p), p.BW, nullptr, p.rt, p.rt > 0 ? d : 0, p.dims.L, p.rt, (int)X->ld, d + p.rt, 0};
                int nb = ceil_div(std::max(p.rt, 1), BJ); nb += nb & 1;
                jb.s[k] = JacSeq{p.BW, p.rt, d, d + p.rt, nb, p.maxoff, p.conv};
                fb.s[k] = FinSeq{p.BW, p.Y, p.sig, p.ord, p.tsum, p.Wsel,
                                 (T *)X_r->data + (size_t)p.dims.rank0 * X_r->ld, sigma ? sigma + p.dims.rank0 : nullptr,
                                 p.rt, p.dims.r, d, d + p.rt, p.dims.L, p.rt, (int)X_r->ld};
                maxnb = std::max(maxnb, nb); maxrt = std::max(maxrt, p.rt); maxr = std::max(maxr, p.dims.r);
            }
            if (maxrt == 0) continue;
            if ((st = launch_gemm_simt<float, T, float, true>(ctx, g, store)) != ATP_OK) return st;
            ATP_KERNEL(ctx, "init_w", 0, 0);
            init_w_kernel<<<dim3(64, cnt), 256, 0, ctx->stream>>>(jb);
            ATP_LAUNCHED(ctx);
            for (int sw = 0; sw < max_sweeps; ++sw) {
                if (sw >= 2 && hsync) {      // host stays at most two sweeps ahead; stop once converged
                    const int slot = (sw - 2) & 3;
                    ATP_CUDA_OK(ctx, cudaEventSynchronize(ctx->ev_flag[slot]));
                    if (ctx->h_flags[slot]) break;
                }
                for (int step = 0; step < maxnb - 1; ++step) {
                    ATP_KERNEL(ctx, "jacobi_pair", 0, 0);
                    jacobi_pair_kernel<<<dim3(maxnb / 2, cnt), 256, 0, ctx->stream>>>(jb, step, tol_rot, tol_rot);
                    ATP_LAUNCHED(ctx);
                }
                ATP_KERNEL(ctx, "jacobi_sweep_end", 0, 0);
                jacobi_sweep_end_kernel<<<1, BMAX, 0, ctx->stream>>>(jb, tol_conv, sw == max_sweeps - 1, ctx->dev_status,
                                                                     ctx->d_flags + (sw & 3));
                ATP_LAUNCHED(ctx);
                if (hsync) {
                    ATP_CUDA_OK(ctx, cudaMemcpyAsync(ctx->h_flags + (sw & 3), ctx->d_flags + (sw & 3), sizeof(int),
                                                     cudaMemcpyDeviceToHost, ctx->stream));
                    ATP_CUDA_OK(ctx, cudaEventRecord(ctx->ev_flag[sw & 3], ctx->stream));
                }
            }
            int npow = 1; while (npow < maxrt) npow <<= 1;
            size_t sm = (size_t)npow * 8;
            if (sm > 48 * 1024) ATP_CUDA_OK(ctx, cudaFuncSetAttribute(sigma_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm));
            ATP_KERNEL(ctx, "sigma_sort", 0, 0);
            sigma_sort_kernel<<<cnt, 1024, sm, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
            ATP_KERNEL(ctx, "colsum", 0, 0);
            colsum_kernel<<<dim3(ceil_div(maxrt, 128), cnt), 128, 0, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
            ATP_KERNEL(ctx, "select", 0, 0);
            select_kernel<T><<<dim3(maxr, cnt), 256, 0, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
            // U_r = Y Wsel
            for (size_t i = i0; i < i1; ++i) {
                SeqPlan &p = bp.seqs[i];
                g.p[i - i0] = GemmProblem{p.Y, p.Wsel, (T *)U_r->data + (size_t)p.dims.row0 * U_r->ld, nullptr,
                                          p.dims.L, p.dims.r, p.rt, p.rt, p.dims.r, (int)U_r->ld, 0};
            }
            if ((st = launch_gemm_simt<float, float, T, false>(ctx, g, store)) != ATP_OK) return st;
    
        } else {
            // Bt = X^T Y (d x r~, i.e. B^T), G = Bt^T Bt, two-sided block Jacobi on G, then
            // X_r = Wsel^T Bt^T and U_r = Y Wsel
            constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
            j3::Batch jb; jb.count = cnt; Fin2Batch fb; fb.count = cnt;
            GemmBatch gg; gg.count = cnt;
            int maxrt = 0, maxr = 0, maxL = 0;
            for (size_t i = i0; i < i1; ++i) {
                SeqPlan &p = bp.seqs[i];
                int k = (int)(i - i0);
                const int ldr = (int)align_up((size_t)std::max(p.rt, 1), 8), ldw = (int)align_up((size_t)std::max(p.dims.r, 1), 8);
                g.p[k] = GemmProblem{Xb(p), p.Y, p.BW, nullptr, p.rt > 0 ? d : 0, p.rt, p.dims.L, (int)X->ld, p.rt, p.rt, 0};
                gg.p[k] = GemmProblem{p.BW, p.BW, p.G, nullptr, p.rt, p.rt, p.rt > 0 ? d : 0, p.rt, p.rt, p.np, 0};
                jb.s[k] = j3::Seq{p.G, p.Wt, p.Vbuf, p.vflag, p.jsync, p.rt, p.np, p.np / j3::JB, 0, 0};
                fb.s[k] = Fin2Seq{p.G, p.Wt, p.Y, p.sig, p.ord, p.tsum, p.Wsel, p.needfix,
                                  (T *)X_r->data + (size_t)p.dims.rank0 * X_r->ld, (T *)U_r->data + (size_t)p.dims.row0 * U_r->ld,
                                  sigma ? sigma + p.dims.rank0 : nullptr, p.rt, p.dims.r, d, p.dims.L, kBf16 ? ldr : p.rt, (int)X_r->ld, (int)U_r->ld, p.np,
                                  nullptr, nullptr, kBf16 ? p.Wsh : nullptr, kBf16 ? p.Wsl : nullptr, ldw, p.tpart};
                maxrt = std::max(maxrt, p.rt); maxr = std::max(maxr, p.dims.r); maxL = std::max(maxL, p.dims.L);
            }
            if (maxrt == 0) continue;
            // bf16 inputs: every product around the rotation runs on the tensor cores with both operands cut
            // into bf16 hi/lo pairs (three MMA products, about 16 mantissa bits per operand); the projected
            // rows Bt, the rotated Bt2 / Y2 and the selected rotation Wsel only ever exist as such pairs.
            // fp32 inputs: the same products on the fp32 units.
            std::vector<tc::HostProblem> hp;
            if constexpr (kBf16) {
                for (size_t i = i0; i < i1; ++i) {      // Bt = X^T (Yb + Yl), d x r~, kept as hi/lo
                    SeqPlan &p = bp.seqs[i];
                    int ldb = (int)align_up((size_t)p.rt, 8);
                    hp.push_back(tc::HostProblem{Xb(p), p.Yb, p.Yl, p.Bth, p.Btl, nullptr, d, p.rt, p.dims.L, (int)X->ld, ldb, ldb, 0});
                }
                if ((st = tc::launch<true, true, tc::OUT_BF16_SPLIT>(ctx, hp, store)) != ATP_OK) return st;
            } else {
                if ((st = launch_gemm_simt<T, float, float, true>(ctx, g, store)) != ATP_OK) return st;
            }
            // Two passes. G squares the condition number of B, so when sigma_1 / sigma_r~ exceeds ~10^3
            // the first diagonalisation resolves the weak components only roughly. Its rotation W1 is
            // orthogonal all the same, so (Bt, Y) <- (Bt W1, Y W1) loses nothing; the rotated rows are
            // graded and nearly orthogonal, their Gram matrix carries errors relative to the row norms,
            // and a short second pass on it finishes the job (a one-sided Jacobi in two strokes).
            // Each pass is one persistent kernel that stops on its own convergence test: nothing is
            // read back by the host.
            for (int pass = 0; pass < 2; ++pass) {
                if constexpr (kBf16) {
                    hp.clear();
                    for (size_t i = i0; i < i1; ++i) {  // G = Bt^T Bt
                        SeqPlan &p = bp.seqs[i];
                        int ldb = (int)align_up((size_t)p.rt, 8);
                        const __nv_bfloat16 *bh = pass == 0 ? p.Bth : p.Zb, *bl = pass == 0 ? p.Btl : p.Zl;
                        tc::HostProblem h{bh, bh, bl, p.G, nullptr, nullptr, p.rt, p.rt, d, ldb, ldb, p.np, 0};
                        h.A2 = bl;
                        hp.push_back(h);
                    }
                    if ((st = tc::launch<true, true, tc::OUT_F32, false, true>(ctx, hp, store, "gemm_tc_gram")) != ATP_OK) return st;
                } else {
                    if ((st = launch_gemm_simt<float, float, float, true, false>(ctx, gg, store, 1, nullptr, 0, "gemm_simt_gram")) != ATP_OK) return st;
                }
                // pass 0 only has to make the rows graded and roughly orthogonal (scaled off-diagonals below
                // 1e-2; on ill-conditioned input it stalls at the noise floor of G, hence the cap of 8 sweeps);
                // the second pass continues the same iteration on the rotated data with the rest of the budget
                const int nsw0 = std::min(8, (max_sweeps + 1) / 2);
                const int nsw = pass == 0 ? nsw0 : std::max(1, max_sweeps - nsw0);
                const float tolc = pass == 0 ? fmaxf(tol_conv, 1e-2f) : tol_conv;
                // fp32 inputs: the block products stay on the fp32 units (the threshold is below split-precision rounding)
                if ((st = j3::launch<kBf16>(ctx, jb, tolc, tolc * 0.1f, nsw, pass == 1)) != ATP_OK) return st;
                if (pass == 0) {
                    // Bt2 = Bt Wt^T (d x r~),  Y2 = Y Wt^T (L x r~);  Wt rows are the eigenvectors
                    if constexpr (kBf16) {
                        SplitBatch sb; sb.count = cnt;
                        double bytes = 0; int maxel = 0;
                        for (size_t i = i0; i < i1; ++i) {
                            SeqPlan &p = bp.seqs[i];
                            sb.s[i - i0] = SplitSeq{p.Wt, p.Wth, p.Wtl, p.np, p.np, p.rt, p.rt};
                            bytes += (double)p.rt * p.rt * 8; maxel = std::max(maxel, p.rt * p.rt);
                        }
                        ATP_KERNEL(ctx, "f32_to_bf16", 0, bytes);
                        launch_pdl(split_bf16_batch_kernel, dim3(std::min(256, ceil_div(maxel, 1024)), sb.count), dim3(256), 0, ctx->stream, sb);
                        ATP_LAUNCHED(ctx);
                        std::vector<tc::HostProblem> h1, h2;
                        for (size_t i = i0; i < i1; ++i) {
                            SeqPlan &p = bp.seqs[i];
                            int ldb = (int)align_up((size_t)p.rt, 8);
                            tc::HostProblem a{p.Bth, p.Wth, p.Wtl, p.Zb, p.Zl, nullptr, d, p.rt, p.rt, ldb, p.np, ldb, 0};
                            a.A2 = p.Btl;
                            h1.push_back(a);
                            tc::HostProblem c{p.Yb, p.Wth, p.Wtl, p.Y2h, p.Y2l, nullptr, p.dims.L, p.rt, p.rt, ldb, p.np, ldb, 0};
                            c.A2 = p.Yl;
                            h2.push_back(c);
                            fb.s[i - i0].Yh = p.Y2h; fb.s[i - i0].Yl = p.Y2l;
                        }
                        if ((st = tc::launch<false, true, tc::OUT_BF16_SPLIT, true, true>(ctx, h1, store, "gemm_tc_rot")) != ATP_OK) return st;
                        if ((st = tc::launch<false, true, tc::OUT_BF16_SPLIT, true, true>(ctx, h2, store, "gemm_tc_rot")) != ATP_OK) return st;
                    } else {
                        GemmBatch r1, r2; r1.count = r2.count = cnt;
                        for (size_t i = i0; i < i1; ++i) {
                            SeqPlan &p = bp.seqs[i];
                            int k = (int)(i - i0);
                            r1.p[k] = GemmProblem{p.BW, p.Wt, p.Z, nullptr, p.rt > 0 ? d : 0, p.rt, p.rt, p.rt, p.np, p.rt, 0};
                            r2.p[k] = GemmProblem{p.Y, p.Wt, p.Y2, nullptr, p.dims.L, p.rt, p.rt, p.rt, p.np, p.rt, 0};
                            gg.p[k].A = p.Z; gg.p[k].B = p.Z;
                            fb.s[k].Y = p.Y2;
                        }
                        if ((st = launch_gemm_simt<float, float, float, false, true>(ctx, r1, store, 1, nullptr, 0, "gemm_simt_rot")) != ATP_OK) return st;
                        if ((st = launch_gemm_simt<float, float, float, false, true>(ctx, r2, store, 1, nullptr, 0, "gemm_simt_rot")) != ATP_OK) return st;
                    }
                }
            }
            int npow = 1; while (npow < maxrt) npow <<= 1;
            ATP_KERNEL(ctx, "colsum", 0, 0);
            colsum2_kernel<<<dim3(ceil_div(maxrt, 32), COLSUM_SLABS, cnt), 256, 0, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
            ATP_KERNEL(ctx, "sigma_sort", 0, 0);
            sigma_sort2_kernel<<<cnt, 1024, (size_t)npow * 8, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
            ATP_KERNEL(ctx, "select", 0, 0);
            select2_kernel<<<dim3(maxr, cnt), 128, 0, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
            // X_r = Wsel^T Bt2^T  and  U_r = Y2 Wsel  (Bt2, Y2: rotated by the first pass)
            if constexpr (kBf16) {
                std::vector<tc::HostProblem> h1, h2;
                for (size_t i = i0; i < i1; ++i) {
                    SeqPlan &p = bp.seqs[i];
                    int ldb = (int)align_up((size_t)p.rt, 8), ldw = (int)align_up((size_t)std::max(p.dims.r, 1), 8);
                    tc::HostProblem a{p.Wsh, p.Zb, p.Zl, (T *)X_r->data + (size_t)p.dims.rank0 * X_r->ld, nullptr, nullptr,
                                      p.dims.r, d, p.rt, ldw, ldb, (int)X_r->ld, 0};
                    a.A2 = p.Wsl;
                    h1.push_back(a);
                    tc::HostProblem c{p.Y2h, p.Wsh, p.Wsl, (T *)U_r->data + (size_t)p.dims.row0 * U_r->ld, nullptr, nullptr,
                                      p.dims.L, p.dims.r, p.rt, ldb, ldw, (int)U_r->ld, 0};
                    c.A2 = p.Y2l;
                    h2.push_back(c);
                }
                if ((st = tc::launch<true, true, tc::OUT_BF16, true, true>(ctx, h1, store, "gemm_tc_out")) != ATP_OK) return st;
                if ((st = tc::launch<false, true, tc::OUT_BF16, false, true>(ctx, h2, store, "gemm_tc_out")) != ATP_OK) return st;
            } else {
                for (size_t i = i0; i < i1; ++i) {
                    SeqPlan &p = bp.seqs[i];
                    int k = (int)(i - i0);
                    g.p[k] = GemmProblem{p.Wsel, p.Z, (T *)X_r->data + (size_t)p.dims.rank0 * X_r->ld, nullptr,
                                         p.dims.r, p.rt > 0 ? d : 0, p.rt, p.dims.r, p.rt, (int)X_r->ld, 0};
                    gg.p[k] = GemmProblem{p.Y2, p.Wsel, (T *)U_r->data + (size_t)p.dims.row0 * U_r->ld, nullptr,
                                          p.dims.L, p.dims.r, p.rt, p.rt, p.dims.r, (int)U_r->ld, 0};
                }
                if ((st = launch_gemm_simt<float, float, T, true, true>(ctx, g, store, 1, nullptr, 0, "gemm_simt_out")) != ATP_OK) return st;
                if ((st = launch_gemm_simt<float, float, T, false>(ctx, gg, store, 1, nullptr, 0, "gemm_simt_out")) != ATP_OK) return st;
            }
            ATP_KERNEL(ctx, "signfix", 0, 0);
            signfix_kernel<T><<<dim3(maxr, cnt), 256, 0, ctx->stream>>>(fb);
            ATP_LAUNCHED(ctx);
        }
    }
    if (forked) {
        for (int gq = 0; gq < 2; ++gq) {
            ATP_CUDA_OK(ctx, cudaEventRecord(ctx->ev_join[gq], ctx->aux[gq]));
            ATP_CUDA_OK(ctx, cudaStreamWaitEvent(main_stream, ctx->ev_join[gq], 0));
        }
    }
    return ATP_OK;
}

extern "C" atp_status atp_principal_basis(atp_ctx *ctx, const atp_mat *X, const atp_seqs *seqs,
                                          const atp_basis_opts *opts, atp_mat *U_r, atp_mat *X_r, float *sigma)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    atp_status st;
    if ((st = check_mat(X)) != ATP_OK || (st = check_mat(U_r)) != ATP_OK || (st = check_mat(X_r)) != ATP_OK) return st;
    int oversample = 64, power_iters = 2, max_sweeps = 24, jbj = 16, jinner = 1, groups = 0; uint64_t seed = 0x243F6A8885A308D3ull;
    bool no_host_sync = false;
    if (opts) {
        // the struct grew by no_host_sync: the shorter layout is still accepted
        if (opts->struct_size < offsetof(atp_basis_opts, no_host_sync)) return ATP_ERR_INVALID_ARG;
        if (opts->struct_size >= sizeof(atp_basis_opts)) no_host_sync = opts->no_host_sync != 0;
        if (opts->oversample >= 0) oversample = opts->oversample;
        if (opts->power_iters >= 0) power_iters = opts->power_iters;
        if (opts->max_sweeps > 0) max_sweeps = opts->max_sweeps;
        seed ^= opts->seed * 0x9E3779B97F4A7C15ull;
        if (opts->jacobi_block == 16 || opts->jacobi_block == 32 || opts->jacobi_block == 1) jbj = opts->jacobi_block;
        else if (opts->jacobi_block != 0) return ATP_ERR_INVALID_ARG;
        if (opts->jacobi_inner > 0) jinner = opts->jacobi_inner;
        groups = opts->groups;
    }
    if (oversample > 4096 || power_iters > 64 || max_sweeps > 200) return ATP_ERR_INVALID_ARG;
    if (U_r->dtype != X->dtype || X_r->dtype != X->dtype) return ATP_ERR_UNSUPPORTED_DTYPE;
    std::vector<SeqDims> sd;
    if ((st = check_seqs(seqs, sd, X->rows)) != ATP_OK) return st;
    int64_t tr = 0; int maxr = 0;
    for (auto &s : sd) {
        if (s.r > X->cols) return ATP_ERR_INVALID_RANK;
        if (std::min<int64_t>(s.L, X->cols) > 4096 && s.r + oversample > 4096) return ATP_ERR_INVALID_RANK;   // sort buffer limit
        tr += s.r; maxr = std::max(maxr, s.r);
    }
    if (U_r->rows != X->rows || U_r->cols < maxr || X_r->rows != tr || X_r->cols != X->cols) return ATP_ERR_INVALID_ARG;
    if (X->rows == 0) return ATP_OK;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    if (X->dtype == ATP_F32) return basis_impl<float>(ctx, X, sd, oversample, power_iters, max_sweeps, seed, jbj, jinner, groups, no_host_sync, U_r, X_r, sigma);
    return basis_impl<__nv_bfloat16>(ctx, X, sd, oversample, power_iters, max_sweeps, seed, jbj, jinner, groups, no_host_sync, U_r, X_r, sigma);
}

// ------------------------------------------------------------------------------------------------
size_t linear_workspace_bytes(const std::vector<SeqDims> &seqs, int64_t d_out);
size_t attention_workspace_bytes(const std::vector<SeqDims> &seqs, int64_t dp);

static atp_status workspace_bytes_impl(atp_ctx *ctx, int op, const atp_seqs *seqs, int64_t d, int64_t d_out,
                                       atp_dtype dtype, int oversample, size_t *bytes)
{
    if (!ctx || !bytes) return ATP_ERR_INVALID_ARG;
    if (dtype != ATP_F32 && dtype != ATP_BF16) return ATP_ERR_UNSUPPORTED_DTYPE;
    *bytes = 0;
    if (op == ATP_OP_NORM) return ATP_OK;
    std::vector<SeqDims> sd;
    atp_status st = check_seqs(seqs, sd, -1);
    if (st != ATP_OK) return st;
    if (d < 1 || d > 0x7fffffff) return ATP_ERR_INVALID_ARG;
    switch (op) {
        case ATP_OP_BASIS: *bytes = basis_workspace_bytes(sd, (int)d, oversample, ctx->sm_count) + 256; return ATP_OK;
        case ATP_OP_ATTENTION: if (d_out < 1) return ATP_ERR_INVALID_ARG; *bytes = attention_workspace_bytes(sd, d_out) + 256; return ATP_OK;
        case ATP_OP_LINEAR: if (d_out < 1) return ATP_ERR_INVALID_ARG; *bytes = linear_workspace_bytes(sd, d_out) + 256; return ATP_OK;
        case ATP_OP_ALTERNATING: *bytes = alternating_workspace_bytes(sd, (int)d) + 256; return ATP_OK;
        default: return ATP_ERR_INVALID_ARG;
    }
}

extern "C" atp_status atp_workspace_bytes(atp_ctx *ctx, int op, const atp_seqs *seqs, int64_t d, int64_t d_out,
                                          atp_dtype dtype, size_t *bytes)
{
    return workspace_bytes_impl(ctx, op, seqs, d, d_out, dtype, 64, bytes);
}

extern "C" atp_status atp_basis_workspace_bytes(atp_ctx *ctx, const atp_seqs *seqs, int64_t d, atp_dtype dtype,
                                                const atp_basis_opts *opts, size_t *bytes)
{
    int oversample = 64;
    if (opts) {
        if (opts->struct_size < offsetof(atp_basis_opts, no_host_sync)) return ATP_ERR_INVALID_ARG;
        if (opts->oversample >= 0) oversample = opts->oversample;
    }
    if (oversample > 4096) return ATP_ERR_INVALID_ARG;
    return workspace_bytes_impl(ctx, ATP_OP_BASIS, seqs, d, 0, dtype, oversample, bytes);
}

// ------------------------------------------------------------------------------------------------
// Self-tests of the bookkeeping around the kernels (used by the test suite).
__global__ void wait_timeout_kernel(unsigned *sync, int *status)
{
    // a group barrier that expects two CTAs while only this one exists: the flag it polls is never set
    if (!j3::group_barrier(sync, 1u, 2u, status + 1, 1u << 12) && threadIdx.x == 0) raise_status(status, ATP_ERR_TIMEOUT);
}

extern "C" atp_status atp_selftest_wait_timeout(atp_ctx *ctx)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    if (!ctx->workspace || ctx->workspace_bytes < 64 * sizeof(unsigned)) return ATP_ERR_WORKSPACE_TOO_SMALL;
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    ATP_CUDA_OK(ctx, cudaMemsetAsync(ctx->workspace, 0, 64 * sizeof(unsigned), ctx->stream));
    ATP_KERNEL(ctx, "wait_timeout", 0, 0);
    wait_timeout_kernel<<<1, 32, 0, ctx->stream>>>((unsigned *)ctx->workspace, ctx->dev_status);
    ATP_LAUNCHED(ctx);
    return ATP_OK;
}

extern "C" int atp_selftest_per_device_once(void)
{
    // the step must run once per device ordinal, again after a failure, and every time for ordinals
    // outside the table
    PerDeviceOnce once;
    int runs = 0;
    auto ok = [&] { ++runs; return cudaSuccess; };
    auto fail = [&] { ++runs; return cudaErrorUnknown; };
    once.run(0, ok); once.run(0, ok); once.run(1, ok); once.run(1, ok); once.run(0, ok);     // 2 runs
    once.run(2, fail); once.run(2, ok); once.run(2, ok);                                      // 2 more
    once.run(-1, ok); once.run(-1, ok); once.run(PerDeviceOnce::MAX_DEV, ok);                 // 3 more
    return runs;
}
