// Cholesky factorisation and inversion of a 64 x 64 Gram matrix in fp64, on 256 threads of a CTA.
// Gs (shared memory, 64 x 64 doubles, row-major) holds G = P^T P of a panel of n <= 64 columns. The
// matrix is scaled to unit diagonal, factored D^-1 G D^-1 = L L^T and the factor inverted; the result
// W = D^-1 L^-T (upper triangular, fp32, 64 x 64 row-major) goes to rinv, so that P W has orthonormal
// columns. A column whose scaled pivot falls below 1e-10 (its part outside the span of the earlier
// columns is below 1e-5 of its norm) is flagged as dependent in flags[0..63].
// Right-looking by blocks of four columns, in registers: thread (br, bc) owns the 4 x 4 blocks of G
// and of X (X starts as the identity and ends as L^-1) at rows 4 br, columns 4 bc. Block step jb:
//   1. the owner of the diagonal block factors it (four pivots) and publishes L_bb and 1 / L_jj;
//   2. the owners of the block column below it solve for their rows of L, the owners of block row jb of
//      X apply L_bb^-1 to it; both publish;
//   3. everybody below subtracts L_i L_k^T from G (columns right of jb) or L_i X_b from X (columns up
//      to jb): 64 independent multiply-adds per thread.
// Two barriers per four columns (named barrier 1, 256 threads: exactly the threads 0..255 must call).
#pragma once
#include "common.cuh"

constexpr int PB = 64;            // orthonormalisation panel width

__device__ __noinline__ void chol_invert_64(const double *Gs, int n, float *rinv, int *flags)
{
    __shared__ double rs[PB];          // 1 / sqrt(diagonal of the Gram matrix)
    __shared__ double lcol4[PB][4];    // block column jb of L (rows below the diagonal block)
    __shared__ double xrow4[4][PB];    // block row jb of L^-1
    __shared__ double Lbb[4][4];       // the factored diagonal block (strictly lower part)
    __shared__ double rinv4[4];        // 1 / L_jj, 0 for a dependent column
    __shared__ int dep[PB];
    auto bar256 = [] { asm volatile("bar.sync 1, 256;" ::: "memory"); };
    const int tid = threadIdx.x;
    const int br = tid >> 4, bc = tid & 15;
    // One 4 x 4 block per thread: it holds the thread's block of G until block step jb = bc has consumed it, and
    // the thread's block of X from then on (a block of G left of the current step is dead, a block of X right of
    // it is still its initial identity / zero block), which halves the register need.
    double blk[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) blk[a][b] = Gs[(4 * br + a) * PB + 4 * bc + b];
    auto to_x = [&]() {
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) blk[a][b] = (br == bc && a == b) ? 1.0 : 0.0;
    };
    if (br == bc) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int i = 4 * br + a;
            rs[i] = (i < n && blk[a][a] > 0.0) ? rsqrt(blk[a][a]) : 0.0;
            dep[i] = 0;
        }
    }
    bar256();
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const double ra = rs[4 * br + a], rb = rs[4 * bc + b];
            blk[a][b] = (br == bc && a == b) ? (ra > 0.0 ? 1.0 : 0.0) : blk[a][b] * ra * rb;
        }
    const int nblk = (n + 3) >> 2;
    for (int jb = 0; jb < nblk; ++jb) {
        if (br == jb && bc == jb) {
            // 1. the diagonal block, column by column; a dependent column gets a unit pivot and zeros below
            double ri[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                double piv = blk[c][c];
#pragma unroll
                for (int k = 0; k < c; ++k) piv = fma(-blk[c][k], blk[c][k], piv);
                const bool bad = !(piv > 1e-10);
                // 1/sqrt from the fp32 approximation and one Newton step (piv is in (1e-10, ~1]): ~2^-44 relative,
                // far below the fp32 precision the result is stored in
                double y = (double)rsqrtf((float)piv);
                y = y * (1.5 - 0.5 * piv * y * y);
                ri[c] = bad ? 0.0 : y;
                if (bad && 4 * jb + c < n) dep[4 * jb + c] = 1;
#pragma unroll
                for (int r = c + 1; r < 4; ++r) {
                    double v = blk[r][c];
#pragma unroll
                    for (int k = 0; k < c; ++k) v = fma(-blk[r][k], blk[c][k], v);
                    blk[r][c] = v * ri[c];
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                rinv4[r] = ri[r];
#pragma unroll
                for (int c = 0; c < 4; ++c) Lbb[r][c] = (c < r) ? blk[r][c] : 0.0;
            }
            to_x();
        }
        bar256();
        if (bc == jb && br > jb) {
            // 2a. rows of L below the diagonal block: l_c = (g_c - sum_{k<c} l_k L_bb[c][k]) / L_cc
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                double l[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    double v = blk[a][c];
#pragma unroll
                    for (int k = 0; k < c; ++k) v = fma(-l[k], Lbb[c][k], v);
                    l[c] = v * rinv4[c];
                    lcol4[4 * br + a][c] = l[c];
                }
            }
            to_x();
        }
        if (br == jb && bc <= jb) {
            // 2b. block row jb of X: forward substitution with L_bb (a dependent column keeps its scale)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const double sc = rinv4[c] > 0.0 ? rinv4[c] : 1.0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    double v = blk[c][b];
#pragma unroll
                    for (int k = 0; k < c; ++k) v = fma(-Lbb[c][k], blk[k][b], v);
                    blk[c][b] = v * sc;
                    xrow4[c][4 * bc + b] = blk[c][b];
                }
            }
        }
        bar256();
        if (br > jb && bc <= br) {
            // 3. trailing update (operands re-read from shared memory per row: registers are scarce here)
            const bool gpart = bc > jb;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                double rb[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) rb[c] = gpart ? lcol4[4 * bc + b][c] : xrow4[c][4 * bc + b];
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    double acc = blk[a][b];
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc = fma(-lcol4[4 * br + a][c], rb[c], acc);
                    blk[a][b] = acc;
                }
            }
        }
    }
    if (bc > br || bc >= nblk) to_x();      // blocks that never became part of X: above the diagonal, beyond n
    // W[k][c] = (L^-1)[c][k] / D_k ; this thread holds (L^-1)[4 br + a][4 bc + b]
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int k = 4 * bc + b;
        const double rk = rs[k];
        float4 w;
        w.x = (float)(rk * blk[0][b]); w.y = (float)(rk * blk[1][b]); w.z = (float)(rk * blk[2][b]); w.w = (float)(rk * blk[3][b]);
        *(float4 *)(rinv + k * PB + 4 * br) = w;
    }
    bar256();
    if (tid < PB) flags[tid] = (tid < n) ? (dep[tid] || !(rs[tid] > 0.0)) : 0;
}


// Orthonormalising factor of a panel that is already close to orthonormal (the second Gram-Schmidt repetition):
// with the Gram matrix scaled to unit diagonal, D^-1/2 G D^-1/2 = I + E, the symmetric factor
//   W = D^-1/2 (I - E/2 + 3/8 E^2)          (P W has orthonormal columns up to 5/16 |E|^3)
// needs one 64^3 product instead of a factorisation and its chain of 64 dependent pivots. Taken only when every
// diagonal entry is positive and the largest absolute row sum of E is at most LOWDIN_LIMIT (then the neglected
// term is below 4e-8); otherwise nothing is written and the caller factors the matrix. Returns the decision
// (block-uniform). Es: a 64 x LDE fp32 tile of shared memory; 256 threads.
constexpr float LOWDIN_LIMIT = 5e-3f;
constexpr int LDE = 72;
__device__ __noinline__ bool lowdin_64(const double *Gs, int n, float *Es, float *rinv, int *flags)
{
    __shared__ double rsq[PB];
    __shared__ float rowsum[PB];
    const int tid = threadIdx.x;
    bool bad = false;
    if (tid < PB) {
        const double d = Gs[tid * PB + tid];
        const bool pos = tid < n && d > 0.0;
        rsq[tid] = pos ? rsqrt(d) : 0.0;
        rowsum[tid] = 0.f;
        bad = tid < n && !pos;
    }
    __syncthreads();
    for (int e = tid; e < PB * PB; e += 256) {
        const int i = e >> 6, j = e & 63;
        float v = 0.f;
        if (i < n && j < n && i != j) v = (float)(Gs[e] * rsq[i] * rsq[j]);
        Es[i * LDE + j] = v;
        float a = fabsf(v);                                      // row i lies in two warps: 32 columns each
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if ((tid & 31) == 0) atomicAdd(&rowsum[i], a);
    }
    __syncthreads();
    if (tid < PB && !(rowsum[tid] <= LOWDIN_LIMIT)) bad = true;
    if (__syncthreads_or(bad)) return false;
    // E^2 (E is symmetric): thread (ty, tx) owns the 4 x 4 block at rows 4 ty, columns 4 tx
    const int tx = tid & 15, ty = tid >> 4;
    float acc[4][4] = {};
#pragma unroll 4
    for (int k = 0; k < PB; ++k) {
        const float4 a = *(const float4 *)&Es[k * LDE + ty * 4];
        const float4 b = *(const float4 *)&Es[k * LDE + tx * 4];
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int r = ty * 4 + i, c = tx * 4 + j;
            float w = 0.f;
            if (r < n && c < n) w = (float)rsq[r] * ((r == c ? 1.f : 0.f) - 0.5f * Es[r * LDE + c] + 0.375f * acc[i][j]);
            rinv[r * PB + c] = w;
        }
    if (tid < PB) flags[tid] = 0;
    return true;
}
