// Persistent block Gram-Schmidt: orthonormalises the columns of the range-finder iterates (Sec. 4.2:
// the basis U must satisfy U^T U = I) for every sequence of a batch in ONE cooperative launch.
//
// Panels of 64 columns, left to right; every panel runs `reps` times through
//   project   C = Q^T P against the finished columns Q (split over row ranges, partials summed in a fixed order)
//   update    P <- P - Q C
//   Gram      S = P^T P accumulated in fp64, scaled, Cholesky-factored and inverted in fp64 (panel_chol.cuh); from the
//             second repetition on, when S is within 5e-3 of the identity, the factor comes from a three-term series
//   apply     P <- P (D^-1 L^-T); columns found dependent are replaced by hash noise, which the next
//             repetition orthonormalises
// With two repetitions (what the extraction asks for) the passes are reordered so that the second projection runs
// beside the single-CTA factorisation of the first repetition and the first apply folds into the second Gram
// pass; see the panel program in the kernel.
// Two repetitions give orthonormality to working precision (the second also repairs the explicit inverse,
// which is only norm-wise stable). Each sequence owns a group of CTAs; the phases of a panel are separated by
// the group's barrier (bounded spin, see jacobi3.cuh) instead of kernel boundaries, and every phase is a list
// of independent 64 x 64 tile jobs dealt out round-robin. The 64^3 tile products run on the tensor cores in
// split TF32 precision (three products, ~2^-21): plain TF32 is not enough even for the first repetition, because
// what a projection leaves of an ill-conditioned panel is far below 2^-11 of the panel. fp32 inputs keep every
// product on the fp32 units.
#pragma once
#include "jacobi3.cuh"
#include "panel_chol.cuh"

namespace orth {

using j3::BLK; using j3::NT; using j3::LDA; using j3::LDB;
constexpr int MAXSEQ = 32;
constexpr int NRED = 8;           // second-level partial Gram sums (chunk ranges)

struct Seq {
    float *M; int n, rt, ld;                  // the iterate: n x rt, fp32, leading dimension ld
    __nv_bfloat16 *hi, *lo; int ldh;          // nullable: the finished columns also go out as a bf16 hi/lo pair
    float *Cpart, *C, *Dpart, *W;             // tile scratch (see scratch_tiles)
    double *gpart, *gpart2;
    int *flags;
    unsigned *sync;                           // 64 words: group barrier (jacobi3.cuh); then one word per CTA of the
                                              // group (its SM)
    int cta0, ncta, index;                    // CTA group (on entry to launch(): ncta = the cap the scratch was
                                              // sized for); index of the sequence in its batch (noise stream)
};
struct Batch { Seq s[MAXSEQ]; int count; };

// Number of 64 x 64 fp32 tiles of Cpart / C / Dpart, fp64 tiles of gpart, for a sequence of n rows and rt
// columns handled by at most `ncta` CTAs.
struct Scratch { size_t cpart, c, dpart, gpart; };
static inline Scratch scratch_tiles(int n, int rt, int ncta)
{
    const size_t nt = (size_t)(n + 63) / 64, nj = (size_t)(rt + 63) / 64;
    return Scratch{(size_t)ncta + nj + 1, nj + 1, (size_t)ncta + nt + 1, nt + 1};
}

// 64 x 64 tile of a row-major fp32 matrix, zero beyond rv rows / cv columns, in two halves so that the loads of
// the next tile can be in flight while the current one is multiplied: fetch_tile (global -> registers, four
// 16-byte pieces per thread) and stash_tile (registers -> shared memory at stride lds).
struct TileRegs { float4 v[4]; };
__device__ __forceinline__ void fetch_tile(TileRegs &tr, const float *src, int ld, int rv, int cv, bool vec)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int f = threadIdx.x + i * NT, r = f >> 4, c = (f & 15) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < rv) {
            const float *p = src + (size_t)r * ld + c;
            if (vec && c + 3 < cv) v = __ldcg((const float4 *)p);
            else {
                if (c < cv) v.x = __ldcg(p);
                if (c + 1 < cv) v.y = __ldcg(p + 1);
                if (c + 2 < cv) v.z = __ldcg(p + 2);
                if (c + 3 < cv) v.w = __ldcg(p + 3);
            }
        }
        tr.v[i] = v;
    }
}
__device__ __forceinline__ void stash_tile(const TileRegs &tr, float *dst, int lds)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int f = threadIdx.x + i * NT, r = f >> 4, c = (f & 15) * 4;
        *(float4 *)(dst + r * lds + c) = tr.v[i];             // lds is a multiple of 4 floats: 16-byte aligned
    }
}
__device__ __forceinline__ void load_tile(float *dst, int lds, const float *src, int ld, int rv, int cv, bool vec)
{
    TileRegs tr;
    fetch_tile(tr, src, ld, rv, cv, vec);
    stash_tile(tr, dst, lds);
}

// sum of base[0], base[stride], ..., base[(count - 1) stride] in that order, eight loads in flight
template <typename T>
__device__ __forceinline__ T ordered_sum(const T *base, size_t stride, int count)
{
    T s = (T)0;
    int i = 0;
    for (; i + 8 <= count; i += 8) {
        T v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __ldcg(base + (size_t)(i + k) * stride);
#pragma unroll
        for (int k = 0; k < 8; ++k) s += v[k];
    }
    for (; i < count; ++i) s += __ldcg(base + (size_t)i * stride);
    return s;
}

// acc += op(A) B on the units chosen by PREC: 0 fp32 FMA, 1 plain TF32, 3 split TF32.
template <int PREC, bool A_TRANS>
__device__ __forceinline__ void tile_mac(const float *As, int lda, const float *Bs, int ldb, int m0, int n0, float (&acc)[4][4])
{
    if (PREC == 3) j3::product64_acc<A_TRANS, false, 3>(As, lda, Bs, ldb, m0, n0, acc);
    else if (PREC == 1) j3::product64_acc<A_TRANS, false, 1>(As, lda, Bs, ldb, m0, n0, acc);
    else {
        const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll 4
        for (int k = 0; k < BLK; ++k) {
            const float a0 = A_TRANS ? As[k * lda + m0 + g] : As[(m0 + g) * lda + k];
            const float a1 = A_TRANS ? As[k * lda + m0 + g + 8] : As[(m0 + g + 8) * lda + k];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const float2 b = *(const float2 *)(Bs + k * ldb + n0 + nt * 8 + 2 * t);
                acc[nt][0] = fmaf(a0, b.x, acc[nt][0]); acc[nt][1] = fmaf(a0, b.y, acc[nt][1]);
                acc[nt][2] = fmaf(a1, b.x, acc[nt][2]); acc[nt][3] = fmaf(a1, b.y, acc[nt][3]);
            }
        }
    }
}

// This thread's part of a 64 x 64 accumulator tile (rows m0 + g, + 8; columns n0 + 8 nt + 2 t, + 1).
__device__ __forceinline__ void store_acc(float *dst, int ld, int m0, int n0, const float (&acc)[4][4])
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const int c = n0 + nt * 8 + 2 * t;
        *(float2 *)(dst + (size_t)(m0 + g) * ld + c) = make_float2(acc[nt][0], acc[nt][1]);
        *(float2 *)(dst + (size_t)(m0 + g + 8) * ld + c) = make_float2(acc[nt][2], acc[nt][3]);
    }
}

// TENSOR: bf16 inputs (tensor-core products); otherwise fp32 FMA everywhere.
template <bool TENSOR>
__global__ void __launch_bounds__(NT, 2)
orth_persistent_kernel(const __grid_constant__ Batch batch, int reps, uint64_t seed, int *status)
{
    extern __shared__ __align__(16) float osm[];
    __shared__ __align__(16) double Gs[PB * PB];
    float *sA = osm, *sB = osm + BLK * LDB;                   // two tiles at stride LDB (covers LDA too)
    int si = 0;
#pragma unroll 1
    for (int i = 1; i < batch.count; ++i) if ((int)blockIdx.x >= batch.s[i].cta0) si = i;
    const Seq &sq = batch.s[si];
    const int rank = (int)blockIdx.x - sq.cta0, tid = threadIdx.x, warp = tid >> 5;
    if (rank >= sq.ncta || sq.n <= 0 || sq.rt <= 0) return;
    const int m0 = (warp & 3) * 16, n0 = (warp >> 2) * 32;
    const int n = sq.n, rt = sq.rt, ld = sq.ld, ncta = sq.ncta;
    const int ntile = (n + 63) / 64, npanel = (rt + 63) / 64;
    const bool vec = (ld & 3) == 0 && ((size_t)sq.M & 15) == 0;
    int *abort_flag = status + 1;
    unsigned gen = 0;
    bool alive = true;
    // Every product needs fp32-like accuracy: a panel of an ill-conditioned iterate lies almost entirely in the span
    // of the finished columns, and what the projection leaves (1e-4 of the panel or less) is the information kept.
    constexpr int P_FINE = TENSOR ? 3 : 0;
    auto barrier = [&]() { alive = j3::group_barrier(sq.sync, ++gen, (unsigned)ncta, abort_flag) && alive; };

    // The CTA that shares an SM with rank 0 (if it belongs to this group) stays out of the work that runs beside
    // rank 0's factorisation, which is a latency chain and slows down under a busy neighbour.
    unsigned smid;
    asm("mov.u32 %0, %%smid;" : "=r"(smid));
    if (tid == 0) sq.sync[64 + rank] = smid;
    barrier();
    __shared__ int mate_s;
    if (tid == 0) mate_s = 1 << 30;
    __syncthreads();
    if (alive) {
        const unsigned sm0 = __ldcg(sq.sync + 64);
        for (int r = 1 + tid; r < ncta; r += NT)
            if (__ldcg(sq.sync + 64 + r) == sm0) atomicMin(&mate_s, r);
    }
    __syncthreads();
    const int mate = mate_s < ncta ? mate_s : -1;
    const bool overlap = reps == 2 && ncta >= 4;
    const int nworkers = ncta - 1 - (mate > 0 ? 1 : 0);
    const int wid = (rank == 0 || rank == mate) ? -1 : rank - 1 - ((mate > 0 && rank > mate) ? 1 : 0);

    // A panel is a short program of four kinds of passes, each written once below:
    //   PF      project (partial C over row ranges, jobs first, first + stride, ...) and / or, on rank 0, the factor
    //           of the panel's Gram matrix; SUMUPD  C = ordered sum of the partials, then partial D = Q C;
    //   GRAM    P -= sum D, optionally P <- P W, written back, Gram matrix in fp64 and its ordered sum;
    //   APPLY   P <- P W, dependent columns refilled, finished columns also as bf16 hi/lo.
    // Classic order per repetition: PF(project) SUMUPD GRAM PF(factor) APPLY. With two repetitions the second
    // projection is taken of the panel BEFORE the first factor is applied ((P - Q Q^T P) W = P W - Q Q^T (P W)), so
    // it runs beside rank 0's factorisation, and the first APPLY folds into the second GRAM pass:
    //   PF(project) SUMUPD GRAM | PF(project beside factor) SUMUPD GRAM(with W) | PF(series factor) APPLY.
    // A panel with dependent columns (their replacements must still be projected) returns to the classic order.
    enum { OP_PF, OP_SUMUPD, OP_GRAM, OP_APPLY };
    for (int pj = 0; pj < npanel && alive; ++pj) {
        const int j0 = pj * 64, w = min(64, rt - j0), nj = pj;            // nj finished panels
        const int KS = nj > 0 ? max(1, min(ntile, (ncta + nj - 1) / nj)) : 1;
        const int tper = (ntile + KS - 1) / KS;
        const int G = nj > 0 ? max(1, min(nj, (ncta + ntile - 1) / ntile)) : 1;
        const int jper = nj > 0 ? (nj + G - 1) / G : 1;
        const int nrange = max(1, min(8, ntile / 64)), cper = (ntile + nrange - 1) / nrange;
        int stage = overlap ? 0 : 30, rep = 0;
        while (stage >= 0 && alive) {
            int op = OP_PF, first = -1, stride = 1, arep = 0;
            bool do_factor = false, series_ok = false, with_w = false, last = false, skip = false;
            switch (stage) {
                // overlapped order
                case 0: op = OP_PF; first = rank; stride = ncta; skip = nj == 0; break;
                case 1: op = OP_SUMUPD; skip = nj == 0; break;
                case 2: op = OP_GRAM; break;
                case 3: op = OP_PF; first = nj > 0 ? wid : -1; stride = nworkers; do_factor = true; break;
                case 4: op = OP_SUMUPD; skip = nj == 0; break;
                case 5: op = OP_GRAM; with_w = true; break;
                case 6: op = OP_PF; do_factor = true; series_ok = true; break;
                case 7: op = OP_APPLY; arep = 1; last = true; break;
                // dependent columns found by the first factor: classic remainder
                case 20: op = OP_APPLY; arep = 0; break;
                case 21: op = OP_PF; first = rank; stride = ncta; skip = nj == 0; break;
                case 22: op = OP_SUMUPD; skip = nj == 0; break;
                case 23: op = OP_GRAM; break;
                case 24: op = OP_PF; do_factor = true; series_ok = true; break;
                case 25: op = OP_APPLY; arep = 1; last = true; break;
                // classic order, any number of repetitions
                case 30: op = OP_PF; first = rank; stride = ncta; skip = nj == 0; break;
                case 31: op = OP_SUMUPD; skip = nj == 0; break;
                case 32: op = OP_GRAM; break;
                case 33: op = OP_PF; do_factor = true; series_ok = rep > 0; break;
                default: op = OP_APPLY; arep = rep; last = rep == reps - 1; break;      // 34
            }
            if (!skip) switch (op) {
            case OP_PF: {
                if (do_factor && rank == 0) {
                    for (int e = tid; e < 4096; e += NT) Gs[e] = ordered_sum(sq.gpart2 + e, 4096, nrange);
                    __syncthreads();
                    // a nearly orthonormal panel gets its factor from a short series instead of the factorisation
                    if (!(series_ok && lowdin_64(Gs, w, sA, sq.W, sq.flags))) chol_invert_64(Gs, w, sq.W, sq.flags);
                    __syncthreads();
                } else if (first >= 0) {
                    for (int it = first; it < nj * KS; it += stride) {
                        const int jb = it / KS, ks = it - jb * KS;
                        float acc[4][4] = {};
                        const int t0 = ks * tper, t1 = min(ntile, (ks + 1) * tper);
                        TileRegs ra, rb;
                        if (t0 < t1) {
                            fetch_tile(ra, sq.M + (size_t)t0 * 64 * ld + jb * 64, ld, min(64, n - t0 * 64), 64, vec);
                            fetch_tile(rb, sq.M + (size_t)t0 * 64 * ld + j0, ld, min(64, n - t0 * 64), w, vec);
                        }
                        for (int t = t0; t < t1; ++t) {
                            stash_tile(ra, sA, LDB);
                            stash_tile(rb, sB, LDB);
                            __syncthreads();
                            if (t + 1 < t1) {                               // next tiles in flight during the product
                                const int rv = min(64, n - (t + 1) * 64);
                                fetch_tile(ra, sq.M + (size_t)(t + 1) * 64 * ld + jb * 64, ld, rv, 64, vec);
                                fetch_tile(rb, sq.M + (size_t)(t + 1) * 64 * ld + j0, ld, rv, w, vec);
                            }
                            tile_mac<P_FINE, true>(sA, LDB, sB, LDB, m0, n0, acc);
                            __syncthreads();
                        }
                        store_acc(sq.Cpart + (size_t)it * 4096, 64, m0, n0, acc);
                    }
                }
                barrier();
            } break;
            case OP_SUMUPD: {
                for (int it = rank; it < nj * 4; it += ncta) {           // a quarter tile per job
                    const int jb = it >> 2;
                    for (int e = (it & 3) * 1024 + tid; e < ((it & 3) + 1) * 1024; e += NT)
                        sq.C[(size_t)jb * 4096 + e] = ordered_sum(sq.Cpart + (size_t)jb * KS * 4096 + e, 4096, KS);
                }
                barrier();
                if (!alive) break;
                for (int it = rank; it < ntile * G; it += ncta) {
                    const int t = it / G, g = it - t * G;
                    const int rv = min(64, n - t * 64);
                    float acc[4][4] = {};
                    const int jb0 = g * jper, jb1 = min(nj, (g + 1) * jper);
                    TileRegs ra, rb;
                    if (jb0 < jb1) {
                        fetch_tile(ra, sq.M + (size_t)t * 64 * ld + jb0 * 64, ld, rv, 64, vec);
                        fetch_tile(rb, sq.C + (size_t)jb0 * 4096, 64, 64, 64, true);
                    }
                    for (int jb = jb0; jb < jb1; ++jb) {
                        stash_tile(ra, sA, LDA);
                        stash_tile(rb, sB, LDB);
                        __syncthreads();
                        if (jb + 1 < jb1) {
                            fetch_tile(ra, sq.M + (size_t)t * 64 * ld + (jb + 1) * 64, ld, rv, 64, vec);
                            fetch_tile(rb, sq.C + (size_t)(jb + 1) * 4096, 64, 64, 64, true);
                        }
                        tile_mac<P_FINE, false>(sA, LDA, sB, LDB, m0, n0, acc);
                        __syncthreads();
                    }
                    store_acc(sq.Dpart + (size_t)it * 4096, 64, m0, n0, acc);
                }
                barrier();
            } break;
            case OP_GRAM: {
                for (int t = rank; t < ntile; t += ncta) {
                    const int rv = min(64, n - t * 64);
                    load_tile(sA, LDA, sq.M + (size_t)t * 64 * ld + j0, ld, rv, w, vec);
                    if (with_w) load_tile(sB, LDB, sq.W, 64, 64, 64, true);
                    __syncthreads();
                    if (nj > 0) {
                        for (int e0 = tid; e0 < 4096; e0 += 4 * NT) {            // four elements, 4 G loads in flight
                            float sacc[4] = {0.f, 0.f, 0.f, 0.f};
                            const float *dp = sq.Dpart + (size_t)t * G * 4096 + e0;
                            for (int g = 0; g < G; ++g) {
                                float x[4];
#pragma unroll
                                for (int q = 0; q < 4; ++q) x[q] = __ldcg(dp + (size_t)g * 4096 + q * NT);
#pragma unroll
                                for (int q = 0; q < 4; ++q) sacc[q] += x[q];
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int e = e0 + q * NT, r = e >> 6, c = e & 63;
                                const float v = sA[r * LDA + c] - sacc[q];
                                sA[r * LDA + c] = (r < rv && c < w) ? v : 0.f;
                                if (!with_w && r < rv && c < w) sq.M[((size_t)t * 64 + r) * ld + j0 + c] = v;
                            }
                        }
                        __syncthreads();
                    }
                    if (with_w) {
                        float acc[4][4] = {};
                        tile_mac<P_FINE, false>(sA, LDA, sB, LDB, m0, n0, acc);
                        __syncthreads();
                        const int lane = tid & 31, g = lane >> 2, tq = lane & 3;
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int r = m0 + g + (i >= 2 ? 8 : 0), c = n0 + nt * 8 + 2 * tq + (i & 1);
                                const bool in = r < rv && c < w;
                                sA[r * LDA + c] = in ? acc[nt][i] : 0.f;
                                if (in) sq.M[((size_t)t * 64 + r) * ld + j0 + c] = acc[nt][i];
                            }
                        __syncthreads();
                    }
                    const int tx = tid & 15, ty = tid >> 4;
                    double acc[4][4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
#pragma unroll 4
                    for (int k = 0; k < 64; ++k) {
                        const float4 a = *(const float4 *)&sA[k * LDA + ty * 4];
                        const float4 b = *(const float4 *)&sA[k * LDA + tx * 4];
                        const double av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc[i][j] = fma(av[i], bv[j], acc[i][j]);
                    }
                    double *dst = sq.gpart + (size_t)t * 4096;
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) dst[(ty * 4 + i) * 64 + tx * 4 + j] = acc[i][j];
                    __syncthreads();
                }
                barrier();
                if (!alive) break;
                // ordered sum of the partial Gram matrices: 16 element slices x (up to 8) chunk ranges
                for (int it = rank; it < 16 * nrange; it += ncta) {
                    const int sl = it & 15, rg = it >> 4, e = sl * 256 + tid;
                    const int c0 = rg * cper, c1 = min(ntile, (rg + 1) * cper);
                    sq.gpart2[(size_t)rg * 4096 + e] = ordered_sum(sq.gpart + (size_t)c0 * 4096 + e, 4096, max(c1 - c0, 0));
                }
                barrier();
            } break;
            default: {                                                   // OP_APPLY
                const uint64_t nseed = seed + 7919ull * (uint64_t)(pj * 2 + arep);
                const float rscale = rsqrtf((float)n * (1.f / 3.f));     // replacement columns of about unit norm
                for (int t = rank; t < ntile; t += ncta) {
                    const int rv = min(64, n - t * 64);
                    load_tile(sA, LDA, sq.M + (size_t)t * 64 * ld + j0, ld, rv, w, vec);
                    load_tile(sB, LDB, sq.W, 64, 64, 64, true);
                    __syncthreads();
                    float acc[4][4] = {};
                    tile_mac<P_FINE, false>(sA, LDA, sB, LDB, m0, n0, acc);
                    const int lane = tid & 31, g = lane >> 2, tq = lane & 3;
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int r = m0 + g + (i >= 2 ? 8 : 0), c = n0 + nt * 8 + 2 * tq + (i & 1);
                            if (r >= rv || c >= w) continue;
                            const int grow = t * 64 + r;
                            float v = acc[nt][i];
                            if (__ldcg(sq.flags + c))
                                v = rscale * hash_uniform(nseed, ((uint64_t)sq.index << 40) ^ ((uint64_t)grow << 8) ^ (uint64_t)c);
                            sq.M[(size_t)grow * ld + j0 + c] = v;
                            if (last && sq.hi) {
                                const __nv_bfloat16 h = __float2bfloat16_rn(v);
                                sq.hi[(size_t)grow * sq.ldh + j0 + c] = h;
                                sq.lo[(size_t)grow * sq.ldh + j0 + c] = __float2bfloat16_rn(v - __bfloat162float(h));
                            }
                        }
                    __syncthreads();
                }
                barrier();
            } break;
            }
            // next stage
            if (stage == 3) {
                const bool dependent = __syncthreads_or(alive && tid < w && __ldcg(sq.flags + tid) != 0) != 0;
                stage = dependent ? 20 : 4;
            } else if (stage == 7 || stage == 25) stage = -1;
            else if (stage == 34) { ++rep; stage = rep < reps ? 30 : -1; }
            else ++stage;
        }
    }
    if (rank == 0 && tid == 0 && !alive) raise_status(status, ATP_ERR_TIMEOUT);
}

__global__ void init_kernel(const __grid_constant__ Batch batch)
{
    const Seq &sq = batch.s[blockIdx.x];
    if (threadIdx.x < 64 && sq.n > 0) sq.sync[threadIdx.x] = 0u;
}

constexpr size_t SMEM_BYTES = (size_t)(2 * BLK * LDB) * sizeof(float);

// Largest number of CTAs a launch hands to one sequence (workspace sizing and launch agree on it).
static inline int max_ctas_per_seq(int sm_count, int nseq) { return std::max(1, 2 * sm_count / std::max(nseq, 1)); }

template <bool TENSOR>
static inline atp_status launch(atp_ctx *ctx, Batch &ob, int reps, uint64_t seed)
{
    if (ob.count <= 0) return ATP_OK;
    static PerDeviceOnce attr_once;
    ATP_CUDA_OK(ctx, attr_once.run(ctx->device, [] {
        return cudaFuncSetAttribute(orth_persistent_kernel<TENSOR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    }));
    int occ = 0;
    ATP_CUDA_OK(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, orth_persistent_kernel<TENSOR>, NT, SMEM_BYTES));
    if (occ < 1) return ATP_ERR_CUDA;
    const int total = ctx->sm_count * std::min(occ, 2);
    double wsum = 0;
    for (int i = 0; i < ob.count; ++i) wsum += (double)ob.s[i].n * ob.s[i].rt;
    if (wsum <= 0) return ATP_OK;
    int next = 0;
    for (int i = 0; i < ob.count; ++i) {
        Seq &q = ob.s[i];
        const int ntile = (q.n + 63) / 64;
        int c = (int)((double)total * ((double)q.n * q.rt / wsum));
        c = std::max(1, std::min(std::min(c, q.ncta), 4 * std::max(ntile, 1)));    // q.ncta: the cap the scratch was sized for
        q.cta0 = next; q.ncta = c; q.index = i;
        next += c;
    }
    if (next > total) return ATP_ERR_INVALID_ARG;      // cannot happen: shares sum to at most `total`
    ATP_KERNEL(ctx, "orth_init", 0, 0);
    init_kernel<<<ob.count, 64, 0, ctx->stream>>>(ob);
    ATP_LAUNCHED(ctx);
    int *status = ctx->dev_status;
    void *args[] = {(void *)&ob, (void *)&reps, (void *)&seed, (void *)&status};
    // bytes: one read and one write of every iterate
    ATP_KERNEL(ctx, "orth_persistent", 0, wsum * 8.0);
    ATP_CUDA_OK(ctx, cudaLaunchCooperativeKernel((const void *)orth_persistent_kernel<TENSOR>, dim3(next), dim3(NT), args, SMEM_BYTES, ctx->stream));
    ATP_LAUNCHED(ctx);
    return ATP_OK;
}

}  // namespace orth
