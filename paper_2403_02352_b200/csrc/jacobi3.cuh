// Persistent two-sided block Jacobi eigensolver for the Gram matrix G = B B^T of the projected input
// (Rayleigh-Ritz step of the basis extraction, Sec. 4.2: the rotation that diagonalises G turns the
// orthonormal range basis into singular vectors, X' = [sigma_i v_i]).
//
// One cooperative launch diagonalises every sequence of a batch. Each sequence owns a fixed group of
// CTAs that loops over sweeps and steps on its own and leaves when its matrix has converged; the
// CTAs of a group meet at a counter in global memory (bounded spin) instead of at kernel boundaries.
// Blocks of 32 rows; a step handles n/64 disjoint block pairs (round-robin order) in two phases:
//   pivot : per pair, the 64 x 64 pivot block is rotated on chip by cyclic Jacobi (first step of a sweep: all
//           2016 pairs of its 64 rows once, in 63 rounds; other steps: the 1024 pairs across its two blocks, in
//           32 rounds). The block lives in registers (see "pivot phase" below); a round is a rotation per row
//           pair, two block barriers and a shift of the pairing. The accumulated row transform Vt (64 x 64)
//           is published. The pivot block of the NEXT step is formed on chip from the matrix before this step's
//           update (pivot_form), so the chain of pivot solves runs beside the update and never waits for it.
//   apply : every 64 x 64 block (p, q) of G becomes Vt_p G_pq Vt_q^T (upper triangle computed, mirror
//           stored), rows of Wt become Vt_p Wt, both in place. The pivot CTAs of the step read blocks of G as they
//           were before the update; a counter of fetched pivot blocks holds the first store of every updating
//           CTA back until they have them on chip. The 64^3 products run on the tensor cores in split
//           precision (three TF32 mma products per fp32 product), which keeps fp32 accuracy; fp32 inputs use the
//           fp32 units.
// G and Wt are stored with a leading dimension padded to a multiple of 64; the padding of G is zero
// (zero diagonal entries are never rotated), the padding of Wt is the identity.
#pragma once
#include "common.cuh"
#include <mutex>
#include <algorithm>

namespace j3 {

constexpr int JB = 32;            // block height
constexpr int BLK = 64;           // pivot block = one pair of blocks
constexpr int NT = 256;           // threads per CTA
constexpr int LDA = 68;           // shared-memory row stride (floats) of A-operand style tiles
constexpr int LDB = 72;           // shared-memory row stride of B-operand style tiles
constexpr int MAXSEQ = 32;        // sequences per launch
constexpr unsigned SPIN_LIMIT = 1u << 22;

struct Seq {
    float *G, *Wt, *Vbuf;         // G, Wt: np x np (ld = np); Vbuf: 2 x npairs x 64 x 64 (by step parity)
    int *vflag;                   // 2 x npairs: the pair rotated in this step
    unsigned *sync;               // 64 words. [0]: arrivals at the group barrier (monotonic); [32]: last
                                  // barrier completed; [1..4]: largest scaled off-diagonal entry of a
                                  // sweep, slot sweep % 4; [5]: sweeps used; [16..17]: work tickets of the update, [20..21]: pivot blocks fetched, both by step parity
    int n, np, nb;                // size, padded size (multiple of 64), number of 32-row blocks (even)
    int cta0, ncta;               // the group of CTAs that owns this sequence
};
struct Batch { Seq s[MAXSEQ]; int count; };

// Bytes of dynamic shared memory: four tile slots of 64 x LDB floats (pivot phase: the old blocks and the
// transforms the pivot block is formed from, then A and Vt; apply phase: Vt_p, Vt_q, T and the G block).
constexpr int SLOT = BLK * LDB;
constexpr size_t SMEM_BYTES = (size_t)4 * SLOT * sizeof(float);

__device__ __forceinline__ void rr_pair(int nb, int step, int t, int &I, int &J)
{
    const int m = nb - 1;
    if (t == 0) { I = m; J = step % m; }
    else { I = (step + t) % m; J = (step - t + m) % m; }
    if (I > J) { const int x = I; I = J; J = x; }
}

// Group barrier number `gen` (1, 2, ...) of a group of `ncta` CTAs: every CTA adds one to the arrival
// counter sync[0] (release); the last one to arrive publishes `gen` in sync[32] (another cache line, so that
// the pollers do not slow the arrivals down); the others poll that word (acquire). Bounded: returns false when
// the wait ran out or another CTA flagged an abort. Data that crosses the barrier is read with L2 loads.
__device__ __forceinline__ bool group_barrier(unsigned *sync, unsigned gen, unsigned ncta, int *abort_flag,
                                              unsigned limit = SPIN_LIMIT)
{
    __syncthreads();
    __shared__ int ok_s;
    if (threadIdx.x == 0) {
        int ok = 1;
        if (ncta > 1) {
            // release / acquire at GPU scope: the block barrier above orders the CTA's writes before thread 0's
            // release, the one below orders its acquire before the CTA's later reads
            unsigned old;
            asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(sync) : "memory");
            unsigned *flag = sync + 32;
            if (old + 1u == gen * ncta) {
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(gen) : "memory");
            } else {
                ok = 0;
                for (unsigned i = 0; i < limit; ++i) {
                    unsigned v;
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
                    if ((int)(v - gen) >= 0) { ok = 1; break; }
                    if ((i & 1023u) == 1023u && *(volatile int *)abort_flag) break;
                }
                if (!ok) *(volatile int *)abort_flag = 1;
            }
        }
        ok_s = ok;
    }
    __syncthreads();
    return ok_s != 0;
}

// Rotation (c, s) that annihilates the (p, q) entry of a symmetric matrix; identity when the entry is
// already small against its diagonal. With a = g_qq - g_pp, b = 2 g_pq, r = sqrt(a^2 + b^2):
//   cos 2t = |a| / r,  c = sqrt((1 + cos 2t) / 2),  s = sign(a) b / (2 r c)      (|t| <= pi/4).
__device__ __forceinline__ float2 rotation(float gpp, float gqq, float gpq, float tol_rot)
{
    float c = 1.f, s = 0.f;
    if (gpq != 0.f && gpq * gpq > tol_rot * tol_rot * fmaxf(gpp, 0.f) * fmaxf(gqq, 0.f)) {
        float a = gqq - gpp, b = 2.f * gpq;
        const float m = fmaxf(fabsf(a), fabsf(b));
        const float sc = m < 1e-18f ? 0x1p60f : (m > 1e18f ? 0x1p-60f : 1.f);
        a *= sc; b *= sc;
        const float rh = rsqrtf(fmaf(a, a, b * b));
        const float c2 = fmaf(0.5f * fabsf(a), rh, 0.5f);
        const float rc = rsqrtf(c2);
        c = c2 * rc;
        s = copysignf(0.5f, a) * b * rh * rc;
    }
    return make_float2(c, s);
}

// ---- pivot phase -------------------------------------------------------------------------------
// The 64 rows of a pivot block sit in 32 "even" and 32 "odd" slots. A phase of width m rotates, in m
// rounds, every even slot k with the odd slots of its own group of m: in round rd with slot
// base(k) + ((k - rd) mod m). The data never moves between rounds, only the pairing shifts, so every
// thread keeps its elements in registers:
//   thread (warp w, lane l) owns the even rows 4w..4w+3 and column slot l of the four quadrants
//     ee[a] = A[E(4w+a)][E(l)]   eo[a] = A[E(4w+a)][O(s(l))]
//     oe[a] = A[O(s(4w+a))][E(l)]   oo[a] = A[O(s(4w+a))][O(s(l))]         s = current pairing
//   and the same rows of the accumulated transform Vt (two logical columns l, l + 32).
// The 2 x 2 problem of pair k is complete in the thread with 4w+a = l, which derives the rotation and
// publishes it; everybody applies the rotations of its four row pairs and of its column pair. Moving
// to the next pairing shifts the odd quadrants by one slot: along the columns by a lane shuffle,
// along the rows inside the thread, except the last of its four rows, which goes to the next warp
// through shared memory (4 floats per thread and round).
// Slot -> logical row (0..31 first block, 32..63 second block) for a phase of width m: the logical
// rows are cut in groups of 2m; the first m of a group are even slots, the last m odd slots. Width 32
// pairs every row of the first block with every row of the second; widths 16, 8, 4, 2, 1 pair the rows
// inside the blocks; together the 63 rounds rotate each of the 2016 pairs exactly once.
constexpr int LDP = 65;           // row stride of the logical A and Vt copies in shared memory
__device__ __forceinline__ int slot_even(int i, int m) { return 2 * m * (i / m) + (i % m); }

__device__ void cross_phase(float *As, float *Vs, float2 *rot, float4 *xch, int m, float tol_rot)
{
    const int tid = threadIdx.x, w = tid >> 5, l = tid & 31;
    float ee[4], eo[4], oe[4], oo[4], ve[4][2], vo[4][2];
    const int cE = slot_even(l, m), cO = cE + m;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int rE = slot_even(4 * w + a, m) * LDP, rO = rE + m * LDP;
        ee[a] = As[rE + cE]; eo[a] = As[rE + cO]; oe[a] = As[rO + cE]; oo[a] = As[rO + cO];
        ve[a][0] = Vs[rE + l]; ve[a][1] = Vs[rE + l + 32];
        vo[a][0] = Vs[rO + l]; vo[a][1] = Vs[rO + l + 32];
    }
    const int ad = l - 4 * w;                                   // 0..3: this thread completes pair 4w + ad
    const int src_lane = (l & ~(m - 1)) | ((l - 1) & (m - 1));  // previous column slot of the group
    const int wg = m >= 8 ? m / 4 : 1;                          // warps per row group
    const int wprev = (w & ~(wg - 1)) | ((w - 1) & (wg - 1));
    for (int rd = 0; rd < m; ++rd) {
        float2 *rt = rot + (rd & 1) * 32;
        if ((unsigned)ad < 4u) {
            const float x = ad == 0 ? ee[0] : ad == 1 ? ee[1] : ad == 2 ? ee[2] : ee[3];
            const float y = ad == 0 ? oo[0] : ad == 1 ? oo[1] : ad == 2 ? oo[2] : oo[3];
            const float z = ad == 0 ? eo[0] : ad == 1 ? eo[1] : ad == 2 ? eo[2] : eo[3];
            rt[l] = rotation(x, y, z, tol_rot);
        }
        __syncthreads();
        const float2 cb = rt[l];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const float2 ca = rt[4 * w + a];
            const float r0 = ca.x * ee[a] - ca.y * oe[a], r1 = ca.x * eo[a] - ca.y * oo[a];
            const float r2 = ca.y * ee[a] + ca.x * oe[a], r3 = ca.y * eo[a] + ca.x * oo[a];
            ee[a] = cb.x * r0 - cb.y * r1; eo[a] = cb.y * r0 + cb.x * r1;
            oe[a] = cb.x * r2 - cb.y * r3; oo[a] = cb.y * r2 + cb.x * r3;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const float x = ve[a][c], y = vo[a][c];
                ve[a][c] = ca.x * x - ca.y * y; vo[a][c] = ca.y * x + ca.x * y;
            }
        }
        if (m == 1) break;
        // next pairing: odd rows shift by one slot inside their group ...
        float4 in;
        if (m >= 8) {
            xch[tid] = make_float4(oe[3], oo[3], vo[3][0], vo[3][1]);
            __syncthreads();
            in = xch[wprev * 32 + l];
        } else if (m == 4) {
            in = make_float4(oe[3], oo[3], vo[3][0], vo[3][1]);
        }
        if (m >= 4) {
#pragma unroll
            for (int a = 3; a > 0; --a) { oe[a] = oe[a - 1]; oo[a] = oo[a - 1]; vo[a][0] = vo[a - 1][0]; vo[a][1] = vo[a - 1][1]; }
            oe[0] = in.x; oo[0] = in.y; vo[0][0] = in.z; vo[0][1] = in.w;
        } else {                                                // m == 2: rows (0,1) and (2,3) swap
#pragma unroll
            for (int a = 0; a < 4; a += 2) {
                float t;
                t = oe[a]; oe[a] = oe[a + 1]; oe[a + 1] = t;
                t = oo[a]; oo[a] = oo[a + 1]; oo[a + 1] = t;
                t = vo[a][0]; vo[a][0] = vo[a + 1][0]; vo[a + 1][0] = t;
                t = vo[a][1]; vo[a][1] = vo[a + 1][1]; vo[a + 1][1] = t;
            }
        }
        // ... and so do the odd columns
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            eo[a] = __shfl_sync(0xffffffffu, eo[a], src_lane);
            oo[a] = __shfl_sync(0xffffffffu, oo[a], src_lane);
        }
    }
    // after m shifts (none for m = 1) every element is back where it was loaded from
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int rE = slot_even(4 * w + a, m) * LDP, rO = rE + m * LDP;
        As[rE + cE] = ee[a]; As[rE + cO] = eo[a]; As[rO + cE] = oe[a]; As[rO + cO] = oo[a];
        Vs[rE + l] = ve[a][0]; Vs[rE + l + 32] = ve[a][1];
        Vs[rO + l] = vo[a][0]; Vs[rO + l + 32] = vo[a][1];
    }
    __syncthreads();
}

// global row / column of local index l of the pair (I, J)
__device__ __forceinline__ int glob_of_loc(int I, int J, int l) { return (l < JB ? I : J) * JB + (l & (JB - 1)); }

// Copies the 64 x 64 pivot block of the pair (I, J) from G to the logical copy As (stride LDP).
__device__ void pivot_load(float *sm, const float *G, int np, int I, int J)
{
    float *As = sm;
    for (int f = threadIdx.x; f < BLK * (BLK / 4); f += NT) {
        const int li = f >> 4, lj = (f & 15) * 4;
        const float4 v = __ldcg((const float4 *)(G + (size_t)glob_of_loc(I, J, li) * np + glob_of_loc(I, J, lj)));
        float *dst = As + li * LDP + lj;
        dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    }
}

// Rotates the 64 x 64 pivot block held in As = sm (stride LDP, complete before the call: the routine starts with
// a block barrier) and publishes the accumulated row transform Vt (new rows = Vt * old rows, logical order) to
// vout. cross_only: the 32 rounds that pair the two blocks' rows; otherwise all 63 rounds. Returns the largest
// scaled off-diagonal entry found in the block before rotating (block-uniform); when it is <= tol_rot nothing is
// rotated or published.
__device__ float pivot_rotate(float *sm, bool cross_only, float tol_rot, float *vout, bool &rotated)
{
    __shared__ float red[NT / 32];
    __shared__ float2 rot[64];
    __shared__ float4 xch[NT];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float *As = sm, *Vs = sm + BLK * LDP;
    for (int e = tid; e < BLK * BLK; e += NT) Vs[(e >> 6) * LDP + (e & 63)] = ((e >> 6) == (e & 63)) ? 1.f : 0.f;
    __syncthreads();
    float mo = 0.f;
    for (int e = tid; e < BLK * BLK; e += NT) {
        const int i = e >> 6, j = e & 63;
        if (i != j) {
            const float dd = fmaxf(As[i * LDP + i], 0.f) * fmaxf(As[j * LDP + j], 0.f);
            if (dd > 0.f) mo = fmaxf(mo, fabsf(As[i * LDP + j]) * rsqrtf(dd));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mo = fmaxf(mo, __shfl_xor_sync(0xffffffffu, mo, o));
    if (lane == 0) red[warp] = mo;
    __syncthreads();
    mo = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) mo = fmaxf(mo, red[w]);
    rotated = mo > tol_rot;
    if (!rotated) return mo;
    cross_phase(As, Vs, rot, xch, 32, tol_rot);
    if (!cross_only)
        for (int m = 16; m >= 1; m >>= 1) cross_phase(As, Vs, rot, xch, m, tol_rot);
    for (int e = tid; e < BLK * BLK; e += NT) vout[e] = Vs[(e >> 6) * LDP + (e & 63)];
    return mo;
}

// ---- apply phase -------------------------------------------------------------------------------
// x = hi + lo + (less than 2^-21 |x|) with hi and lo in TF32 (low 13 mantissa bits zero): hi is x cut to TF32, lo
// the remainder cut the same way. Two logic operations and one subtraction; the cvt.rna.tf32 conversion would
// round instead of cut, but it is a slow-path instruction and bounded the whole product (2997 -> 2273 cycles).
__device__ __forceinline__ void split_tf32(float x, uint32_t &hi, uint32_t &lo)
{
    hi = __float_as_uint(x) & 0xffffe000u;
    lo = __float_as_uint(x - __uint_as_float(hi)) & 0xffffe000u;
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// acc (this warp's 16 x 32 part of a 64 x 64 result, rows m0.., columns n0..) = As * Bop, K = 64, in
// split precision: x = hi + lo with both parts in TF32, product = lo*hi + hi*lo + hi*hi (the lo*lo term
// is below fp32 rounding). As[m][k] at stride LDA; Bop[k][n] = Bs[k * ldb + n], or Bs[n * ldb + k] when
// B_TRANS. Strides LDA = 68 and LDB = 72 make every fragment load conflict-free.
template <bool B_TRANS>
__device__ __forceinline__ void product64(const float *As, const float *Bs, int ldb, int m0, int n0, float (&acc)[4][4])
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
#pragma unroll 2
    for (int k0 = 0; k0 < BLK; k0 += 8) {
        uint32_t ah[4], al[4];
        split_tf32(As[(m0 + g) * LDA + k0 + t], ah[0], al[0]);
        split_tf32(As[(m0 + g + 8) * LDA + k0 + t], ah[1], al[1]);
        split_tf32(As[(m0 + g) * LDA + k0 + t + 4], ah[2], al[2]);
        split_tf32(As[(m0 + g + 8) * LDA + k0 + t + 4], ah[3], al[3]);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int n = n0 + nt * 8 + g;
            uint32_t bh[2], bl[2];
            if (B_TRANS) {
                split_tf32(Bs[n * ldb + k0 + t], bh[0], bl[0]);
                split_tf32(Bs[n * ldb + k0 + t + 4], bh[1], bl[1]);
            } else {
                split_tf32(Bs[(k0 + t) * ldb + n], bh[0], bl[0]);
                split_tf32(Bs[(k0 + t + 4) * ldb + n], bh[1], bl[1]);
            }
            mma_tf32(acc[nt], al, bh);
            mma_tf32(acc[nt], ah, bl);
            mma_tf32(acc[nt], ah, bh);
        }
    }
}

// General form for other kernels: acc += op(A) * op(B) over K = 64, NPASS = 3 (split precision, as above) or
// 1 (plain TF32, ~2^-11 relative per term). A_TRANS: A[m][k] = As[k * lda + m] (use stride LDB = 72);
// otherwise As[m * lda + k] (stride LDA = 68). B as in product64.
template <bool A_TRANS, bool B_TRANS, int NPASS>
__device__ __forceinline__ void product64_acc(const float *As, int lda, const float *Bs, int ldb, int m0, int n0, float (&acc)[4][4])
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll 2
    for (int k0 = 0; k0 < BLK; k0 += 8) {
        float af[4];
        if (A_TRANS) {
            af[0] = As[(k0 + t) * lda + m0 + g]; af[1] = As[(k0 + t) * lda + m0 + g + 8];
            af[2] = As[(k0 + t + 4) * lda + m0 + g]; af[3] = As[(k0 + t + 4) * lda + m0 + g + 8];
        } else {
            af[0] = As[(m0 + g) * lda + k0 + t]; af[1] = As[(m0 + g + 8) * lda + k0 + t];
            af[2] = As[(m0 + g) * lda + k0 + t + 4]; af[3] = As[(m0 + g + 8) * lda + k0 + t + 4];
        }
        uint32_t ah[4], al[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (NPASS == 3) split_tf32(af[i], ah[i], al[i]);
            else { ah[i] = __float_as_uint(af[i]); al[i] = 0u; }
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int n = n0 + nt * 8 + g;
            float b0, b1;
            if (B_TRANS) { b0 = Bs[n * ldb + k0 + t]; b1 = Bs[n * ldb + k0 + t + 4]; }
            else { b0 = Bs[(k0 + t) * ldb + n]; b1 = Bs[(k0 + t + 4) * ldb + n]; }
            uint32_t bh[2], bl[2];
            if (NPASS == 3) { split_tf32(b0, bh[0], bl[0]); split_tf32(b1, bh[1], bl[1]); }
            else { bh[0] = __float_as_uint(b0); bh[1] = __float_as_uint(b1); }
            if (NPASS == 3) { mma_tf32(acc[nt], al, bh); mma_tf32(acc[nt], ah, bl); }
            mma_tf32(acc[nt], ah, bh);
        }
    }
}

// The same product on the fp32 FMA units, with the ownership layout of the tensor-core version (this
// thread: rows m0 + g and m0 + g + 8, columns n0 + 8 nt + 2 t, + 1). Used for fp32 inputs, whose
// convergence threshold (1e-6) sits below the rounding of the split-precision product (~2^-21).
template <bool B_TRANS>
__device__ __forceinline__ void product64_fma(const float *As, const float *Bs, int ldb, int m0, int n0, float (&acc)[4][4])
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
#pragma unroll 2
    for (int k0 = 0; k0 < BLK; k0 += 4) {
        const float4 a0 = *(const float4 *)(As + (m0 + g) * LDA + k0);
        const float4 a1 = *(const float4 *)(As + (m0 + g + 8) * LDA + k0);
        const float av0[4] = {a0.x, a0.y, a0.z, a0.w}, av1[4] = {a1.x, a1.y, a1.z, a1.w};
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int n = n0 + nt * 8 + 2 * t;
                float b0, b1;
                if (B_TRANS) { b0 = Bs[n * ldb + k0 + kk]; b1 = Bs[(n + 1) * ldb + k0 + kk]; }
                else { const float2 b = *(const float2 *)(Bs + (k0 + kk) * ldb + n); b0 = b.x; b1 = b.y; }
                acc[nt][0] = fmaf(av0[kk], b0, acc[nt][0]); acc[nt][1] = fmaf(av0[kk], b1, acc[nt][1]);
                acc[nt][2] = fmaf(av1[kk], b0, acc[nt][2]); acc[nt][3] = fmaf(av1[kk], b1, acc[nt][3]);
            }
        }
    }
}

// Forms, on chip, the pivot block that a pair of the NEXT step will have once the current step's update is done,
// from the state before that update. The pair's first block sits in half h1 of the current pair p1, its second in
// half h2 of the current pair p2. With W1 / W2 the 32 rows of Vt_p1 / Vt_p2 that produce those blocks (rows of
// the identity where the pair was not rotated: f1 / f2 = 0) and X_ab the old blocks between the pairs a and b,
//   N = [ W1 X11 W1^T   W1 X12 W2^T ]
//       [   (mirror)    W2 X22 W2^T ]
// in three 64^3 products: [W1 X11; W2 X22] and W1 X12 first, then the multiplication by [W1; W2]^T from the
// right. The result lands in As = sm (stride LDP). So the chain of pivot solves never waits for the update.
template <bool TENSOR>
__device__ void pivot_form(float *sm, const Seq &sq, const float *Gsrc, const float *Vcur, int step, int p1, int h1, int f1, int p2, int h2, int f2, unsigned *fetched)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    float *Wc = sm, *S1 = sm + SLOT, *S2 = sm + 2 * SLOT, *S3 = sm + 3 * SLOT;
    int I1, J1, I2, J2;
    rr_pair(sq.nb, step, p1, I1, J1);
    rr_pair(sq.nb, step, p2, I2, J2);
    const int np = sq.np;
    for (int f = tid; f < BLK * (BLK / 4); f += NT) {
        const int i = f >> 4, c = (f & 15) * 4;
        const bool up = i < JB;
        const int row = (up ? h1 : h2) * JB + (i & (JB - 1));
        float4 w;
        if (up ? f1 : f2) w = __ldcg((const float4 *)(Vcur + (size_t)(up ? p1 : p2) * BLK * BLK + row * BLK + c));
        else w = make_float4(row == c ? 1.f : 0.f, row == c + 1 ? 1.f : 0.f, row == c + 2 ? 1.f : 0.f, row == c + 3 ? 1.f : 0.f);
        *(float4 *)(Wc + i * LDA + c) = w;
        const size_t r1 = (size_t)glob_of_loc(I1, J1, i) * np, r2 = (size_t)glob_of_loc(I2, J2, i) * np;
        *(float4 *)(S1 + i * LDB + c) = __ldcg((const float4 *)(Gsrc + r1 + glob_of_loc(I1, J1, c)));
        *(float4 *)(S2 + i * LDB + c) = __ldcg((const float4 *)(Gsrc + r2 + glob_of_loc(I2, J2, c)));
        *(float4 *)(S3 + i * LDB + c) = __ldcg((const float4 *)(Gsrc + r1 + glob_of_loc(I2, J2, c)));
    }
    __syncthreads();
    if (tid == 0) atomicAdd(fetched, 1u);                       // the old blocks are on chip: the update may overwrite them
    const int m0 = (warp & 3) * 16, n0 = (warp >> 2) * 32;
    const bool up = m0 < JB;
    const bool on_tensor = TENSOR;
    float accd[4][4], acco[4][4];
    if (on_tensor) product64<false>(Wc, up ? S1 : S2, LDB, m0, n0, accd);
    else product64_fma<false>(Wc, up ? S1 : S2, LDB, m0, n0, accd);
    if (up) {
        if (on_tensor) product64<false>(Wc, S3, LDB, m0, n0, acco);
        else product64_fma<false>(Wc, S3, LDB, m0, n0, acco);
    }
    __syncthreads();
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const int c = n0 + nt * 8 + 2 * t;
        *(float2 *)(S1 + (m0 + g) * LDA + c) = make_float2(accd[nt][0], accd[nt][1]);
        *(float2 *)(S1 + (m0 + g + 8) * LDA + c) = make_float2(accd[nt][2], accd[nt][3]);
        if (up) {
            *(float2 *)(S2 + (m0 + g) * LDA + c) = make_float2(acco[nt][0], acco[nt][1]);
            *(float2 *)(S2 + (m0 + g + 8) * LDA + c) = make_float2(acco[nt][2], acco[nt][3]);
        }
    }
    __syncthreads();
    const bool lower_left = !up && n0 == 0;                     // mirror of the upper right part
    if (!lower_left) {
        const float *Ta = (up && n0 != 0) ? S2 : S1;
        if (on_tensor) product64<true>(Ta, Wc, LDA, m0, n0, accd);
        else product64_fma<true>(Ta, Wc, LDA, m0, n0, accd);
    }
    __syncthreads();
    float *As = sm;
    if (!lower_left) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int i = m0 + g + (e >> 1) * 8, j = n0 + nt * 8 + 2 * t + (e & 1);
                As[i * LDP + j] = accd[nt][e];
                if (up && n0 != 0) As[j * LDP + i] = accd[nt][e];
            }
    }
}

// The update of a step is cut into strips. A strip of G: blocks (p, q0 .. q0 + cnt - 1) of the upper triangle,
// updated in place together with their mirrors; a strip of Wt: the rows of pair p, column chunks
// c0 .. c0 + cnt - 1 of 64, in place. The pivot CTAs of the same step read blocks of G as they were before the
// update: before its first store of a step a CTA makes sure that all of them have fetched theirs (Fetched). Along a strip Vt_p stays in shared memory and
// the next block is fetched into registers while the current one is multiplied. Short strips win at r~ = 2112: with
// 296 CTAs a step has only a few items per CTA, and the last ones to finish set the time of the step (strips of
// 2 + 3 blocks: 39.9 us per step, 1 + 2: 37.3 us).
constexpr int SEG_G = 1, SEG_W = 2;

__device__ __forceinline__ void store_tile_acc(float *dst, int ld, int m0, int n0, const float (&acc)[4][4])
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const int c = n0 + nt * 8 + 2 * t;
        *(float2 *)(dst + (m0 + g) * ld + c) = make_float2(acc[nt][0], acc[nt][1]);
        *(float2 *)(dst + (m0 + g + 8) * ld + c) = make_float2(acc[nt][2], acc[nt][3]);
    }
}

struct Fetched {
    const unsigned *count; unsigned target; int *abort_flag;   // counter of pivot blocks fetched in this step, its final value
    bool ok;                                                    // already seen complete by this CTA
};
// Block-uniform, bounded: false when the wait ran out.
__device__ bool wait_fetched(Fetched &f)
{
    if (f.ok) return true;
    __shared__ int ok_s;
    if (threadIdx.x == 0) {
        int ok = 0;
        for (unsigned i = 0; i < SPIN_LIMIT; ++i) {
            if (*(volatile const unsigned *)f.count >= f.target) { ok = 1; break; }
            if ((i & 1023u) == 1023u && *(volatile int *)f.abort_flag) break;
        }
        if (!ok) *(volatile int *)f.abort_flag = 1;
        ok_s = ok;
    }
    __syncthreads();
    f.ok = ok_s != 0;
    return f.ok;
}

template <bool TENSOR>
__device__ bool g_strip(float *sm, const Seq &sq, float *G, const float *Vbuf, const int *vflag, int step, int p, int q0, int cnt, Fetched &fetched)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int m0 = (warp & 3) * 16, n0 = (warp >> 2) * 32, np = sq.np;
    float *Vp = sm, *Vq = sm + BLK * LDA, *Tm = sm + 2 * BLK * LDA, *Bk = sm + 3 * BLK * LDA;
    const int fp = __ldcg(vflag + p);
    int Ip, Jp;
    rr_pair(sq.nb, step, p, Ip, Jp);
    float4 x[4];
    auto fetch = [&](int q) {
        int Iq, Jq;
        rr_pair(sq.nb, step, q, Iq, Jq);
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int f = tid + it * NT, i = f >> 4, c = (f & 15) * 4;
            x[it] = __ldcg((const float4 *)(G + (size_t)glob_of_loc(Ip, Jp, i) * np + glob_of_loc(Iq, Jq, c)));
        }
    };
    if (fp) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int f = tid + it * NT, i = f >> 4, c = (f & 15) * 4;
            *(float4 *)(Vp + i * LDA + c) = __ldcg((const float4 *)(Vbuf + (size_t)p * BLK * BLK + i * BLK + c));
        }
    }
    fetch(q0);
    for (int j = 0; j < cnt; ++j) {
        const int q = q0 + j, fq = __ldcg(vflag + q);
        int Iq, Jq;
        rr_pair(sq.nb, step, q, Iq, Jq);
        if (!fp && !fq) {                                        // unchanged block
            if (j + 1 < cnt) fetch(q + 1);
            continue;
        }
        // the block goes to the B tile when a row transform comes first, else straight to the T tile
        float *blk_dst = fp ? Bk : Tm;
        const int blk_ld = fp ? LDB : LDA;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int f = tid + it * NT, i = f >> 4, c = (f & 15) * 4;
            *(float4 *)(blk_dst + i * blk_ld + c) = x[it];
            if (fq) *(float4 *)(Vq + i * LDA + c) = __ldcg((const float4 *)(Vbuf + (size_t)q * BLK * BLK + i * BLK + c));
        }
        __syncthreads();
        if (j + 1 < cnt) fetch(q + 1);
        float acc[4][4];
        if (fp) {
            if (TENSOR) product64<false>(Vp, Bk, LDB, m0, n0, acc);  // T = Vt_p * block
            else product64_fma<false>(Vp, Bk, LDB, m0, n0, acc);
            if (fq) {
                store_tile_acc(Tm, LDA, m0, n0, acc);
                __syncthreads();
            }
        }
        if (fq) {                                                // out = T * Vt_q^T
            if (TENSOR) product64<true>(Tm, Vq, LDA, m0, n0, acc);
            else product64_fma<true>(Tm, Vq, LDA, m0, n0, acc);
        }
        if (!wait_fetched(fetched)) return false;
        const int gr0 = glob_of_loc(Ip, Jp, m0 + g), gr1 = glob_of_loc(Ip, Jp, m0 + g + 8);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int gc = glob_of_loc(Iq, Jq, n0 + nt * 8 + 2 * t);     // gc, gc + 1 are contiguous
            *(float2 *)(G + (size_t)gr0 * np + gc) = make_float2(acc[nt][0], acc[nt][1]);
            *(float2 *)(G + (size_t)gr1 * np + gc) = make_float2(acc[nt][2], acc[nt][3]);
            if (q != p) {                                        // mirror block
                G[(size_t)gc * np + gr0] = acc[nt][0]; G[(size_t)(gc + 1) * np + gr0] = acc[nt][1];
                G[(size_t)gc * np + gr1] = acc[nt][2]; G[(size_t)(gc + 1) * np + gr1] = acc[nt][3];
            }
        }
        __syncthreads();                                         // tiles are reused by the next block
    }
    return true;
}

template <bool TENSOR>
__device__ void wt_strip(float *sm, const Seq &sq, const float *Vbuf, const int *vflag, int step, int p, int c0, int cnt)
{
    if (!__ldcg(vflag + p)) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int m0 = (warp & 3) * 16, n0 = (warp >> 2) * 32, np = sq.np;
    float *Vp = sm, *Bk = sm + 3 * BLK * LDA;
    int Ip, Jp;
    rr_pair(sq.nb, step, p, Ip, Jp);
    float4 x[4];
    auto fetch = [&](int chunk) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int f = tid + it * NT, i = f >> 4, c = (f & 15) * 4;
            x[it] = __ldcg((const float4 *)(sq.Wt + (size_t)glob_of_loc(Ip, Jp, i) * np + chunk * BLK + c));
        }
    };
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int f = tid + it * NT, i = f >> 4, c = (f & 15) * 4;
        *(float4 *)(Vp + i * LDA + c) = __ldcg((const float4 *)(Vbuf + (size_t)p * BLK * BLK + i * BLK + c));
    }
    fetch(c0);
    const int gr0 = glob_of_loc(Ip, Jp, m0 + g), gr1 = glob_of_loc(Ip, Jp, m0 + g + 8);
    for (int j = 0; j < cnt; ++j) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int f = tid + it * NT, i = f >> 4, c = (f & 15) * 4;
            *(float4 *)(Bk + i * LDB + c) = x[it];
        }
        __syncthreads();
        if (j + 1 < cnt) fetch(c0 + j + 1);
        float acc[4][4];
        if (TENSOR) product64<false>(Vp, Bk, LDB, m0, n0, acc);
        else product64_fma<false>(Vp, Bk, LDB, m0, n0, acc);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int gc = (c0 + j) * BLK + n0 + nt * 8 + 2 * t;
            *(float2 *)(sq.Wt + (size_t)gr0 * np + gc) = make_float2(acc[nt][0], acc[nt][1]);
            *(float2 *)(sq.Wt + (size_t)gr1 * np + gc) = make_float2(acc[nt][2], acc[nt][3]);
        }
        __syncthreads();                                         // the B tile is reused by the next chunk
    }
}

// Work items of the update: first the strips of G (row by row of the upper triangle), then the strips of Wt.
__host__ __device__ __forceinline__ int strips_of_g(int npairs)
{
    int n = 0;
    for (int p = 0; p < npairs; ++p) n += (npairs - p + SEG_G - 1) / SEG_G;
    return n;
}
template <bool TENSOR>
__device__ bool apply_item(float *sm, const Seq &sq, const float *Vbuf, const int *vflag, int step, int idx, int npairs, int items_g, int nw, Fetched &fetched)
{
    if (idx < items_g) {
        int p = 0;
        for (;;) {
            const int n = (npairs - p + SEG_G - 1) / SEG_G;
            if (idx < n) break;
            idx -= n; ++p;
        }
        const int q0 = p + idx * SEG_G;
        return g_strip<TENSOR>(sm, sq, sq.G, Vbuf, vflag, step, p, q0, min(SEG_G, npairs - q0), fetched);
    } else {
        idx -= items_g;
        const int nseg = (nw + SEG_W - 1) / SEG_W, p = idx / nseg, c0 = (idx - p * nseg) * SEG_W;
        wt_strip<TENSOR>(sm, sq, Vbuf, vflag, step, p, c0, min(SEG_W, nw - c0));
    }
    return true;
}

// ---- the kernel --------------------------------------------------------------------------------
// Schedule of a group. The pivot block of a pair of step s+1 is a function of the matrix before the update of
// step s and of two transforms of step s (pivot_form), all of which are complete at the barrier that ends step
// s-1. Every step therefore runs, side by side,
//   1. the pivot solves of the NEXT step (a few CTAs; this chain of rotation rounds is the critical path), and
//   2. the update of this step, its blocks handed out by a ticket counter so that the pivot CTAs join in when
//      they are through,
// followed by one group barrier. The update works in place; before its first store of a step a CTA waits
// (as a rule not at all: it has a block to load and multiply first) until every pivot CTA has fetched the
// blocks it forms its pivot block from. Vt and the rotated-flags are double buffered by step parity, because
// the pivots of step s+1 publish while the update of step s still reads.
// status[0]: sticky device status word of the context; status[1]: abort flag of bounded waits.
constexpr int MAXPAIRS = 72;                  // np <= 4608

template <bool TENSOR>
__global__ void __launch_bounds__(NT, 2)
jacobi_persistent_kernel(const __grid_constant__ Batch batch, float tol_conv, float tol_rot, int max_sweeps,
                         int raise_not_converged, int *status)
{
    extern __shared__ __align__(16) float j3sm[];
    __shared__ short pair_of[2 * MAXPAIRS];       // block -> 2 * pair + half, for the current step
    __shared__ int ticket_s;
    int si = 0;
#pragma unroll 1
    for (int i = 1; i < batch.count; ++i) if ((int)blockIdx.x >= batch.s[i].cta0) si = i;
    const Seq &sq = batch.s[si];
    const int rank = (int)blockIdx.x - sq.cta0, tid = threadIdx.x;
    if (rank >= sq.ncta || sq.np <= 0) return;
    const int npairs = sq.nb / 2, nw = sq.np / BLK;
    const int items_g = strips_of_g(npairs), total = items_g + npairs * ((nw + SEG_W - 1) / SEG_W);
    const int nsteps = sq.nb - 1;
    int *abort_flag = status + 1;
    unsigned gen = 0, gstep = 0;
    bool converged = false, alive = true;

    // rotates the block held in shared memory for pair pr of (sweep, step); publishes to parity par
    auto pivot_finish = [&](int sweep, int step, int pr, int par) {
        bool rotated;
        const float mo = pivot_rotate(j3sm, step > 0, tol_rot, sq.Vbuf + ((size_t)par * npairs + pr) * BLK * BLK, rotated);
        if (tid == 0) {
            sq.vflag[par * npairs + pr] = rotated ? 1 : 0;
            atomicMax(sq.sync + 1 + sweep % 4, __float_as_uint(mo));
        }
        __syncthreads();
    };

    // prologue: the pivots of the very first step, straight from G
    for (int pr = rank; pr < npairs; pr += sq.ncta) {
        int I, J;
        rr_pair(sq.nb, 0, pr, I, J);
        pivot_load(j3sm, sq.G, sq.np, I, J);
        pivot_finish(0, 0, pr, 0);
    }
    alive = group_barrier(sq.sync, ++gen, (unsigned)sq.ncta, abort_flag);

    int sweep = 0;
    for (; sweep < max_sweeps && alive; ++sweep) {
        if (rank == 0 && tid == 0) sq.sync[1 + (sweep + 2) % 4] = 0u;      // slot of sweep + 2, last read two sweeps ago
        for (int step = 0; step < nsteps && alive; ++step, ++gstep) {
            const int par = (int)(gstep & 1u);
            const bool has_next = !(sweep == max_sweeps - 1 && step == nsteps - 1);
            const int nstep = step + 1 == nsteps ? 0 : step + 1, nsweep = sweep + (step + 1 == nsteps ? 1 : 0);
            const float *Vcur = sq.Vbuf + (size_t)par * npairs * BLK * BLK;
            const int *fcur = sq.vflag + par * npairs;
            // a step in which no pair was rotated needs no update
            const bool any_rot = __syncthreads_or(tid < npairs && __ldcg(fcur + tid) != 0) != 0;
            if (rank == 0 && tid == 0) {                                  // tickets and fetch count of the next step
                sq.sync[16 + (par ^ 1)] = 0u;
                sq.sync[20 + (par ^ 1)] = 0u;
            }
            Fetched fetched{sq.sync + 20 + par, has_next ? (unsigned)npairs : 0u, abort_flag, false};
            // 1. pivots of the next step
            if (has_next && rank < npairs) {
                if (tid < npairs) {
                    int I, J;
                    rr_pair(sq.nb, step, tid, I, J);
                    pair_of[I] = (short)(2 * tid); pair_of[J] = (short)(2 * tid + 1);
                }
                __syncthreads();
                for (int pr = rank; pr < npairs; pr += sq.ncta) {
                    int I2, J2;
                    rr_pair(sq.nb, nstep, pr, I2, J2);
                    const int p1 = pair_of[I2] >> 1, h1 = pair_of[I2] & 1, p2 = pair_of[J2] >> 1, h2 = pair_of[J2] & 1;
                    const int f1 = __ldcg(fcur + p1), f2 = __ldcg(fcur + p2);
                    if (!f1 && !f2) {
                        pivot_load(j3sm, sq.G, sq.np, I2, J2);
                        __syncthreads();
                        if (tid == 0) atomicAdd(sq.sync + 20 + par, 1u);
                    } else pivot_form<TENSOR>(j3sm, sq, sq.G, Vcur, step, p1, h1, f1, p2, h2, f2, sq.sync + 20 + par);
                    pivot_finish(nsweep, nstep, pr, par ^ 1);
                }
            }
            // 2. the update, by tickets (the next one is requested while a block is processed)
            if (tid == 0) ticket_s = any_rot ? (int)atomicAdd(sq.sync + 16 + par, 1u) : total;
            __syncthreads();
            int t = ticket_s;
            while (t < total && alive) {
                int tn = 0;
                if (tid == 0) tn = (int)atomicAdd(sq.sync + 16 + par, 1u);
                alive = apply_item<TENSOR>(j3sm, sq, Vcur, fcur, step, t, npairs, items_g, nw, fetched);
                __syncthreads();
                if (tid == 0) ticket_s = tn;
                __syncthreads();
                t = ticket_s;
            }
            alive = group_barrier(sq.sync, ++gen, (unsigned)sq.ncta, abort_flag) && alive;
        }
        if (!alive) break;
        const float mo = __uint_as_float(*(volatile unsigned *)(sq.sync + 1 + sweep % 4));
        if (mo <= tol_conv) { converged = true; ++sweep; break; }
    }
    if (rank == 0 && tid == 0) {
        if (!alive) raise_status(status, ATP_ERR_TIMEOUT);
        else if (!converged && raise_not_converged) raise_status(status, ATP_ERR_NOT_CONVERGED);
        sq.sync[5] = (unsigned)sweep;
    }
}

// Wt = identity, padding of G = 0, synchronisation words = 0; a non-finite entry of G (an input with Inf / NaN,
// or one whose squares overflow fp32) raises ATP_ERR_RANGE. grid (x, count).
__global__ void init_kernel(const __grid_constant__ Batch batch, int *status)
{
    bool bad = false;
    const Seq &sq = batch.s[blockIdx.y];
    const size_t n2 = (size_t)sq.np * sq.np;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n2; e += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / sq.np), j = (int)(e - (size_t)i * sq.np);
        sq.Wt[e] = (i == j) ? 1.f : 0.f;
        if (i >= sq.n || j >= sq.n) sq.G[e] = 0.f;
        else if (!isfinite(sq.G[e])) bad = true;
    }
    if (__syncthreads_or(bad) && threadIdx.x == 0) raise_status(status, ATP_ERR_RANGE);
    if (blockIdx.x == 0 && sq.np > 0) {
        if (threadIdx.x < 64) sq.sync[threadIdx.x] = 0u;
    }
}

// Host side: hands every sequence a group of CTAs in proportion to the size of its update (at most one
// CTA per block of the update, at least one) and launches the kernel cooperatively, so that all
// groups are resident together and the group barriers cannot starve.
template <bool TENSOR>
static inline atp_status launch(atp_ctx *ctx, Batch &jb, float tol_conv, float tol_rot, int max_sweeps, bool raise_not_converged)
{
    if (jb.count <= 0) return ATP_OK;
    static std::mutex mu;
    static int occ_dev[64] = {};
    int occ = 0;
    {
        std::lock_guard<std::mutex> lk(mu);
        const int dv = ctx->device;
        if (dv < 0 || dv >= 64 || occ_dev[dv] == 0) {
            ATP_CUDA_OK(ctx, cudaFuncSetAttribute(jacobi_persistent_kernel<TENSOR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
            ATP_CUDA_OK(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, jacobi_persistent_kernel<TENSOR>, NT, SMEM_BYTES));
            if (occ < 1) return ATP_ERR_CUDA;
            if (dv >= 0 && dv < 64) occ_dev[dv] = occ;
        } else occ = occ_dev[dv];
    }
    const int total = ctx->sm_count * std::min(occ, 2);
    double wsum = 0;
    for (int i = 0; i < jb.count; ++i) wsum += (double)jb.s[i].np * jb.s[i].np;
    if (wsum <= 0) return ATP_OK;
    int next = 0;
    for (int i = 0; i < jb.count; ++i) {
        Seq &q = jb.s[i];
        const int npairs = q.nb / 2;
        int items = npairs * ((q.np / BLK + SEG_W - 1) / SEG_W);                 // strips of the update
        for (int pp = 0; pp < npairs; ++pp) items += (npairs - pp + SEG_G - 1) / SEG_G;
        int c = (int)((double)total * ((double)q.np * q.np / wsum));
        c = std::max(1, std::min(c, std::max(items, 1)));
        if (q.np <= 0) c = 1;
        q.cta0 = next; q.ncta = c;
        next += c;
    }
    if (next > total) return ATP_ERR_INVALID_ARG;      // cannot happen: shares sum to at most `total`
    ATP_KERNEL(ctx, "jacobi_init", 0, wsum * 4.0);
    init_kernel<<<dim3(std::max(64, 4 * ctx->sm_count / jb.count), jb.count), 256, 0, ctx->stream>>>(jb, ctx->dev_status);
    ATP_LAUNCHED(ctx);
    int *status = ctx->dev_status;
    int ms = max_sweeps, rn = raise_not_converged ? 1 : 0;
    void *args[] = {(void *)&jb, (void *)&tol_conv, (void *)&tol_rot, (void *)&ms, (void *)&rn, (void *)&status};
    // bytes: one read and one write of G and Wt (what the kernel must move at least; it runs from L2)
    ATP_KERNEL(ctx, "jacobi_persistent", 0, wsum * 16.0);
    ATP_CUDA_OK(ctx, cudaLaunchCooperativeKernel((const void *)jacobi_persistent_kernel<TENSOR>, dim3(next), dim3(NT), args, SMEM_BYTES, ctx->stream));
    ATP_LAUNCHED(ctx);
    return ATP_OK;
}

}  // namespace j3
