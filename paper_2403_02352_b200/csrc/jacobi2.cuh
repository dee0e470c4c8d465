// Two-sided block Jacobi eigensolver for the small Gram matrix G = B B^T (r~ x r~, fp32, resident in
// L2): the rotation that diagonalises G turns the orthonormal range basis into singular vectors
// (Rayleigh-Ritz step of the basis extraction, Sec. 4.2: X' = [sigma_i v_i]).
// Blocks of 16 rows; a step handles r~/32 disjoint pairs (round-robin order) with two launches:
//   jac2_local : per pair, the 32x32 diagonal block is swept on chip (cyclic Jacobi: all its pairs in
//                the first step of a sweep, when every block meets exactly one partner, and only the
//                pairs that couple the two blocks in the other steps, so that a sweep rotates every
//                pair of rows exactly once), the accumulated row operations Vt are published
//                (stored transposed);
//   jac2_apply : every 32x32 block (p, q) becomes Vt_p G_pq Vt_q^T, rows of Wt become Vt_p Wt.
// G entries carry errors relative to the norms of the rows of B they come from (B is graded by the
// QR-ordered range basis), which is what Jacobi needs to resolve small eigenvalues next to large ones.
#pragma once
#include "common.cuh"

constexpr int J2MAX = 32;         // sequences per launch

struct Jac2Seq { float *G; float *Wt; float *Vbuf; int *vflag; int rt, nb; unsigned *maxoff; int *conv; };
struct Jac2Batch { Jac2Seq s[J2MAX]; int count; };

__device__ __forceinline__ void rr_pair2(int nb, int step, int t, int &I, int &J)
{
    int m = nb - 1;
    if (t == 0) { I = m; J = step % m; }
    else { I = (step + t) % m; J = (step - t + m) % m; }
    if (I > J) { int x = I; I = J; J = x; }
}
template <int BJ2>
__device__ __forceinline__ int jac2_row(int I, int J, int i, int rt)
{
    int g = (i < BJ2) ? I * BJ2 + i : J * BJ2 + (i - BJ2);
    return g < rt ? g : -1;
}

__global__ void jac2_init_kernel(const __grid_constant__ Jac2Batch batch)
{
    const Jac2Seq &sq = batch.s[blockIdx.y];
    size_t n = (size_t)sq.rt * sq.rt;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        int i = (int)(e / sq.rt), k = (int)(e - (size_t)i * sq.rt);
        sq.Wt[e] = (i == k) ? 1.f : 0.f;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { *sq.maxoff = 0u; *sq.conv = 0; }
}

// Rotation (c, s) that annihilates the (p, q) entry of a symmetric matrix; identity when the entry is
// already small against its diagonal. With a = g_qq - g_pp, b = 2 g_pq, r = sqrt(a^2 + b^2):
//   cos 2t = |a| / r,  c = sqrt((1 + cos 2t) / 2),  s = sign(a) b / (2 r c)      (|t| <= pi/4),
// two reciprocal square roots in a row instead of two divisions and two roots; c^2 + s^2 = 1 to a few
// ulp, ample for a basis stored in bf16. a and b are rescaled when their squares would leave the
// fp32 range.
__device__ __forceinline__ float2 jac2_rotation(float gpp, float gqq, float gpq, float tol_rot, bool &did)
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
        did = true;
    }
    return make_float2(c, s);
}

// BJ2: block height (16 or 32); the local problem is BLK x BLK with BLK = 2 BJ2, solved by (BLK/2)^2
// threads. The sweep is a chain of BLK - 1 dependent rotation steps, so the time of a step is the
// length of one thread's instruction chain plus ONE block barrier: thread (a, b) owns, in every step,
// the 2x2 block (rows of pair a, columns of pair b) of A and the two column pairs {2b, 2b+1} of the rows
// of pair a of V. It derives the two rotations it needs (pair a, pair b) itself from the previous step's
// A (all threads that need a rotation compute the same values from the same inputs), reads A from one
// buffer and writes the other.
#define JAC2_LOCAL_SMEM(BLK) ((size_t)(3 * (BLK) * ((BLK) + 1)) * sizeof(float))
template <int BJ2>
__global__ void __launch_bounds__(BJ2 * BJ2)
jac2_local_kernel(const __grid_constant__ Jac2Batch batch, int step, float tol_rot, int max_inner, int cross_only)
{
    constexpr int BLK = 2 * BJ2, HP = BLK / 2, NT = HP * HP;
    pdl_trigger();
    const Jac2Seq &sq = batch.s[blockIdx.y];
    const int npairs = sq.nb / 2;
    const int pair = blockIdx.x;
    int I, J;
    rr_pair2(sq.nb, step % (sq.nb - 1), pair < npairs ? pair : 0, I, J);
    extern __shared__ __align__(16) float j2l[];       // JAC2_LOCAL_SMEM(BLK) bytes
    float (*Ab)[BLK][BLK + 1] = (float (*)[BLK][BLK + 1])j2l;                     // two copies of A
    float (*V)[BLK + 1] = (float (*)[BLK + 1])(j2l + 2 * BLK * (BLK + 1));
    __shared__ float red[NT / 32];
    __shared__ int rotated;
    __shared__ uchar2 sched[BLK - 1][HP];              // round-robin schedule of the local sweep
    const int tid = threadIdx.x;
    // cross_only: the BJ2 steps that pair every row of block I with every row of block J once; otherwise
    // the full round-robin over all BLK rows (which also rotates the pairs inside I and inside J)
    const int nsteps = cross_only ? BJ2 : BLK - 1;
    for (int e = tid; e < nsteps * HP; e += NT) {
        int p_, q_;
        if (cross_only) { p_ = e % HP; q_ = BJ2 + (e % HP + e / HP) % BJ2; }
        else rr_pair2(BLK, e / HP, e % HP, p_, q_);
        sched[e / HP][e % HP] = make_uchar2((unsigned char)p_, (unsigned char)q_);
    }
    pdl_wait();                                        // nothing above touches global memory
    if (pair >= npairs || *sq.conv) return;
    for (int e = tid; e < BLK * BLK; e += NT) {
        int i = e / BLK, j = e % BLK;
        int gi = jac2_row<BJ2>(I, J, i, sq.rt), gj = jac2_row<BJ2>(I, J, j, sq.rt);
        Ab[0][i][j] = (gi >= 0 && gj >= 0) ? sq.G[(size_t)gi * sq.rt + gj] : 0.f;
        V[i][j] = (i == j) ? 1.f : 0.f;
    }
    if (tid == 0) rotated = 0;
    __syncthreads();
    float mo = 0.f;
    for (int e = tid; e < BLK * BLK; e += NT) {
        int i = e / BLK, j = e % BLK;
        if (i != j) {
            const float dd = fmaxf(Ab[0][i][i], 0.f) * fmaxf(Ab[0][j][j], 0.f);
            if (dd > 0.f) mo = fmaxf(mo, fabsf(Ab[0][i][j]) * rsqrtf(dd));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mo = fmaxf(mo, __shfl_xor_sync(0xffffffffu, mo, o));
    if ((tid & 31) == 0) red[tid >> 5] = mo;
    __syncthreads();
    mo = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) mo = fmaxf(mo, red[w]);
    if (tid == 0) atomicMax(sq.maxoff, __float_as_uint(mo));
    if (mo <= tol_rot) {
        if (tid == 0) sq.vflag[pair] = 0;
        return;
    }
    const int ba = tid / HP, bb = tid % HP;            // 2x2 block (pair ba rows, pair bb columns)
    int cur = 0;
    for (int sweep = 0; sweep < max_inner; ++sweep) {
        for (int st = 0; st < nsteps; ++st) {
            const float (*Ao)[BLK + 1] = Ab[cur];
            float (*An)[BLK + 1] = Ab[cur ^ 1];
            const uchar2 ra = sched[st][ba], rb = sched[st][bb];
            // loads of this step first (independent), then the arithmetic, then the stores
            const float bpp = Ao[rb.x][rb.x], bqq = Ao[rb.y][rb.y], bpq = Ao[rb.x][rb.y];
            const float g00 = Ao[ra.x][rb.x], g01 = Ao[ra.x][rb.y], g10 = Ao[ra.y][rb.x], g11 = Ao[ra.y][rb.y];
            const int vc = 2 * bb;
            const float v00 = V[ra.x][vc], v01 = V[ra.x][vc + 1], v10 = V[ra.y][vc], v11 = V[ra.y][vc + 1];
            bool did = false;
            // lane l derives the rotation of pair l mod HP (its column pair); the row pair's comes by shuffle
            const float2 cb = jac2_rotation(bpp, bqq, bpq, tol_rot, did);
            float2 ca;
            ca.x = __shfl_sync(0xffffffffu, cb.x, ba & 31);
            ca.y = __shfl_sync(0xffffffffu, cb.y, ba & 31);
            const float r00 = ca.x * g00 - ca.y * g10, r01 = ca.x * g01 - ca.y * g11;
            const float r10 = ca.y * g00 + ca.x * g10, r11 = ca.y * g01 + ca.x * g11;
            An[ra.x][rb.x] = cb.x * r00 - cb.y * r01; An[ra.x][rb.y] = cb.y * r00 + cb.x * r01;
            An[ra.y][rb.x] = cb.x * r10 - cb.y * r11; An[ra.y][rb.y] = cb.y * r10 + cb.x * r11;
            V[ra.x][vc] = ca.x * v00 - ca.y * v10; V[ra.x][vc + 1] = ca.x * v01 - ca.y * v11;
            V[ra.y][vc] = ca.y * v00 + ca.x * v10; V[ra.y][vc + 1] = ca.y * v01 + ca.x * v11;
            if (did && max_inner > 1) rotated = 1;
            cur ^= 1;
            __syncthreads();
        }
        if (max_inner > 1) {
            const int any = rotated;
            __syncthreads();
            if (!any) break;
            if (tid == 0) rotated = 0;
            __syncthreads();
        }
    }
    float *dst = sq.Vbuf + (size_t)pair * BLK * BLK;
    for (int e = tid; e < BLK * BLK; e += NT) dst[e] = V[e % BLK][e / BLK];   // transposed: what jac2_apply reads
    if (tid == 0) sq.vflag[pair] = 1;
}

// grid: (npairs (npairs + 1) / 2 + npairs ceil(rt/BLK), 1, batch); dynamic shared memory: JAC2_APPLY_SMEM(BLK) bytes.
// G is symmetric: only blocks (p, q) with q >= p are computed, the mirror block is written from the
// transposed register tile. Each thread owns an MR x 4 tile (MR = 2 or 4) of the BLK x BLK block; every shared-memory
// operand is read as one 16-byte vector per 16 multiply-adds, and when the row length of G is a multiple
// of four the global traffic is 16-byte vectors too (the 16 or 32 columns of a block are contiguous).
#define JAC2_APPLY_SMEM(BLK) ((size_t)(4 * (BLK) * ((BLK) + 4)) * sizeof(float))
template <int BJ2, int MR>
__global__ void __launch_bounds__(BJ2 * BJ2 / MR, BJ2 == 16 ? 12 : 1)      // 12 CTAs per SM: one wave at batch 16, r~ = 320
jac2_apply_kernel(const __grid_constant__ Jac2Batch batch, int step)
{
    constexpr int BLK = 2 * BJ2, NT = BLK * BLK / (4 * MR), LD4 = BLK + 4, Q = BLK / 4;   // Q: 4-vectors per row
    pdl_trigger();
    const Jac2Seq &sq = batch.s[blockIdx.z];
    const int npairs = sq.nb / 2;
    // blockIdx.x enumerates the blocks (p, q >= p) of the upper triangle row by row, then the
    // (pair, column chunk) blocks of Wt
    const int ntri = npairs * (npairs + 1) / 2, nw = (sq.rt + BLK - 1) / BLK;
    int idx = blockIdx.x;
    const bool in_range = idx < ntri + npairs * nw;
    if (!in_range) idx = 0;
    const bool gblock = idx < ntri;
    int p = 0, q = 0, wchunk = 0;
    if (gblock) {
        while (idx >= npairs - p) { idx -= npairs - p; ++p; }
        q = p + idx;
    } else {
        idx -= ntri;
        p = idx / nw; wchunk = idx - p * nw;
    }
    pdl_wait();                             // nothing above touches global memory
    if (!in_range) return;
    // the three flags travel together (one memory latency), then the decision
    const int conv = *sq.conv;
    const int fp = sq.vflag[p];
    const int fq = gblock ? sq.vflag[q] : 0;
    if (conv) return;
    if (gblock ? (!fp && !fq) : !fp) return;
    const int tid = threadIdx.x;
    const int rt = sq.rt;
    const bool vec = (rt & 3) == 0;
    extern __shared__ __align__(16) float j2sm[];
    float *VpT = j2sm;                      // [BLK][LD4]  VpT[k][r] = Vt_p[r][k]
    float *TmT = VpT + BLK * LD4;           // [BLK][LD4]  TmT[k][r] = T[r][k]
    float *Bk = TmT + BLK * LD4;            // [BLK][LD4]  B[k][c]
    float *VqT = Bk + BLK * LD4;            // [BLK][LD4]  VqT[k][c] = Vt_q[c][k]
    int Ip, Jp, Iq = 0, Jq = 0;
    rr_pair2(sq.nb, step % (sq.nb - 1), p, Ip, Jp);
    const int cb = wchunk * BLK;
    if (gblock) rr_pair2(sq.nb, step % (sq.nb - 1), q, Iq, Jq);
    // global column of local column c (a multiple of 4): the 4-vector starting there is contiguous
    auto gcol = [&](int c) -> int { return gblock ? ((c < BJ2) ? Iq * BJ2 + c : Jq * BJ2 + (c - BJ2)) : cb + c; };
    auto grow = [&](int r) -> int { return (r < BJ2) ? Ip * BJ2 + r : Jp * BJ2 + (r - BJ2); };
    const float *src_b = gblock ? sq.G : sq.Wt;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int f = tid; f < BLK * Q; f += NT) {
        const int i = f / Q, c = (f % Q) * 4;
        // the published rotations are stored transposed: element (k, r) of the copy is Vt[r][k]
        float4 vp = fp ? *(const float4 *)(sq.Vbuf + (size_t)p * BLK * BLK + i * BLK + c)
                       : make_float4(i == c ? 1.f : 0.f, i == c + 1 ? 1.f : 0.f, i == c + 2 ? 1.f : 0.f, i == c + 3 ? 1.f : 0.f);
        *(float4 *)&VpT[i * LD4 + c] = vp;
        if (gblock) {
            float4 vq = fq ? *(const float4 *)(sq.Vbuf + (size_t)q * BLK * BLK + i * BLK + c)
                           : make_float4(i == c ? 1.f : 0.f, i == c + 1 ? 1.f : 0.f, i == c + 2 ? 1.f : 0.f, i == c + 3 ? 1.f : 0.f);
            *(float4 *)&VqT[i * LD4 + c] = vq;
        }
        const int gi = grow(i), gc = gcol(c);
        float4 bv = zero4;
        if (gi < rt) {
            const float *src = src_b + (size_t)gi * rt + gc;
            if (vec) { if (gc < rt) bv = *(const float4 *)src; }
            else {
                if (gc < rt) bv.x = src[0];
                if (gc + 1 < rt) bv.y = src[1];
                if (gc + 2 < rt) bv.z = src[2];
                if (gc + 3 < rt) bv.w = src[3];
            }
        }
        *(float4 *)&Bk[i * LD4 + c] = bv;
    }
    __syncthreads();
    const int r0 = (tid / Q) * MR, c0 = (tid % Q) * 4;
    float acc[MR][4];
    // acc = (rows r0.. of the operand stored transposed in At) * Bm
    auto product = [&](const float *At, const float *Bm) {
#pragma unroll
        for (int i = 0; i < MR; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll
        for (int k = 0; k < BLK; ++k) {
            float av[MR];
            if (MR == 4) { const float4 a = *(const float4 *)&At[k * LD4 + r0]; av[0] = a.x; av[1] = a.y; av[MR - 2] = a.z; av[MR - 1] = a.w; }
            else { const float2 a = *(const float2 *)&At[k * LD4 + r0]; av[0] = a.x; av[1] = a.y; }
            const float4 b = *(const float4 *)&Bm[k * LD4 + c0];
#pragma unroll
            for (int i = 0; i < MR; ++i) {
                acc[i][0] = fmaf(av[i], b.x, acc[i][0]); acc[i][1] = fmaf(av[i], b.y, acc[i][1]);
                acc[i][2] = fmaf(av[i], b.z, acc[i][2]); acc[i][3] = fmaf(av[i], b.w, acc[i][3]);
            }
        }
    };
    product(VpT, Bk);                       // T = Vt_p * B
    if (!gblock) {                          // rows of Wt: Vt_p * Wt
        const int gc = cb + c0;
#pragma unroll
        for (int i = 0; i < MR; ++i) {
            const int gi = grow(r0 + i);
            if (gi >= rt || gc >= rt) continue;
            float *dst = sq.Wt + (size_t)gi * rt + gc;
            if (vec) *(float4 *)dst = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
            else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (gc + j < rt) dst[j] = acc[i][j];
            }
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (MR == 4) *(float4 *)&TmT[(c0 + j) * LD4 + r0] = make_float4(acc[0][j], acc[1][j], acc[MR - 2][j], acc[MR - 1][j]);
        else *(float2 *)&TmT[(c0 + j) * LD4 + r0] = make_float2(acc[0][j], acc[1][j]);
    }
    __syncthreads();
    product(TmT, VqT);                      // Out = T * Vt_q^T
    const int gi0 = grow(r0), gj0 = gcol(c0);   // rows gi0.. and columns gj0..gj0+3 are contiguous
#pragma unroll
    for (int i = 0; i < MR; ++i) {
        if (gi0 + i >= rt || gj0 >= rt) continue;
        float *dst = sq.G + (size_t)(gi0 + i) * rt + gj0;
        if (vec) *(float4 *)dst = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        else {
#pragma unroll
            for (int j = 0; j < 4; ++j) if (gj0 + j < rt) dst[j] = acc[i][j];
        }
    }
    if (q != p) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (gj0 + j >= rt || gi0 >= rt) continue;
            float *dst = sq.G + (size_t)(gj0 + j) * rt + gi0;
            if (vec && MR == 4) *(float4 *)dst = make_float4(acc[0][j], acc[1][j], acc[MR - 2][j], acc[MR - 1][j]);
            else if (vec) *(float2 *)dst = make_float2(acc[0][j], acc[1][j]);
            else {
#pragma unroll
                for (int i = 0; i < MR; ++i) if (gi0 + i < rt) dst[i] = acc[i][j];
            }
        }
    }
}

// One block of J2MAX threads. Besides the per-sequence flags it writes *all_conv = 1 when every
// sequence of the launch has converged (read back by the host to stop enqueueing sweeps).
__global__ void jac2_sweep_end_kernel(const __grid_constant__ Jac2Batch batch, float tol_conv, int last, int *dev_status, int *all_conv)
{
    const int b = threadIdx.x;
    int done = 1;
    pdl_trigger();
    pdl_wait();
    if (b < batch.count) {
        const Jac2Seq &sq = batch.s[b];
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
