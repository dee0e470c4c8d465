// atp_attention: Eq. 6 projections of the r-row representation, then attention of every query
// on the r principal keys/values (the procedure of Eq. 1 with K', V' in place of K, V).
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "attention_tc.cuh"
#include <type_traits>
#include <math.h>

constexpr int ATT_MAX_BATCH = 32;
struct AttnSeq { const float *Q, *K, *V; void *O; int L, r; };
struct AttnBatch { AttnSeq s[ATT_MAX_BATCH]; int count; };

// One CTA: 64 queries of one head of one sequence; keys in blocks of 64; online softmax in fp32.
// Shared: Qt[dh][68], Kt[dh][68] (transposed tiles), Vs[64][dh], Ps[64][65].
template <typename TO>
__global__ void __launch_bounds__(256)
attn_simt_kernel(const __grid_constant__ AttnBatch batch, int dh, int ldq, int ldkv, int ldo, float scale)
{
    extern __shared__ __align__(16) float smem[];
    const AttnSeq &sq = batch.s[blockIdx.z];
    const int q0 = blockIdx.x * 64;
    if (q0 >= sq.L) return;
    const int head = blockIdx.y;
    float *Qt = smem;                       // dh x 68
    float *Kt = Qt + (size_t)dh * 68;       // dh x 68
    float *Vs = Kt + (size_t)dh * 68;       // 64 x dh
    float *Ps = Vs + (size_t)64 * dh;       // 64 x 65
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int hoff = head * dh;

    for (int e = tid; e < 64 * dh; e += 256) {
        int row = e / dh, c = e - row * dh;
        float v = 0.f;
        if (q0 + row < sq.L) v = sq.Q[(size_t)(q0 + row) * ldq + hoff + c];
        Qt[c * 68 + row] = v;
    }
    float m_run[4], l_run[4], acc[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m_run[i] = -INFINITY; l_run[i] = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
    }
    const int ncol = dh / 16;               // columns of O per thread (dh is a multiple of 16)

    for (int k0 = 0; k0 < sq.r; k0 += 64) {
        __syncthreads();                    // previous block's Vs / Ps / Kt no longer in use
        for (int e = tid; e < 64 * dh; e += 256) {
            int row = e / dh, c = e - row * dh;
            float kv = 0.f, vv = 0.f;
            if (k0 + row < sq.r) {
                kv = sq.K[(size_t)(k0 + row) * ldkv + hoff + c];
                vv = sq.V[(size_t)(k0 + row) * ldkv + hoff + c];
            }
            Kt[c * 68 + row] = kv;
            Vs[row * dh + c] = vv;
        }
        __syncthreads();
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
        for (int c = 0; c < dh; ++c) {
            float4 a = *(const float4 *)&Qt[c * 68 + ty * 4];
            float4 b = *(const float4 *)&Kt[c * 68 + tx * 4];
            float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[i][j] = fmaf(av[i], bv[j], s[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s[i][j] = (k0 + tx * 4 + j < sq.r) ? s[i][j] * scale : -INFINITY;
                mx = fmaxf(mx, s[i][j]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float m_new = fmaxf(m_run[i], mx);          // finite: every block holds at least one valid key
            float alpha = expf(m_run[i] - m_new);       // exp(-inf) = 0 on the first block
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float p = expf(s[i][j] - m_new);
                Ps[(ty * 4 + i) * 65 + tx * 4 + j] = p;
                sum += p;
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            l_run[i] = l_run[i] * alpha + sum;
            m_run[i] = m_new;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] *= alpha;
        }
        __syncthreads();
        for (int k = 0; k < 64; ++k) {
            float p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = Ps[(ty * 4 + i) * 65 + k];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j < ncol) {
                    float v = Vs[k * dh + tx + 16 * j];
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(p[i], v, acc[i][j]);
                }
            }
        }
    }
    TO *O = (TO *)sq.O;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int row = q0 + ty * 4 + i;
        if (row >= sq.L) continue;
        float inv = 1.f / l_run[i];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (j < ncol) O[(size_t)row * ldo + hoff + tx + 16 * j] = from_f32<TO>(acc[i][j] * inv);
    }
}

// Rotary positions (Sec. 4.2, position-encoding paragraph): every row of M (fp32, rows x dp) is rotated
// by its position: the pair of coordinates (2j, 2j+1) of each head turns by pos * base^(-2j/d_h).
// pos: per-row positions or nullptr (row index inside its sequence, given by seq_row0). The angle is
// formed in fp64: at position 3e4 an fp32 angle would already be off by 2e-3 rad.
struct RopeSeq { float *K, *Q; int L, row0; };
struct RopeBatch { RopeSeq s[32]; int count; };
__global__ void __launch_bounds__(256) rope_kernel(const __grid_constant__ RopeBatch batch, int dp, int dh, double log2_base,
                                                   const int *pos)
{
    const RopeSeq &q = batch.s[blockIdx.y];
    const int half = dp / 2;
    const size_t n = (size_t)q.L * half;
    for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < n; e += (size_t)gridDim.x * 256) {
        const int l = (int)(e / half), pr = (int)(e - (size_t)l * half);
        const int j = pr % (dh / 2);
        const double p = pos ? (double)pos[q.row0 + l] : (double)l;
        double sn, c;
        sincos(p * exp2(-2.0 * j / dh * log2_base), &sn, &c);
        const float cf = (float)c, sf = (float)sn;
        float *k = q.K + (size_t)l * dp + 2 * pr, *x = q.Q + (size_t)l * dp + 2 * pr;
        const float ka = k[0], kb = k[1], xa = x[0], xb = x[1];
        k[0] = ka * cf - kb * sf; k[1] = ka * sf + kb * cf;
        x[0] = xa * cf - xb * sf; x[1] = xa * sf + xb * cf;
    }
}

struct AttnPlan { float *Qp, *Kp, *Vp, *Q, *Kf; __nv_bfloat16 *Qph, *Qpl, *Kh, *Kl, *Vb, *Qh, *Ql; float *nrm; };
static void plan_attn(Arena &ar, int64_t tr, int64_t tl, int64_t dp, int64_t nseq, AttnPlan &p)
{
    p.Qp = ar.take<float>((size_t)tr * dp);
    p.Kp = ar.take<float>((size_t)tr * dp);
    p.Vp = ar.take<float>((size_t)tr * dp);
    p.Q = ar.take<float>((size_t)tl * dp);
    p.Kf = ar.take<float>((size_t)tl * dp);                                     // full keys U_r K' (rotary positions only)
    p.Qph = ar.take<__nv_bfloat16>((size_t)tr * align_up((size_t)dp, 8));     // Q' as a bf16 hi/lo pair (tensor-core path)
    p.Qpl = ar.take<__nv_bfloat16>((size_t)tr * align_up((size_t)dp, 8));
    p.Kh = ar.take<__nv_bfloat16>((size_t)tr * align_up((size_t)dp, 8));      // fused tensor-core attention operands
    p.Kl = ar.take<__nv_bfloat16>((size_t)tr * align_up((size_t)dp, 8));
    p.Vb = ar.take<__nv_bfloat16>((size_t)tr * align_up((size_t)dp, 8));
    p.Qh = ar.take<__nv_bfloat16>((size_t)tl * align_up((size_t)dp, 8));
    p.Ql = ar.take<__nv_bfloat16>((size_t)tl * align_up((size_t)dp, 8));
    p.nrm = ar.take<float>((size_t)(tl / 128 + nseq) * dp + (size_t)(tr / 128 + nseq) * dp);    // per head norms: query tiles, key blocks
}
size_t attention_workspace_bytes(const std::vector<SeqDims> &seqs, int64_t dp)
{
    int64_t tr = 0, tl = 0;
    for (auto &s : seqs) { tr += s.r; tl += s.L; }
    Arena ar(nullptr, (size_t)-1);
    AttnPlan p;
    plan_attn(ar, tr, tl, dp, (int64_t)seqs.size(), p);
    return ar.off;
}

template <typename T>
static atp_status attention_impl(atp_ctx *ctx, const atp_mat *X, const atp_mat *U_r, const atp_mat *X_r,
                                 const atp_mat *WQ, const atp_mat *WK, const atp_mat *WV, int heads,
                                 const std::vector<SeqDims> &seqs, int q_mode, float scale, float rope_base, const int *positions,
                                 atp_mat *O)
{
    const int d = (int)X_r->cols, dp = (int)WQ->cols, dh = dp / heads;
    const bool rope = rope_base > 0.f;
    int64_t tr = 0, tl = 0;
    for (auto &s : seqs) { tr += s.r; tl += s.L; }
    Arena ar(ctx->workspace, ctx->workspace_bytes);
    AttnPlan pl;
    plan_attn(ar, tr, tl, dp, (int64_t)seqs.size(), pl);
    if (ar.overflow || !ctx->workspace) return ATP_ERR_WORKSPACE_TOO_SMALL;
    atp_status st;
    GemmEpi store{EPI_STORE, nullptr};
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if ((dh == 64 || dh == 128) && !rope) {
            // bf16, head width 64 or 128: everything on the tensor cores. K' and Q are produced as
            // bf16 hi/lo pairs by the GEMM epilogues, V' as bf16; the fused kernel does the rest.
            const int ldq = (int)align_up((size_t)dp, 8);
            std::vector<tc::HostProblem> g1, g2;
            g1.push_back(tc::HostProblem{X_r->data, WK->data, nullptr, pl.Kh, pl.Kl, nullptr, (int)tr, dp, d, (int)X_r->ld, (int)WK->ld, ldq, 0});
            if (q_mode == ATP_Q_LOWRANK)
                g1.push_back(tc::HostProblem{X_r->data, WQ->data, nullptr, pl.Qph, pl.Qpl, nullptr, (int)tr, dp, d, (int)X_r->ld, (int)WQ->ld, ldq, 0});
            else
                g1.push_back(tc::HostProblem{X->data, WQ->data, nullptr, pl.Qh, pl.Ql, nullptr, (int)tl, dp, d, (int)X->ld, (int)WQ->ld, ldq, 0});
            if ((st = tc::launch<false, false, tc::OUT_BF16_SPLIT>(ctx, g1, store)) != ATP_OK) return st;
            g2.push_back(tc::HostProblem{X_r->data, WV->data, nullptr, pl.Vb, nullptr, nullptr, (int)tr, dp, d, (int)X_r->ld, (int)WV->ld, ldq, 0});
            if ((st = tc::launch<false, false, tc::OUT_BF16>(ctx, g2, store)) != ATP_OK) return st;
            if (q_mode == ATP_Q_LOWRANK) {
                std::vector<tc::HostProblem> qe;
                for (auto &s : seqs)
                    if (s.L > 0)
                        qe.push_back(tc::HostProblem{(const T *)U_r->data + (size_t)s.row0 * U_r->ld, pl.Qph + (size_t)s.rank0 * ldq,
                                                     pl.Qpl + (size_t)s.rank0 * ldq, pl.Qh + (size_t)s.row0 * ldq, pl.Ql + (size_t)s.row0 * ldq,
                                                     nullptr, s.L, dp, s.r, (int)U_r->ld, ldq, ldq, 0});
                if ((st = tc::launch<false, true, tc::OUT_BF16_SPLIT>(ctx, qe, store)) != ATP_OK) return st;
            }
            std::vector<atc::HostSeq> hs;
            float *nrm = pl.nrm;
            for (auto &s : seqs)
                if (s.L > 0) {
                    float *qmax = nrm, *kmax = nrm + (size_t)heads * ceil_div(s.L, 128);
                    nrm += (size_t)heads * (ceil_div(s.L, 128) + ceil_div(s.r, 128));
                    hs.push_back(atc::HostSeq{pl.Qh + (size_t)s.row0 * ldq, pl.Ql + (size_t)s.row0 * ldq, pl.Kh + (size_t)s.rank0 * ldq,
                                              pl.Kl + (size_t)s.rank0 * ldq, pl.Vb + (size_t)s.rank0 * ldq,
                                              (T *)O->data + (size_t)s.row0 * O->ld, s.L, s.r, ldq, ldq, (int)O->ld, dp, qmax, kmax});
                }
            return dh == 64 ? atc::launch<64>(ctx, hs, heads, scale) : atc::launch<128>(ctx, hs, heads, scale);
        }
        // bf16, other head widths: projections on the tensor cores with fp32 results. Q' is kept as a bf16 hi/lo pair so
        // that the expansion Q = U_r Q' loses nothing against fp32 (the logits reach magnitudes of
        // 10^2, where a bf16-rounded query would move the softmax).
        const int ldq = (int)align_up((size_t)dp, 8);
        std::vector<tc::HostProblem> kv;
        kv.push_back(tc::HostProblem{X_r->data, WK->data, nullptr, pl.Kp, nullptr, nullptr, (int)tr, dp, d, (int)X_r->ld, (int)WK->ld, dp, 0});
        kv.push_back(tc::HostProblem{X_r->data, WV->data, nullptr, pl.Vp, nullptr, nullptr, (int)tr, dp, d, (int)X_r->ld, (int)WV->ld, dp, 0});
        if (q_mode == ATP_Q_FULL)
            kv.push_back(tc::HostProblem{X->data, WQ->data, nullptr, pl.Q, nullptr, nullptr, (int)tl, dp, d, (int)X->ld, (int)WQ->ld, dp, 0});
        if ((st = tc::launch<false, false, tc::OUT_F32>(ctx, kv, store)) != ATP_OK) return st;
        if (q_mode == ATP_Q_LOWRANK) {
            std::vector<tc::HostProblem> qp;
            qp.push_back(tc::HostProblem{X_r->data, WQ->data, nullptr, pl.Qph, pl.Qpl, nullptr, (int)tr, dp, d, (int)X_r->ld, (int)WQ->ld, ldq, 0});
            if ((st = tc::launch<false, false, tc::OUT_BF16_SPLIT>(ctx, qp, store)) != ATP_OK) return st;
            std::vector<tc::HostProblem> qe;
            for (auto &s : seqs)
                if (s.L > 0)
                    qe.push_back(tc::HostProblem{(const T *)U_r->data + (size_t)s.row0 * U_r->ld, pl.Qph + (size_t)s.rank0 * ldq,
                                                 pl.Qpl + (size_t)s.rank0 * ldq, pl.Q + (size_t)s.row0 * dp, nullptr, nullptr,
                                                 s.L, dp, s.r, (int)U_r->ld, ldq, dp, 0});
            if ((st = tc::launch<false, true, tc::OUT_F32>(ctx, qe, store)) != ATP_OK) return st;
        }
    } else {
    {   // Q', K', V' = X_r W (Eq. 6), all sequences at once
        GemmBatch b; b.count = (q_mode == ATP_Q_LOWRANK) ? 3 : 2;
        const atp_mat *Ws[3] = {WK, WV, WQ};
        float *outs[3] = {pl.Kp, pl.Vp, pl.Qp};
        for (int i = 0; i < b.count; ++i)
            b.p[i] = GemmProblem{X_r->data, Ws[i]->data, outs[i], nullptr, (int)tr, dp, d, (int)X_r->ld, (int)Ws[i]->ld, dp, 0};
        if ((st = launch_gemm_simt<T, T, float, false>(ctx, b, store)) != ATP_OK) return st;
    }
    if (q_mode == ATP_Q_LOWRANK) {      // Q = U_r Q'
        std::vector<GemmProblem> ps;
        for (auto &s : seqs)
            if (s.L > 0)
                ps.push_back(GemmProblem{(const T *)U_r->data + (size_t)s.row0 * U_r->ld, pl.Qp + (size_t)s.rank0 * dp,
                                         pl.Q + (size_t)s.row0 * dp, nullptr, s.L, dp, s.r, (int)U_r->ld, dp, dp, 0});
        st = for_each_chunk(ps, [&](const GemmBatch &b) { return launch_gemm_simt<T, float, float, false>(ctx, b, store); });
        if (st != ATP_OK) return st;
    } else {                            // Q = X W_Q
        GemmBatch b; b.count = 1;
        b.p[0] = GemmProblem{X->data, WQ->data, pl.Q, nullptr, (int)tl, dp, d, (int)X->ld, (int)WQ->ld, dp, 0};
        if ((st = launch_gemm_simt<T, T, float, false>(ctx, b, store)) != ATP_OK) return st;
    }
    }
    if (rope) {
        // K = U_r K' (Eq. 6), rows of K and Q rotated by their positions, principal keys K'_rot = U_r^T K_rot
        std::vector<GemmProblem> up, down;
        RopeBatch rb; rb.count = 0;
        auto flush_rope = [&]() -> atp_status {
            if (rb.count == 0) return ATP_OK;
            int maxL = 0;
            for (int i = 0; i < rb.count; ++i) maxL = std::max(maxL, rb.s[i].L);
            ATP_KERNEL(ctx, "rope", 0, 0);
            rope_kernel<<<dim3(std::min(512, ceil_div(maxL * (dp / 2), 256)), rb.count), 256, 0, ctx->stream>>>(
                rb, dp, dh, log2((double)rope_base), positions);
            ATP_LAUNCHED(ctx);
            rb.count = 0;
            return ATP_OK;
        };
        for (auto &sq : seqs)
            if (sq.L > 0)
                up.push_back(GemmProblem{(const T *)U_r->data + (size_t)sq.row0 * U_r->ld, pl.Kp + (size_t)sq.rank0 * dp,
                                         pl.Kf + (size_t)sq.row0 * dp, nullptr, sq.L, dp, sq.r, (int)U_r->ld, dp, dp, 0});
        st = for_each_chunk(up, [&](const GemmBatch &b) { return launch_gemm_simt<T, float, float, false>(ctx, b, store, 1, nullptr, 0, "gemm_simt_rope"); });
        if (st != ATP_OK) return st;
        for (auto &sq : seqs)
            if (sq.L > 0) {
                rb.s[rb.count++] = RopeSeq{pl.Kf + (size_t)sq.row0 * dp, pl.Q + (size_t)sq.row0 * dp, sq.L, sq.row0};
                if (rb.count == 32 && (st = flush_rope()) != ATP_OK) return st;
            }
        if ((st = flush_rope()) != ATP_OK) return st;
        for (auto &sq : seqs)
            if (sq.L > 0)
                down.push_back(GemmProblem{(const T *)U_r->data + (size_t)sq.row0 * U_r->ld, pl.Kf + (size_t)sq.row0 * dp,
                                           pl.Kp + (size_t)sq.rank0 * dp, nullptr, sq.r, dp, sq.L, (int)U_r->ld, dp, dp, 0});
        st = for_each_chunk(down, [&](const GemmBatch &b) { return launch_gemm_simt<T, float, float, true>(ctx, b, store, 1, nullptr, 0, "gemm_simt_rope"); });
        if (st != ATP_OK) return st;
    }
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (dh == 64 || dh == 128) {
            // rotary positions with a tensor-core head width: the fp32 K'_rot, Q_rot and V' are cut into the
            // bf16 (hi/lo) operands of the fused kernel
            const int ldq = (int)align_up((size_t)dp, 8);
            ATP_KERNEL(ctx, "f32_to_bf16", 0, (double)(2 * tr + tl) * dp * 8);
            tc::f32_to_bf16_split_kernel<<<1024, 256, 0, ctx->stream>>>(pl.Kp, dp, pl.Kh, pl.Kl, ldq, (int)tr, dp);
            ATP_LAUNCHED(ctx);
            tc::f32_to_bf16_split_kernel<<<1024, 256, 0, ctx->stream>>>(pl.Q, dp, pl.Qh, pl.Ql, ldq, (int)tl, dp);
            ATP_LAUNCHED(ctx);
            tc::f32_to_bf16_split_kernel<<<1024, 256, 0, ctx->stream>>>(pl.Vp, dp, pl.Vb, pl.Qpl, ldq, (int)tr, dp);   // lo part unused
            ATP_LAUNCHED(ctx);
            std::vector<atc::HostSeq> hs;
            float *nrm = pl.nrm;
            for (auto &sq : seqs)
                if (sq.L > 0) {
                    float *qmax = nrm, *kmax = nrm + (size_t)heads * ceil_div(sq.L, 128);
                    nrm += (size_t)heads * (ceil_div(sq.L, 128) + ceil_div(sq.r, 128));
                    hs.push_back(atc::HostSeq{pl.Qh + (size_t)sq.row0 * ldq, pl.Ql + (size_t)sq.row0 * ldq, pl.Kh + (size_t)sq.rank0 * ldq,
                                              pl.Kl + (size_t)sq.rank0 * ldq, pl.Vb + (size_t)sq.rank0 * ldq,
                                              (T *)O->data + (size_t)sq.row0 * O->ld, sq.L, sq.r, ldq, ldq, (int)O->ld, dp, qmax, kmax});
                }
            return dh == 64 ? atc::launch<64>(ctx, hs, heads, scale) : atc::launch<128>(ctx, hs, heads, scale);
        }
    }
    size_t smem = ((size_t)dh * 68 * 2 + (size_t)64 * dh + 64 * 65) * sizeof(float);
    ATP_CUDA_OK(ctx, cudaFuncSetAttribute(attn_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    for (size_t i = 0; i < seqs.size(); i += ATT_MAX_BATCH) {
        AttnBatch ab; ab.count = 0; int maxL = 0; double fl = 0, by = 0;
        for (size_t j = i; j < seqs.size() && ab.count < ATT_MAX_BATCH; ++j) {
            const SeqDims &s = seqs[j];
            if (s.L == 0) continue;
            ab.s[ab.count++] = AttnSeq{pl.Q + (size_t)s.row0 * dp, pl.Kp + (size_t)s.rank0 * dp, pl.Vp + (size_t)s.rank0 * dp,
                                       (T *)O->data + (size_t)s.row0 * O->ld, s.L, s.r};
            if (s.L > maxL) maxL = s.L;
            fl += 4.0 * s.L * s.r * dp;
            by += (2.0 * s.r * dp + s.L * dp) * sizeof(float) + (double)s.L * dp * sizeof(T);
        }
        if (ab.count == 0) continue;
        dim3 grid(ceil_div(maxL, 64), heads, ab.count);
        ATP_KERNEL(ctx, "attn_simt", fl, by);
        attn_simt_kernel<T><<<grid, 256, smem, ctx->stream>>>(ab, dh, dp, dp, (int)O->ld, scale);
        ATP_LAUNCHED(ctx);
    }
    return ATP_OK;
}

extern "C" atp_status atp_attention(atp_ctx *ctx, const atp_mat *X, const atp_mat *U_r, const atp_mat *X_r,
                                    const atp_mat *W_Q, const atp_mat *W_K, const atp_mat *W_V, int heads,
                                    const atp_seqs *seqs, const atp_attn_opts *opts, atp_mat *O)
{
    if (!ctx) return ATP_ERR_INVALID_ARG;
    atp_status st;
    if ((st = check_mat(U_r)) != ATP_OK || (st = check_mat(X_r)) != ATP_OK || (st = check_mat(W_Q)) != ATP_OK ||
        (st = check_mat(W_K)) != ATP_OK || (st = check_mat(W_V)) != ATP_OK || (st = check_mat(O)) != ATP_OK)
        return st;
    int q_mode = ATP_Q_LOWRANK; float scale = 0.f, rope_base = 0.f; const int32_t *positions = nullptr;
    if (opts) {
        // the struct grew by the rotary fields: a caller built against the shorter layout gets no rotation
        if (opts->struct_size < offsetof(atp_attn_opts, rope_base)) return ATP_ERR_INVALID_ARG;
        q_mode = opts->q_mode; scale = opts->scale;
        if (opts->struct_size >= sizeof(atp_attn_opts)) { rope_base = opts->rope_base; positions = opts->positions; }
    }
    if (rope_base < 0.f || (rope_base > 0.f && rope_base <= 1.f)) return ATP_ERR_INVALID_ARG;
    if (q_mode != ATP_Q_LOWRANK && q_mode != ATP_Q_FULL) return ATP_ERR_INVALID_ARG;
    if (q_mode == ATP_Q_FULL) {
        if (!X || (st = check_mat(X)) != ATP_OK) return st != ATP_OK ? st : ATP_ERR_INVALID_ARG;
        if (X->rows != U_r->rows || X->cols != X_r->cols || X->dtype != X_r->dtype) return ATP_ERR_INVALID_ARG;
    }
    const atp_dtype dt = X_r->dtype;
    if (U_r->dtype != dt || W_Q->dtype != dt || W_K->dtype != dt || W_V->dtype != dt || O->dtype != dt)
        return ATP_ERR_UNSUPPORTED_DTYPE;
    const int64_t d = X_r->cols, dp = W_Q->cols;
    if (W_Q->rows != d || W_K->rows != d || W_V->rows != d || W_K->cols != dp || W_V->cols != dp) return ATP_ERR_INVALID_ARG;
    if (heads < 1 || dp % heads != 0) return ATP_ERR_INVALID_ARG;
    const int64_t dh = dp / heads;
    if (dh % 16 != 0 || dh > 128) return ATP_ERR_INVALID_ARG;     // head widths 16..128 in steps of 16
    std::vector<SeqDims> sd;
    if ((st = check_seqs(seqs, sd, U_r->rows)) != ATP_OK) return st;
    int64_t tr = 0; int maxr = 0;
    for (auto &s : sd) { tr += s.r; if (s.r > maxr) maxr = s.r; }
    if (X_r->rows != tr || U_r->cols < maxr || O->rows != U_r->rows || O->cols != dp) return ATP_ERR_INVALID_ARG;
    if (U_r->rows == 0) return ATP_OK;
    if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)dh);
    ATP_CUDA_OK(ctx, cudaSetDevice(ctx->device));
    if (dt == ATP_F32) return attention_impl<float>(ctx, X, U_r, X_r, W_Q, W_K, W_V, heads, sd, q_mode, scale, rope_base, positions, O);
    return attention_impl<__nv_bfloat16>(ctx, X, U_r, X_r, W_Q, W_K, W_V, heads, sd, q_mode, scale, rope_base, positions, O);
}
