// Batched bf16 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulator in TMEM, operands
// staged in shared memory by TMA with the 128-byte swizzle): C = epilogue(op(A) * B).
//   A: M x K row-major (K-major operand) or K x M row-major (M-major operand), bf16
//   B: K x N row-major (N-major operand) or N x K row-major (K-major operand), bf16; optionally a
//      second matrix B_lo of the same shape whose product is accumulated on top (split precision:
//      B = B_hi + B_lo), and a second matrix A_lo as well: A_hi B_hi + A_hi B_lo + A_lo B_hi carries
//      about 16 mantissa bits of both operands, for fp32 data cut into bf16 hi/lo pairs
//   C: M x N row-major, fp32 or bf16, or a bf16 hi/lo pair; D (optional): M x N fp32
// One CTA computes one 128 x 128 tile: warp 4 issues the TMA loads, warp 5 allocates TMEM and issues
// the MMAs, warps 0-3 read the accumulator back (tcgen05.ld) and run the epilogue. Extents come
// from per-problem tensor maps, so ragged M, N, K are zero-filled by TMA and masked at the store.
// Every mbarrier wait is bounded; on expiry the kernel records ATP_ERR_TIMEOUT and winds down.
#pragma once
#include "common.cuh"
#include "gemm_simt.cuh"
#include <cuda.h>

namespace tc {

constexpr int BM = 128, BN = 128, BK = 64;
constexpr int MAX_PROB = 16;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

struct Problem {
    CUtensorMap ta, ta2, tb, tb2; // ta2 / tb2 only with a split A / B
    void *C; void *C2; const float *D;
    int M, N, K, ldc, ldd;
    int tile0, tiles_n, tiles_m; // first linear tile index of this problem, tiles along N and along M
};
struct Batch {
    Problem p[MAX_PROB];
    int count, total_tiles;
};

enum OutKind { OUT_F32 = 0, OUT_BF16 = 1, OUT_BF16_SPLIT = 2 };

// ---- PTX wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The same MMA with the A operand in tensor memory (M = 128 lanes = rows, two 16-bit K elements per
// 32-bit column): only B is read from shared memory.
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// The same load without the wait: several loads can be in flight, then one tmem_ld_wait().
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, Blackwell version field set.
//   K-major tile  (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart):        lbo unused, sbo = 1024
//   MN-major tile (k-rows of 64 bf16 along M/N, 8-row groups 1024 B apart,
//                  64-element chunks `lbo` bytes apart):                        lbo = chunk stride, sbo = 1024
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;      // descriptor version
    d |= (uint64_t)2 << 61;      // SWIZZLE_128B
    return d;
}
// Instruction descriptor for kind::f16 with bf16 operands and fp32 accumulation.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool a_mn_major, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <bool SPLIT_B, bool SPLIT_A = false> struct Cfg {
    static constexpr int STAGES = SPLIT_A ? 3 : (SPLIT_B ? 4 : 3);
    static constexpr int A_BYTES = BM * BK * 2;                 // 16 KB
    static constexpr int B_BYTES = BK * BN * 2;                 // 16 KB
    static constexpr int B_OFF = A_BYTES * (SPLIT_A ? 2 : 1);
    static constexpr int STAGE_BYTES = B_OFF + B_BYTES * (SPLIT_B ? 2 : 1);
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <bool A_MN, bool SPLIT_B, int OUT, bool B_KMAJ = false, bool SPLIT_A = false>
__global__ void __launch_bounds__(192)
gemm_tc_kernel(const __grid_constant__ Batch batch, GemmEpi epi, int *dev_status)
{
    using C_ = Cfg<SPLIT_B, SPLIT_A>;
    static_assert(!SPLIT_A || SPLIT_B, "a split A comes with a split B");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                // swizzled tiles need 1024-byte alignment
    uint8_t *gbase = smem_raw + (base - raw);
    const uint32_t bars = base + C_::STAGES * C_::STAGE_BYTES;   // full[S], empty[S], tmem_full, then tmem slot
    uint32_t *tmem_slot = (uint32_t *)(gbase + C_::STAGES * C_::STAGE_BYTES + 8 * (2 * C_::STAGES + 1));
    __shared__ int abort_flag;

    // which tile
    const int tile = blockIdx.x;
    int pi = 0;
#pragma unroll 1
    for (int i = 1; i < batch.count; ++i) if (tile >= batch.p[i].tile0) pi = i;
    const Problem &pr = batch.p[pi];
    const int lt = tile - pr.tile0;
    // Where N is much larger than M, consecutive CTAs walk along M: they share a tile of the large operand B, and
    // the operand that is re-read from L2 is the small one, A (a 4096 x 2048 x 11008 product read 1 GB
    // from DRAM in row-major tile order: its 45 MB B operand was evicted by the streamed epilogue operand).
    const bool along_m = pr.tiles_n > 2 * pr.tiles_m;
    const int m0 = (along_m ? lt % pr.tiles_m : lt / pr.tiles_n) * BM, n0 = (along_m ? lt / pr.tiles_m : lt % pr.tiles_n) * BN;
    const int num_kt = (pr.K + BK - 1) / BK;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < C_::STAGES; ++s) { mbar_init(bars + 8 * s, 1); mbar_init(bars + 8 * (C_::STAGES + s), 1); }
        mbar_init(bars + 8 * (2 * C_::STAGES), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) tmem_alloc(smem_u32(tmem_slot), BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 4) {
        if (lane == 0) {
            for (int kt = 0; kt < num_kt; ++kt) {
                const int s = kt % C_::STAGES;
                if (kt >= C_::STAGES && !mbar_wait(bars + 8 * (C_::STAGES + s), ((kt / C_::STAGES) - 1) & 1, &abort_flag)) break;
                const uint32_t full = bars + 8 * s;
                const uint32_t sa = base + s * C_::STAGE_BYTES, sb = sa + C_::B_OFF;
                mbar_expect_tx(full, C_::STAGE_BYTES);
                const int k0 = kt * BK;
                if (!A_MN) {
                    tma_load_2d(sa, &pr.ta, k0, m0, full);                       // box {64 k, 128 m}
                    if (SPLIT_A) tma_load_2d(sa + C_::A_BYTES, &pr.ta2, k0, m0, full);
                } else {
                    tma_load_2d(sa, &pr.ta, m0, k0, full);                       // box {64 m, 64 k} x 2
                    tma_load_2d(sa + 8192, &pr.ta, m0 + 64, k0, full);
                    if (SPLIT_A) {
                        tma_load_2d(sa + C_::A_BYTES, &pr.ta2, m0, k0, full);
                        tma_load_2d(sa + C_::A_BYTES + 8192, &pr.ta2, m0 + 64, k0, full);
                    }
                }
                if (B_KMAJ) {
                    tma_load_2d(sb, &pr.tb, k0, n0, full);                       // box {64 k, 128 n}
                    if (SPLIT_B) tma_load_2d(sb + C_::B_BYTES, &pr.tb2, k0, n0, full);
                } else {
                    tma_load_2d(sb, &pr.tb, n0, k0, full);                       // box {64 n, 64 k} x 2
                    tma_load_2d(sb + 8192, &pr.tb, n0 + 64, k0, full);
                    if (SPLIT_B) {
                        tma_load_2d(sb + C_::B_BYTES, &pr.tb2, n0, k0, full);
                        tma_load_2d(sb + C_::B_BYTES + 8192, &pr.tb2, n0 + 64, k0, full);
                    }
                }
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BM, BN, A_MN, !B_KMAJ);
            bool ok = true;
            for (int kt = 0; kt < num_kt && ok; ++kt) {
                const int s = kt % C_::STAGES;
                ok = mbar_wait(bars + 8 * s, (kt / C_::STAGES) & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sa = base + s * C_::STAGE_BYTES, sb = sa + C_::B_OFF;
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {
                    auto adesc = [&](uint32_t a0) { return A_MN ? smem_desc(a0 + kk * 2048, 8192, 1024) : smem_desc(a0 + kk * 32, 16, 1024); };
                    auto bdesc = [&](uint32_t b0) { return B_KMAJ ? smem_desc(b0 + kk * 32, 16, 1024) : smem_desc(b0 + kk * 2048, 8192, 1024); };
                    const uint64_t ad = adesc(sa), bd = bdesc(sb);
                    // small terms first, the hi * hi product last
                    if (SPLIT_A) umma_bf16(tmem_base, adesc(sa + C_::A_BYTES), bd, idesc, (kt > 0 || kk > 0) ? 1u : 0u);
                    if (SPLIT_B) umma_bf16(tmem_base, ad, bdesc(sb + C_::B_BYTES), idesc, (SPLIT_A || kt > 0 || kk > 0) ? 1u : 0u);
                    umma_bf16(tmem_base, ad, bd, idesc, (SPLIT_B || kt > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bars + 8 * (C_::STAGES + s));        // frees the stage once these MMAs have read it
            }
            umma_commit(bars + 8 * (2 * C_::STAGES));            // accumulator complete
        }
    } else {
        // epilogue warps 0..3: TMEM lane = row of the tile
        int ok_i = 0;
        if (lane == 0) ok_i = mbar_wait(bars + 8 * (2 * C_::STAGES), 0, &abort_flag) ? 1 : 0;
        const bool ok = __shfl_sync(0xffffffffu, ok_i, 0) != 0;      // warp-uniform: tcgen05.ld is warp-collective
        tc_fence_after();
        const int row = m0 + warp * 32 + lane;
        if (ok) {
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + c, r);
                const int col0 = n0 + c;
                if (row < pr.M && col0 < pr.N) {
                    float v[32];
                    const bool full_chunk = (col0 + 32 <= pr.N);
                    // the D operand of this thread's 32 columns: eight 16-byte loads in flight instead of 32 scalar ones
                    const bool d_vec = (epi.kind == EPI_D_MINUS || epi.kind == EPI_SILU_D_MUL) && full_chunk &&
                                       ((pr.ldd & 3) == 0) && (((size_t)pr.D & 15) == 0);
                    float dv[32];
                    if (d_vec) {
                        const float4 *dp = (const float4 *)(pr.D + (size_t)row * pr.ldd + col0);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float4 q = __ldg(dp + j);
                            dv[4 * j] = q.x; dv[4 * j + 1] = q.y; dv[4 * j + 2] = q.z; dv[4 * j + 3] = q.w;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float x = __uint_as_float(r[j]);
                        const int col = col0 + j;
                        if (col < pr.N) {
                            switch (epi.kind) {
                                case EPI_D_MINUS: x = (d_vec ? dv[j] : pr.D[(size_t)row * pr.ldd + col]) - x; break;
                                case EPI_BIAS: if (epi.bias) x += epi.bias[col]; break;
                                case EPI_BIAS_GELU: if (epi.bias) x += epi.bias[col]; x = gelu_erf_f(x); break;
                                case EPI_SILU_D_MUL: x = silu_f(d_vec ? dv[j] : pr.D[(size_t)row * pr.ldd + col]) * x; break;
                                default: break;
                            }
                        }
                        v[j] = x;
                    }
                    if (OUT == OUT_F32) {
                        float *dst = (float *)pr.C + (size_t)row * pr.ldc + col0;
                        if (full_chunk && ((pr.ldc & 3) == 0)) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *(float4 *)(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
                            for (int j = 0; j < 32 && col0 + j < pr.N; ++j) dst[j] = v[j];
                        }
                    } else {
                        __nv_bfloat16 *dst = (__nv_bfloat16 *)pr.C + (size_t)row * pr.ldc + col0;
                        __nv_bfloat16 *dst2 = (OUT == OUT_BF16_SPLIT) ? (__nv_bfloat16 *)pr.C2 + (size_t)row * pr.ldc + col0 : nullptr;
                        if (full_chunk && ((pr.ldc & 7) == 0)) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                __nv_bfloat162 h[4], l[4];
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    h[t] = __floats2bfloat162_rn(v[j + 2 * t], v[j + 2 * t + 1]);
                                    if (OUT == OUT_BF16_SPLIT)
                                        l[t] = __floats2bfloat162_rn(v[j + 2 * t] - __low2float(h[t]), v[j + 2 * t + 1] - __high2float(h[t]));
                                }
                                *(uint4 *)(dst + j) = *(uint4 *)h;
                                if (OUT == OUT_BF16_SPLIT) *(uint4 *)(dst2 + j) = *(uint4 *)l;
                            }
                        } else {
                            for (int j = 0; j < 32 && col0 + j < pr.N; ++j) {
                                __nv_bfloat16 h = __float2bfloat16_rn(v[j]);
                                dst[j] = h;
                                if (OUT == OUT_BF16_SPLIT) dst2[j] = __float2bfloat16_rn(v[j] - __bfloat162float(h));
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag && dev_status) raise_status(dev_status, ATP_ERR_TIMEOUT);
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, BN);
    }
}

// ---- host side ---------------------------------------------------------------------------------
// Tensor map over a row-major bf16 matrix (rows x cols, ld elements): box {64 cols, box_rows rows}, 128-byte swizzle.
// The driver entry point is looked up at run time (the library does not link against libcuda, so it
// still loads on machines without a driver, where only the symbol table is inspected).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static inline EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}
static inline bool make_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct HostProblem {
    const void *A; const void *B; const void *B2; void *C; void *C2; const float *D;
    int M, N, K, lda, ldb, ldc, ldd;
    const void *A2 = nullptr;     // low part of a split A
};

static inline bool operands_ok(const HostProblem &h)
{
    auto al = [](const void *p) { return ((uintptr_t)p & 15) == 0; };
    return al(h.A) && al(h.B) && (!h.B2 || al(h.B2)) && (h.lda % 8 == 0) && (h.ldb % 8 == 0) && h.M > 0 && h.N > 0 && h.K > 0;
}

template <bool A_MN, bool SPLIT_B, int OUT, bool B_KMAJ = false, bool SPLIT_A = false>
static atp_status launch(atp_ctx *ctx, const std::vector<HostProblem> &probs, GemmEpi epi, const char *tag = nullptr)
{
    using C_ = Cfg<SPLIT_B, SPLIT_A>;
    static PerDeviceOnce attr_once;        // the shared-memory opt-in is a per-device attribute
    ATP_CUDA_OK(ctx, attr_once.run(ctx->device, [] {
        return cudaFuncSetAttribute(gemm_tc_kernel<A_MN, SPLIT_B, OUT, B_KMAJ, SPLIT_A>, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM);
    }));
    size_t i = 0;
    while (i < probs.size()) {
        Batch b; b.count = 0; b.total_tiles = 0;
        double flops = 0, bytes = 0;
        for (; i < probs.size() && b.count < MAX_PROB; ++i) {
            const HostProblem &h = probs[i];
            if (h.M <= 0 || h.N <= 0 || h.K <= 0) continue;
            Problem &p = b.p[b.count];
            bool ok = A_MN ? make_map(&p.ta, h.A, h.K, h.M, h.lda, 64) : make_map(&p.ta, h.A, h.M, h.K, h.lda, BM);
            if (SPLIT_A) ok = ok && h.A2 && (A_MN ? make_map(&p.ta2, h.A2, h.K, h.M, h.lda, 64) : make_map(&p.ta2, h.A2, h.M, h.K, h.lda, BM));
            auto bmap = [&](CUtensorMap *m, const void *ptr) { return B_KMAJ ? make_map(m, ptr, h.N, h.K, h.ldb, BN) : make_map(m, ptr, h.K, h.N, h.ldb, 64); };
            ok = ok && bmap(&p.tb, h.B);
            if (SPLIT_B) ok = ok && h.B2 && bmap(&p.tb2, h.B2);
            if (!ok) return ATP_ERR_INVALID_ARG;
            p.C = h.C; p.C2 = h.C2; p.D = h.D; p.M = h.M; p.N = h.N; p.K = h.K; p.ldc = h.ldc; p.ldd = h.ldd;
            p.tiles_n = ceil_div(h.N, BN);
            p.tiles_m = ceil_div(h.M, BM);
            p.tile0 = b.total_tiles;
            b.total_tiles += ceil_div(h.M, BM) * p.tiles_n;
            b.count++;
            flops += 2.0 * h.M * h.N * h.K * (SPLIT_A ? 3 : (SPLIT_B ? 2 : 1));
            bytes += 2.0 * ((double)h.M * h.K + (double)h.K * h.N * (SPLIT_B ? 2 : 1)) + (double)h.M * h.N * (OUT == OUT_F32 ? 4 : (OUT == OUT_BF16 ? 2 : 4));
        }
        if (b.count == 0) continue;
        ATP_KERNEL(ctx, tag ? tag : (SPLIT_A ? "gemm_tc_split3" : (SPLIT_B ? "gemm_tc_split" : "gemm_tc")), flops, bytes);
        gemm_tc_kernel<A_MN, SPLIT_B, OUT, B_KMAJ, SPLIT_A><<<b.total_tiles, 192, C_::SMEM, ctx->stream>>>(b, epi, ctx->dev_status);
        ATP_LAUNCHED(ctx);
    }
    return ATP_OK;
}

// fp32 -> bf16 copy (rows x cols), destination leading dimension ldd (multiple of 8 for TMA).
static __global__ void f32_to_bf16_kernel(const float *src, int lds, __nv_bfloat16 *dst, int ldd, int rows, int cols)
{
    size_t n = (size_t)rows * cols;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        int r = (int)(e / cols), c = (int)(e - (size_t)r * cols);
        dst[(size_t)r * ldd + c] = __float2bfloat16_rn(src[(size_t)r * lds + c]);
    }
}

// fp32 -> bf16 hi/lo pair: hi = bf16(x), lo = bf16(x - hi).
static __global__ void f32_to_bf16_split_kernel(const float *src, int lds, __nv_bfloat16 *hi, __nv_bfloat16 *lo, int ldd, int rows, int cols)
{
    size_t n = (size_t)rows * cols;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        int r = (int)(e / cols), c = (int)(e - (size_t)r * cols);
        float x = src[(size_t)r * lds + c];
        __nv_bfloat16 h = __float2bfloat16_rn(x);
        hi[(size_t)r * ldd + c] = h;
        lo[(size_t)r * ldd + c] = __float2bfloat16_rn(x - __bfloat162float(h));
    }
}

}  // namespace tc
