/*
 * libatp -- the per-layer prefill hot path of ATP (attention on top principal keys)
 * for NVIDIA B200 (sm_100a).
 *
 * The three main calls follow the paper's statement of the problem:
 *
 *   atp_principal_basis(X, r)                     -> (U_r, X_r)   Eq. 3, Eq. 5, Sec. 4.2, Eq. 9
 *   atp_attention(X, U_r, X_r, W_Q, W_K, W_V, h)  -> O            Eq. 6, Eq. 1 on r principal keys
 *   atp_lowrank_linear(U_r, X_r, W)               -> Y            Sec. 4.3 (linear layers on the
 *                                                                 r-row representation)
 *   atp_input_norm(X [, residual])                -> X_n          the "Norm" box of Fig. 3
 *   atp_alternating_basis(X, V0, inner)           -> (U, X')      Algorithm 1 (appendix B)
 *   atp_svd_entropy(sigma)                        -> (mu, rank)   Eq. 4
 *
 * General conventions
 *   - Plain C ABI. Every matrix is row-major with a leading dimension `ld` in elements.
 *   - Every `data` pointer is DEVICE memory owned by the caller; every pointer inside
 *     `atp_seqs` and every options struct is HOST memory, read during the call only.
 *   - The library allocates no tensors. Scratch memory is a caller-owned device buffer handed
 *     over with atp_set_workspace(); its required size comes from atp_workspace_bytes().
 *     atp_create() allocates one small device status word and a pinned staging page, freed by
 *     atp_destroy().
 *   - Calls only enqueue work and return; they never wait for results, except
 *     atp_poll_device_status(). atp_principal_basis runs its iterations (orthonormalisation, Jacobi
 *     sweeps) inside persistent kernels that stop on their own convergence tests; nothing is read
 *     back by the host. The one exception is the one-sided Jacobi variant (opts->jacobi_block = 1),
 *     which reads its convergence flags while it enqueues sweeps and may block the calling thread
 *     until the GPU is within two sweeps of it (atp_basis_opts.no_host_sync turns that off).
 *     Work is ordered on the context's stream (atp_set_stream).
 *   - Errors the host can detect are returned at once and nothing is launched. Conditions only
 *     the device can see (ATP_ERR_NOT_CONVERGED: a Jacobi iteration that hit its sweep limit;
 *     ATP_ERR_TIMEOUT: a bounded wait - an mbarrier of a tensor-core pipeline, a barrier between
 *     the CTAs of a persistent kernel - that ran out; ATP_ERR_RANGE: a non-finite entry in the
 *     Gram matrix of the projected input, i.e. Inf / NaN in X or squares beyond fp32) are recorded
 *     in the status word, first one wins, and read back by atp_poll_device_status(); no kernel
 *     traps or spins without bound. Outputs of a call that raised one of them are unspecified.
 *   - dtype ATP_BF16 needs 16-byte aligned base pointers and `ld` a multiple of 8; otherwise
 *     ATP_ERR_INVALID_ARG is returned.
 *
 * Batches and ragged lengths: several independent sequences are packed row-wise.
 *   X, U_r, O, Y hold sum(L_b) rows; sequence b owns rows [row_off[b], row_off[b+1]).
 *   X_r holds sum(r_b) rows;         sequence b owns rows [rank_off[b], rank_off[b+1]).
 *   U_r has at least max(r_b) columns; sequence b uses the first r_b of them.
 *   sigma holds sum(r_b) floats laid out like the rows of X_r.
 * batch = 1 with row_off = {0, L} is the plain (X, r) call of the paper.
 */
#ifndef ATP_H_
#define ATP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Exported symbols (the library is built with hidden default visibility). */
#if defined(__GNUC__)
#define ATP_API __attribute__((visibility("default")))
#else
#define ATP_API
#endif

typedef enum {
    ATP_OK = 0,
    ATP_ERR_INVALID_ARG = 1,
    ATP_ERR_INVALID_RANK = 2,
    ATP_ERR_UNSUPPORTED_DTYPE = 3,
    ATP_ERR_WORKSPACE_TOO_SMALL = 4,
    ATP_ERR_CUDA = 5,
    ATP_ERR_NOT_CONVERGED = 6,
    ATP_ERR_TIMEOUT = 7,
    ATP_ERR_RANGE = 8,
    ATP_ERR_STATIC_SCRATCH_LIMIT = 9
} atp_status;

typedef enum { ATP_F32 = 0, ATP_BF16 = 1 } atp_dtype;

/* Device matrix, row-major; element (i, j) lives at data + (i*ld + j) * sizeof(dtype). */
typedef struct {
    void *data;
    atp_dtype dtype;
    int64_t rows, cols, ld;
} atp_mat;

/* Packed batch description; all three arrays are HOST memory. */
typedef struct {
    int32_t batch;
    const int32_t *row_off;   /* batch + 1 entries: rows of X / U_r / O / Y per sequence */
    const int32_t *rank;      /* batch entries: r_b                                       */
    const int32_t *rank_off;  /* batch + 1 entries: rows of X_r per sequence               */
} atp_seqs;

typedef enum { ATP_OP_BASIS = 0, ATP_OP_ATTENTION = 1, ATP_OP_LINEAR = 2, ATP_OP_NORM = 3, ATP_OP_ALTERNATING = 4 } atp_op;
typedef enum { ATP_Q_LOWRANK = 0, ATP_Q_FULL = 1 } atp_q_mode;
typedef enum { ATP_ACT_NONE = 0, ATP_ACT_GELU = 1, ATP_ACT_SWIGLU = 2 } atp_act;
typedef enum { ATP_NORM_RMS = 0, ATP_NORM_LAYER = 1 } atp_norm_kind;

/* Options. Set struct_size = sizeof(the struct); a NULL options pointer selects the defaults
 * (every numeric field below also treats 0 / negative as "default" where noted). */
typedef struct {
    uint32_t struct_size;
    int32_t oversample;    /* extra columns of the range finder; < 0: default 64              */
    int32_t power_iters;   /* subspace (power) iterations;        < 0: default 2              */
    int32_t max_sweeps;    /* Jacobi sweep limit;                 <= 0: default 24            */
    uint64_t seed;         /* seed of the +-1 test matrix                                      */
    int32_t jacobi_block;  /* 0 (default), 16 or 32: two-sided block Jacobi on the Gram matrix of the      */
                           /* projected rows, blocks of 32 rows (16 is accepted and means the same);       */
                           /* 1: one-sided Jacobi on the projected rows themselves (no Gram matrix)        */
    int32_t jacobi_inner;  /* accepted for compatibility, ignored                                          */
    int32_t groups;        /* one-sided variant only: 2 = split the batch in two groups on internal        */
                           /* streams (forked from and joined to the context's stream); otherwise ignored  */
    int32_t no_host_sync;  /* one-sided variant only. 0: the call reads the device's convergence flags     */
                           /* while it enqueues sweeps and stops early (it may block the calling thread).  */
                           /* Non-zero: nothing is read back; max_sweeps sweeps are enqueued, those of      */
                           /* converged sequences return at once. The default variant never reads back.    */
} atp_basis_opts;

typedef struct {
    uint32_t struct_size;
    int32_t q_mode;        /* atp_q_mode; LOWRANK: Q = U_r (X_r W_Q) (Eq. 6); FULL: Q = X W_Q  */
    float scale;           /* logit scale; <= 0: 1/sqrt(d_h)                                   */
    float rope_base;       /* 0: no positions. > 1: rotary positions (Sec. 4.2, "Combine with
                              Position Encoding"): the full keys K = U_r K' and the queries are
                              rotated row by row - the coordinate pair (2j, 2j+1) of every head by
                              position * rope_base^(-2j/d_h) - and the principal keys become
                              K'_rot = U_r^T K_rot. Values are not rotated.                      */
    const int32_t *positions; /* DEVICE, sum(L_b) ints, or NULL: a row's index in its sequence  */
} atp_attn_opts;

typedef struct {
    uint32_t struct_size;
    int32_t act;           /* atp_act                                                          */
    const float *bias;     /* device, d_out floats, nullable; added before the activation      */
    const atp_mat *W_gate; /* host struct, device data; required for ATP_ACT_SWIGLU            */
} atp_linear_opts;

typedef struct atp_ctx atp_ctx;

/* Context: binds a CUDA device; holds the stream, the workspace pointer and the status word. */
ATP_API atp_status atp_create(atp_ctx **ctx, int device);
ATP_API atp_status atp_destroy(atp_ctx *ctx);
/* cuda_stream is a cudaStream_t (NULL = default stream). */
ATP_API atp_status atp_set_stream(atp_ctx *ctx, void *cuda_stream);
/* Scratch bytes `op` needs for this batch (d = columns of X / X_r; d_out = columns of the widest
 * weight the call will see, i.e. d' for attention, d_out for a linear layer, ignored otherwise). */
ATP_API atp_status atp_workspace_bytes(atp_ctx *ctx, int op, const atp_seqs *seqs, int64_t d, int64_t d_out,
                               atp_dtype dtype, size_t *bytes);
/* The same for atp_principal_basis with the options it will be called with (the oversampling changes
 * the size; atp_workspace_bytes(ATP_OP_BASIS, ...) answers for the defaults). opts may be NULL. */
ATP_API atp_status atp_basis_workspace_bytes(atp_ctx *ctx, const atp_seqs *seqs, int64_t d, atp_dtype dtype,
                                             const atp_basis_opts *opts, size_t *bytes);
/* dev_ptr: device memory, 256-byte aligned, stays owned by the caller. Contents are scratch. */
ATP_API atp_status atp_set_workspace(atp_ctx *ctx, void *dev_ptr, size_t bytes);

/*
 * Norm box of Fig. 3 (unit gain): Y = norm(X + residual). RMSNorm x/sqrt(mean(x^2)+eps) or
 * LayerNorm (x-mean)/sqrt(var+eps), row by row, statistics in fp32. residual is nullable.
 * Y may alias X. All three share shape (rows x cols) and dtype.
 */
ATP_API atp_status atp_input_norm(atp_ctx *ctx, const atp_mat *X, const atp_mat *residual, int kind, float eps,
                          atp_mat *Y);

/*
 * Principal basis (Eq. 3, Eq. 5, Sec. 4.2): for every sequence b, the top-r_b left singular
 * vectors U_r (L_b x r_b, orthonormal columns) and X_r = U_r^T X = [sigma_1 v_1; ..; sigma_r v_r]
 * (r_b x d), components sorted by sigma descending, i.e. the minimiser of Eq. 9. Computed by a
 * randomised range finder with subspace iteration, block Gram-Schmidt orthonormalisation (one
 * persistent kernel per iterate) and a block Jacobi rotation of the small projected problem
 * (two-sided on the Gram matrix of the projected rows, two passes of one persistent kernel each;
 * one-sided on the rows themselves with opts->jacobi_block = 1) - not by a full SVD - so
 * the subspace is the optimal one up to the range finder's error; opts->power_iters trades passes
 * over X for that. The Jacobi sweeps stop on a device-side convergence test (largest scaled
 * off-diagonal <= 1e-6 for f32, 3e-5 for bf16); opts->max_sweeps bounds them, and a sequence that
 * has not converged by then raises ATP_ERR_NOT_CONVERGED on the device status word.
 * Sign of each component: sum of the column of U_r >= 0; if that sum is within 1e-6*sqrt(L_b) of
 * zero, the largest-magnitude entry of the row of X_r is positive.
 *   X      in   sum(L_b) x d                      (f32 or bf16)
 *   U_r    out  sum(L_b) x (>= max r_b), same dtype as X; columns >= r_b of a sequence untouched
 *   X_r    out  sum(r_b) x d, same dtype as X
 *   sigma  out  device, sum(r_b) floats, nullable
 * Requires 1 <= r_b <= min(L_b, d) (else ATP_ERR_INVALID_RANK).
 */
ATP_API atp_status atp_principal_basis(atp_ctx *ctx, const atp_mat *X, const atp_seqs *seqs,
                               const atp_basis_opts *opts, atp_mat *U_r, atp_mat *X_r, float *sigma);

/*
 * Attention of all queries on the r principal keys and values (Eq. 6, then the procedure of
 * Eq. 1 with K', V' in place of K, V; Fig. 2): Q' = X_r W_Q, K' = X_r W_K, V' = X_r W_V,
 * Q = U_r Q' (or X W_Q with q_mode FULL), and per head h (column block of width d'/heads)
 * O_h = Softmax(Q_h K'_h^T * scale) V'_h over the r_b keys of the sequence. No mask.
 *   X    in  sum(L_b) x d, nullable unless q_mode == ATP_Q_FULL
 *   W_*  in  d x d' each (so that X W matches Eq. 2); heads must divide d'
 *   O    out sum(L_b) x d', same dtype as U_r
 */
ATP_API atp_status atp_attention(atp_ctx *ctx, const atp_mat *X, const atp_mat *U_r, const atp_mat *X_r,
                         const atp_mat *W_Q, const atp_mat *W_K, const atp_mat *W_V, int heads,
                         const atp_seqs *seqs, const atp_attn_opts *opts, atp_mat *O);

/*
 * Linear layer through the low-rank representation (Sec. 4.3): Y = act(U_r (X_r W) + bias);
 * with ATP_ACT_SWIGLU, Y = silu(U_r (X_r W_gate)) * (U_r (X_r W)). GELU is the erf form.
 *   W  in  d_in x d_out;  Y out sum(L_b) x d_out, same dtype as U_r
 */
ATP_API atp_status atp_lowrank_linear(atp_ctx *ctx, const atp_mat *U_r, const atp_mat *X_r, const atp_mat *W,
                              const atp_seqs *seqs, const atp_linear_opts *opts, atp_mat *Y);

/* Synchronises the stream, returns and clears the device-side status (ATP_OK if none): see the general
 * conventions above for ATP_ERR_NOT_CONVERGED, ATP_ERR_TIMEOUT, ATP_ERR_RANGE. */
ATP_API atp_status atp_poll_device_status(atp_ctx *ctx);
/* Number of kernels this context has launched since creation (for accounting). */
ATP_API int64_t atp_launch_count(const atp_ctx *ctx);
ATP_API const char *atp_status_string(atp_status s);

/*
 * Per-kernel timing (tracing aid, not part of the paper's method). Between start and stop every
 * kernel launch of this context is bracketed by a pair of CUDA events on the context's stream,
 * which slows the calls down: never leave it on while measuring throughput. stop synchronises and
 * writes one text line per kernel name into buf (host memory, cap bytes, always NUL-terminated):
 *   "<name> <launches> <total ms> <algorithmic flops> <algorithmic bytes>\n"
 * *needed (nullable) receives the size a complete report takes.
 */
ATP_API atp_status atp_profile_start(atp_ctx *ctx);
ATP_API atp_status atp_profile_stop(atp_ctx *ctx, char *buf, size_t cap, size_t *needed);

/*
 * Self-tests of the library's own bookkeeping (no counterpart in the paper; used by the test suite).
 * atp_selftest_wait_timeout enqueues a kernel whose inter-CTA barrier can never complete (it expects
 * a second CTA that does not exist) with a short wait limit: the kernel gives up and raises
 * ATP_ERR_TIMEOUT on the status word, which the next atp_poll_device_status returns; the context stays
 * usable. It needs a workspace of at least 256 bytes.
 * atp_selftest_per_device_once runs the once-per-device set-up helper (kernel attributes, symbol
 * addresses) through a fixed script on the host and returns how often the guarded step ran (7).
 */
ATP_API atp_status atp_selftest_wait_timeout(atp_ctx *ctx);
ATP_API int atp_selftest_per_device_once(void);

/*
 * Low-rank linear layer without any allocation (the paper has no counterpart: this entry point
 * exists for deployment, not for the method). It computes what atp_lowrank_linear computes,
 * Y = act(U_r (X_r W) + bias) with act NONE or GELU, for callers that may not allocate device
 * memory at all: code running inside another program's memory pool, or a latency-critical loop
 * where cudaMalloc / cudaFree are forbidden. Such callers cannot use atp_create (it allocates a
 * status word) nor supply a workspace, so this call takes no context: it runs on the device that
 * is current, on the given stream (cudaStream_t, NULL = default), and keeps its intermediate
 * X_r W in a fixed buffer of ATP_STATIC_SCRATCH_BYTES that is part of the library image. Every GPU
 * that loads the library holds that buffer until the process exits.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine; inputs and outputs are the
 *     caller's, as in atp_lowrank_linear (same layouts, same dtype rules). SwiGLU is not offered.
 *   - Limit: sum(r_b) * d_out * 4 bytes must fit in ATP_STATIC_SCRATCH_BYTES, otherwise
 *     ATP_ERR_STATIC_SCRATCH_LIMIT is returned and nothing is launched.
 *   - There is no context, hence no status word: a bounded wait of the tensor-core pipeline that
 *     ran out (ATP_ERR_TIMEOUT elsewhere) ends the kernel early here without being reported.
 *   - The first call on each device looks up the buffer's device address; make that first call
 *     before starting any stream capture on that device.
 *   - All calls share the one buffer, and it keeps whatever the previous call left in it. The
 *     intermediate is rewritten in full before it is read, so no clearing is needed, but two calls
 *     that overlap on the GPU (different streams, no ordering between them) race on it: order them.
 */
#define ATP_STATIC_SCRATCH_BYTES (8u << 20)
ATP_API atp_status atp_lowrank_linear_static(void *cuda_stream, const atp_mat *U_r, const atp_mat *X_r,
                                             const atp_mat *W, const atp_seqs *seqs, const atp_linear_opts *opts,
                                             atp_mat *Y);

/*
 * Algorithm 1 (appendix B; described in Sec. 4.2): the paper's own approximate extraction by
 * alternating rank-1 fits with deflation. For every sequence b and component i < r_b, starting from
 * v = row (rank_off[b] + i) of V0:  `inner` rounds of  u = R v / |v|^2,  v = R^T u / |u|^2  on the
 * deflated matrix R (R = X for i = 0), then R <- R - u v^T. Outputs, as Sec. 4.2 puts the scale into
 * v:  U_r[:, i] = u / |u|  and  X_r[i, :] = v |u|.  The columns of U_r are NOT orthonormalised and not
 * sorted; no sign rule is applied (the result is fixed by V0). The paper runs inner = 2.
 *   X      in   sum(L_b) x d                      (f32 or bf16)
 *   V0     in   sum(r_b) x d, f32                 the start vectors (the method's random draw is an
 *                                                 input, so that two implementations can be compared)
 *   inner  in   1..64
 *   U_r    out  sum(L_b) x max_b(r_b), same dtype as X
 *   X_r    out  sum(r_b) x d, same dtype as X
 * Arithmetic: R, u, v are held in fp32, every dot product accumulates in fp64.
 * Workspace: atp_workspace_bytes(ATP_OP_ALTERNATING, seqs, d, 0, dtype). r_b <= min(L_b, d).
 * Errors: as atp_principal_basis (no convergence status: the iteration count is fixed).
 */
ATP_API atp_status atp_alternating_basis(atp_ctx *ctx, const atp_mat *X, const atp_seqs *seqs, const atp_mat *V0,
                                         int inner, atp_mat *U_r, atp_mat *X_r);

/*
 * SVD entropy (Eq. 4) and the rank it suggests (Sec. 3): for each of `batch` groups of singular
 * values, mu = -log2(sum_i sbar_i^2) with sbar_i = sigma_i / sum_j sigma_j, and rank = ceil(2^mu).
 *   sigma    in   device, f32, packed groups
 *   offsets  in   HOST, batch + 1 ints: group b is sigma[offsets[b] .. offsets[b+1]); offsets[0] = 0
 *   mu       out  device, f32, batch values
 *   rank     out  device, int32, batch values; may be NULL
 * Sums, the logarithm and the ceiling are taken in fp64 (an exact power of two such as 8 equal values
 * gives rank 8, not 9: 1e-9 is subtracted before the ceiling). An empty or all-zero group gives mu = 0,
 * rank = 0. The entropy describes the WHOLE spectrum: feed it the sigma of a full-rank call
 * (r_b = min(L_b, d)) of atp_principal_basis.
 */
ATP_API atp_status atp_svd_entropy(atp_ctx *ctx, const float *sigma, const int32_t *offsets, int32_t batch, float *mu,
                                   int32_t *rank);

#ifdef __cplusplus
}
#endif
#endif /* ATP_H_ */
