"""GPU parity tests: the CUDA path (through the C-ABI binding) against the CPU oracle.

T1  invariants of the basis the GPU returns (orthonormality, X_r = U_r^T X, optimal residual,
    X_r X_r^T diagonal, sigma).
T2  stage parity: oracle attention / linear evaluated in double on the very (U_r, X_r) the GPU
    produced, and GPU attention / linear run on the oracle's basis. This is the binding check
    for O and Y: bars 1e-4 (fp32) and 2e-2 (bf16), max|G-R| / max|R|.
T3  end to end on inputs with a spectral gap at r (exact-rank, distinct sigma).
"""
import math

import numpy as np
import pytest
import torch

import atp_inputs as ai
import oracle
from gpu_util import TOL, basis_invariants, rel_err, residual_ok, tdtype, to_dev, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2403_02352_b200 as atp
    c = atp.Context(0)
    yield c
    c.close()


def _atp():
    import paper_2403_02352_b200 as atp
    return atp


def _weights(rng, d, dout, dtype, n=3):
    return [ai.finish(ai.gaussian_weight(rng, d, dout), dtype) for _ in range(n)]


def _noisy(rng, L, d, k, dtype, noise=0.02, decay=0.85):
    x, s = ai.planted_matrix(rng, L, d, decay ** np.arange(k), noise)
    return ai.finish(x, dtype)


# ------------------------------------------------------------------------------- linear (a5)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("act", [None, "gelu", "swiglu"])
def test_lowrank_linear_vs_oracle(ctx, dtype, act):
    atp = _atp()
    rng = np.random.default_rng(10)
    L, d, dout, r = 203, 96, 136, 37                   # ragged against the 64-wide tiles
    X = _noisy(rng, L, d, 12, "f64")
    U, Xr, _ = oracle.principal_basis(X, r)
    U, Xr = ai.finish(U, dtype), ai.finish(Xr, dtype)
    W, Wg = _weights(rng, d, dout, dtype, 2)
    bias = rng.standard_normal(dout).astype(np.float32) if act != "swiglu" else None
    ref = oracle.lowrank_linear(U, Xr, W, bias=bias, W_gate=Wg if act == "swiglu" else None, act=act)
    Y = atp.atp_lowrank_linear(ctx, to_dev(U, dtype), to_dev(Xr, dtype), to_dev(W, dtype), [L], [r],
                               bias=torch.from_numpy(bias).cuda() if bias is not None else None, act=act,
                               W_gate=to_dev(Wg, dtype) if act == "swiglu" else None)
    ctx.poll()
    assert rel_err(to_np(Y), ref) <= TOL[dtype]


# ---------------------------------------------------------------------------- attention (a2-a4)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("q_mode", ["lowrank", "full"])
@pytest.mark.parametrize("L,d,heads,dh,r", [(150, 128, 2, 64, 45), (70, 96, 3, 32, 70), (257, 256, 2, 128, 129)])
def test_attention_on_oracle_basis(ctx, dtype, q_mode, L, d, heads, dh, r):
    atp = _atp()
    rng = np.random.default_rng(L + r)
    dp = heads * dh
    X = _noisy(rng, L, d, 10, dtype)
    U, Xr, _ = oracle.principal_basis(X, r)
    U, Xr = ai.finish(U, dtype), ai.finish(Xr, dtype)
    WQ, WK, WV = _weights(rng, d, dp, dtype)
    ref = oracle.attention(X, U, Xr, WQ, WK, WV, heads, q_mode=1 if q_mode == "full" else 0)
    O = atp.atp_attention(ctx, to_dev(X, dtype), to_dev(U, dtype), to_dev(Xr, dtype), to_dev(WQ, dtype),
                          to_dev(WK, dtype), to_dev(WV, dtype), heads, [L], [r], q_mode=q_mode)
    ctx.poll()
    assert rel_err(to_np(O), ref) <= TOL[dtype]


def test_attention_scale_override_and_single_key(ctx):
    atp = _atp()
    rng = np.random.default_rng(77)
    L, d, heads, dh = 40, 64, 2, 32
    X = _noisy(rng, L, d, 6, "f32")
    U, Xr, _ = oracle.principal_basis(X, 1)
    WQ, WK, WV = _weights(rng, d, heads * dh, "f32")
    O = atp.atp_attention(ctx, None, to_dev(U, "f32"), to_dev(Xr, "f32"), to_dev(WQ, "f32"), to_dev(WK, "f32"),
                          to_dev(WV, "f32"), heads, [L], [1])
    ctx.poll()
    assert rel_err(to_np(O), np.tile(Xr @ WV, (L, 1))) <= 1e-5        # softmax over one key
    U, Xr, _ = oracle.principal_basis(X, 9)
    ref = oracle.attention(None, U, Xr, WQ, WK, WV, heads, scale=0.05)
    O = atp.atp_attention(ctx, None, to_dev(U, "f32"), to_dev(Xr, "f32"), to_dev(WQ, "f32"), to_dev(WK, "f32"),
                          to_dev(WV, "f32"), heads, [L], [9], scale=0.05)
    ctx.poll()
    assert rel_err(to_np(O), ref) <= 1e-4


# ------------------------------------------------------------------------------- basis (a1)
def _run_basis(ctx, seqs, dtype, **kw):
    atp = _atp()
    X = np.concatenate([s for s, _ in seqs], axis=0)
    lengths = [s.shape[0] for s, _ in seqs]
    ranks = [r for _, r in seqs]
    U, Xr, sig = atp.atp_principal_basis(ctx, to_dev(X, dtype), lengths, ranks, **kw)
    ctx.poll()
    U, Xr, sig = to_np(U), to_np(Xr), to_np(sig.reshape(-1, 1)).ravel()
    out = []
    ro = np.concatenate([[0], np.cumsum(lengths)]); ko = np.concatenate([[0], np.cumsum(ranks)])
    for b, (s, r) in enumerate(seqs):
        out.append((U[ro[b]:ro[b + 1], :r], Xr[ko[b]:ko[b + 1]], sig[ko[b]:ko[b + 1]]))
    return out


def _check_t1(X, U, Xr, sig, dtype, ratio_tol):
    inv = basis_invariants(X, U, Xr, sig)
    eps = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -23
    assert inv["orth"] <= (2e-2 if dtype == "bf16" else 5e-5), inv
    assert inv["xr_vs_utx"] <= 8 * eps, inv            # relative to sigma_1
    assert residual_ok(inv["res_sub"], inv["opt"], inv["normX"], dtype, ratio_tol), inv
    assert inv["offdiag"] <= (5e-2 if dtype == "bf16" else 1e-4), inv
    assert inv["sigma_vs_rows"] <= 4 * eps, inv
    assert inv["sorted"], inv
    return inv


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,d,r,k", [(300, 200, 40, 16), (200, 300, 64, 24), (130, 513, 33, 8)])
def test_basis_invariants_noisy(ctx, dtype, L, d, r, k):
    rng = np.random.default_rng(L * 7 + d)
    X = _noisy(rng, L, d, k, dtype)
    (U, Xr, sig), = _run_basis(ctx, [(X, r)], dtype)
    _check_t1(X, U, Xr, sig, dtype, 3e-2)


@pytest.mark.parametrize("jb", [1, 32])
def test_basis_invariants_other_jacobi_variants_fp32(ctx, jb):
    """jacobi_block = 1: the one-sided rotation of the projected rows themselves; 32: 64x64 diagonal blocks."""
    rng = np.random.default_rng(91 + jb)
    X = _noisy(rng, 300, 200, 16, "f32")
    (U, Xr, sig), = _run_basis(ctx, [(X, 40)], "f32", jacobi_block=jb)
    _check_t1(X, U, Xr, sig, "f32", 3e-2)


def test_basis_more_power_iterations_approach_the_optimum(ctx):
    rng = np.random.default_rng(5)
    X = _noisy(rng, 256, 192, 10, "f32")
    ratios = []
    for q in (0, 2, 8):
        (U, Xr, sig), = _run_basis(ctx, [(X, 48)], "f32", power_iters=q)
        ratios.append(basis_invariants(X, U, Xr, sig)["res_ratio"])
    assert ratios[0] > ratios[1] > ratios[2] >= 1.0 - 1e-6
    assert ratios[2] <= 1.0 + 3e-3


@pytest.mark.parametrize("L,d,k", [(160, 224, 20), (224, 160, 20)])
def test_basis_exact_rank_recovery_fp32(ctx, L, d, k):
    X, s = ai.exact_rank(L, d, k, dtype="f32", decay=0.8, seed=L)
    for r in (k, k + 13):
        (U, Xr, sig), = _run_basis(ctx, [(X, r)], "f32")
        assert np.abs(U.T @ U - np.eye(r)).max() < 1e-4
        assert np.linalg.norm(U @ Xr - X) <= 2e-5 * np.linalg.norm(X)           # Eq. 5 on exact-rank input
        assert np.allclose(sig[:k], s, rtol=2e-5)
        if r > k:
            assert np.abs(Xr[k:]).max() <= 1e-4 * s[0]


def test_basis_edge_cases(ctx):
    rng = np.random.default_rng(3)
    # r = 1, r = min(L, d) on both orientations, a zero matrix, an empty sequence in the batch
    X1 = _noisy(rng, 90, 70, 5, "f32")
    (U, Xr, sig), = _run_basis(ctx, [(X1, 1)], "f32")
    s = np.linalg.svd(X1, compute_uv=False)
    assert abs(sig[0] - s[0]) <= 1e-4 * s[0] and U.sum() >= 0
    for X in (X1, X1.T.copy()):
        n = min(X.shape)
        (U, Xr, sig), = _run_basis(ctx, [(X, n)], "f32")
        assert np.abs(U.T @ U - np.eye(n)).max() < 5e-5
        assert np.linalg.norm(U @ Xr - X) <= 1e-4 * np.linalg.norm(X)
        assert np.allclose(sig, np.linalg.svd(X, compute_uv=False), rtol=1e-3, atol=1e-5 * s[0])
    Z = np.zeros((48, 32))
    (U, Xr, sig), = _run_basis(ctx, [(Z, 8)], "f32")
    assert np.all(Xr == 0) and np.all(sig == 0)
    assert np.abs(U.T @ U - np.eye(8)).max() < 1e-4
    outs = _run_basis(ctx, [(X1, 10), (np.zeros((0, 70)), 0), (X1[:40], 7)], "f32")
    assert outs[1][0].shape[0] == 0
    _check_t1(X1, *outs[0], "f32", 5e-2)
    _check_t1(X1[:40], *outs[2], "f32", 5e-2)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_batch_end_to_end_stage_parity(ctx, dtype):
    """Packed batch with ragged lengths and ranks (r_b = L_b // 4), T1 + T2 per sequence."""
    atp = _atp()
    rng = np.random.default_rng(42)
    d, heads, dh = 128, 2, 64
    lengths = [130, 77, 200, 64]
    ranks = [l // 4 for l in lengths]
    Xs = [_noisy(rng, l, d, 9, dtype) for l in lengths]
    WQ, WK, WV = _weights(rng, d, d, dtype)
    Wl, = _weights(rng, d, 96, dtype, 1)
    Xd = to_dev(np.concatenate(Xs), dtype)
    U, Xr, sig = atp.atp_principal_basis(ctx, Xd, lengths, ranks)
    O = atp.atp_attention(ctx, Xd, U, Xr, to_dev(WQ, dtype), to_dev(WK, dtype), to_dev(WV, dtype), heads, lengths, ranks)
    Y = atp.atp_lowrank_linear(ctx, U, Xr, to_dev(Wl, dtype), lengths, ranks, act="gelu")
    ctx.poll()
    Un, Xrn, sn, On, Yn = to_np(U), to_np(Xr), to_np(sig.reshape(-1, 1)).ravel(), to_np(O), to_np(Y)
    ro = np.concatenate([[0], np.cumsum(lengths)]); ko = np.concatenate([[0], np.cumsum(ranks)])
    for b in range(len(lengths)):
        Ub, Xrb = Un[ro[b]:ro[b + 1], :ranks[b]], Xrn[ko[b]:ko[b + 1]]
        _check_t1(Xs[b], Ub, Xrb, sn[ko[b]:ko[b + 1]], dtype, 5e-2)
        assert rel_err(On[ro[b]:ro[b + 1]], oracle.attention(None, Ub, Xrb, WQ, WK, WV, heads)) <= TOL[dtype]
        assert rel_err(Yn[ro[b]:ro[b + 1]], oracle.lowrank_linear(Ub, Xrb, Wl, act="gelu")) <= TOL[dtype]


def test_end_to_end_on_gap_input_fp32(ctx):
    """T3: exact-rank input with distinct sigma and r = rank: GPU basis -> GPU attention against
    oracle basis -> oracle attention. The bar is looser than T2's because the logits amplify the
    fp32 rounding of the basis before the exponential."""
    atp = _atp()
    L, d, k, heads = 192, 128, 12, 2
    X, s = ai.exact_rank(L, d, k, dtype="f32", decay=0.7, seed=9)
    rng = np.random.default_rng(1)
    WQ, WK, WV = _weights(rng, d, d, "f32")
    Uo, Xro, _ = oracle.principal_basis(X, k)
    assert np.abs(Uo.sum(0)).min() > 1e-3 * math.sqrt(L)         # signs well determined on this input
    ref = oracle.attention(None, Uo, Xro, WQ, WK, WV, heads)
    Xd = to_dev(X, "f32")
    U, Xr, sig = atp.atp_principal_basis(ctx, Xd, [L], [k])
    O = atp.atp_attention(ctx, None, U, Xr, to_dev(WQ, "f32"), to_dev(WK, "f32"), to_dev(WV, "f32"), heads, [L], [k])
    ctx.poll()
    assert rel_err(to_np(U) @ to_np(Xr), Uo @ Xro) <= 1e-5
    assert rel_err(to_np(O), ref) <= 2e-3


# ------------------------------------------------------------------------------- norm (a0)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("kind", ["rms", "layer"])
def test_norm_vs_oracle(ctx, dtype, kind):
    atp = _atp()
    rng = np.random.default_rng(8)
    X = ai.finish(rng.standard_normal((67, 200)) * 2 + 0.5, dtype)
    R = ai.finish(rng.standard_normal((67, 200)), dtype)
    for res in (None, R):
        ref = oracle.norm(X, residual=res, kind=kind, eps=1e-5)
        Y = atp.atp_input_norm(ctx, to_dev(X, dtype), to_dev(res, dtype) if res is not None else None, kind=kind, eps=1e-5)
        ctx.poll()
        assert rel_err(to_np(Y), ref) <= (1e-5 if dtype == "f32" else 8e-3)


# ------------------------------------------------------------------------------- host errors
def test_host_detected_errors(ctx):
    atp = _atp()
    from paper_2403_02352_b200 import binding as B
    X = torch.zeros((16, 8), device="cuda")
    with pytest.raises(atp.AtpError) as e:
        atp.atp_principal_basis(ctx, X, [16], [9])                # r > d
    assert e.value.code == B.ERR_INVALID_RANK
    with pytest.raises(atp.AtpError) as e:
        atp.atp_principal_basis(ctx, X, [16], [0])
    assert e.value.code == B.ERR_INVALID_RANK
    with pytest.raises(atp.AtpError) as e:
        atp.atp_principal_basis(ctx, X, [15], [4])                # rows do not add up
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(atp.AtpError) as e:
        atp.atp_principal_basis(ctx, X.double(), [16], [4])
    assert e.value.code == B.ERR_UNSUPPORTED_DTYPE
    ctx.set_workspace(torch.empty(256, dtype=torch.uint8, device="cuda"))
    with pytest.raises(atp.AtpError) as e:
        atp.atp_principal_basis(ctx, X, [16], [4], auto_workspace=False)
    assert e.value.code == B.ERR_WORKSPACE_TOO_SMALL
    U = torch.zeros((16, 4), device="cuda"); Xr = torch.zeros((4, 8), device="cuda"); W = torch.zeros((8, 12), device="cuda")
    with pytest.raises(atp.AtpError) as e:
        atp.atp_attention(ctx, None, U, Xr, W, W, W, 5, [16], [4])   # heads do not divide d'
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(atp.AtpError) as e:
        atp.atp_lowrank_linear(ctx, U, Xr, W, [16], [4], act="swiglu")   # gate weight missing
    assert e.value.code == B.ERR_INVALID_ARG
    ctx.poll()
