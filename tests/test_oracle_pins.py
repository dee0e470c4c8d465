"""Pins of the CPU oracle against things the paper and the mathematics fix.

None of these tests calls the CUDA library. Each one would fail for a plausible
mistake in the oracle (dropped term, wrong sign or index, transposed operand).
"""
import itertools
import math
import os

import numpy as np
import pytest

import atp_inputs as ai
import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


# ----------------------------------------------------------------------------- SVD (Eq. 3)
def _golden():
    out = []
    for line in open(os.path.join(HERE, "golden", "svd_closed_forms.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, mat, sv = [p.strip() for p in line.split("|")]
        rows = [[eval(e, {"sqrt": math.sqrt}) for e in r.split(",")] for r in mat.split(";")]
        svals = [eval(e, {"sqrt": math.sqrt}) for e in sv.split(",")]
        out.append((name, np.array(rows, dtype=float), np.array(svals, dtype=float)))
    return out


@pytest.mark.parametrize("name,X,sv", _golden(), ids=[g[0] for g in _golden()])
def test_svd_closed_forms(name, X, sv):
    U, S, Vt, _ = oracle.svd_jacobi(X)
    assert np.allclose(S, sv, rtol=1e-12, atol=1e-13)
    assert np.allclose((U * S) @ Vt, X, atol=1e-13)
    n = min(X.shape)
    assert np.allclose(U.T @ U, np.eye(n), atol=1e-13)
    assert np.allclose(Vt @ Vt.T, np.eye(n), atol=1e-13)


@pytest.mark.parametrize("L,d", [(40, 64), (64, 40), (33, 33), (1, 7), (7, 1)])
def test_svd_reconstruction_orthonormality_and_lapack(L, d):
    rng = np.random.default_rng(L * 100 + d)
    X = rng.standard_normal((L, d))
    U, S, Vt, sweeps = oracle.svd_jacobi(X)
    n = min(L, d)
    assert sweeps < 60
    assert np.abs((U * S) @ Vt - X).max() <= 1e-12 * np.abs(X).max()
    assert np.abs(U.T @ U - np.eye(n)).max() < 1e-13
    assert np.abs(Vt @ Vt.T - np.eye(n)).max() < 1e-13
    assert np.all(np.diff(S) <= 0)
    assert np.allclose(S, np.linalg.svd(X, compute_uv=False), rtol=1e-12)   # library cross-check


@pytest.mark.parametrize("L,d,k", [(48, 80, 12), (80, 48, 12)])
def test_svd_planted_spectrum_closed_form(L, d, k):
    rng = np.random.default_rng(5)
    X, s = ai.planted_matrix(rng, L, d, 0.7 ** np.arange(k), 0.0)
    U, S, Vt, _ = oracle.svd_jacobi(X)
    assert np.allclose(S[:k], s, rtol=1e-12)
    assert np.all(S[k:] <= 1e-12 * s[0])
    # rank-deficient: the completed vectors must still be orthonormal
    n = min(L, d)
    assert np.abs(U.T @ U - np.eye(n)).max() < 1e-12
    assert np.abs(Vt @ Vt.T - np.eye(n)).max() < 1e-12


def test_svd_rank_one_and_permutation():
    a = np.array([1.0, -2.0, 3.0, 0.5]); b = np.array([2.0, 0.0, -1.0])
    U, S, Vt, _ = oracle.svd_jacobi(np.outer(a, b))
    assert np.isclose(S[0], np.linalg.norm(a) * np.linalg.norm(b), rtol=1e-14)
    assert np.allclose(np.abs(U[:, 0]), np.abs(a) / np.linalg.norm(a), atol=1e-14)
    assert np.allclose(np.abs(Vt[0]), np.abs(b) / np.linalg.norm(b), atol=1e-14)
    P = np.eye(5)[[2, 0, 4, 1, 3]] * np.array([5.0, 4, 3, 2, 1])[:, None]
    U, S, Vt, _ = oracle.svd_jacobi(P)
    assert np.allclose(S, [5, 4, 3, 2, 1])
    assert np.allclose((U * S) @ Vt, P, atol=1e-14)


# ------------------------------------------------ principal basis (Eq. 5, Sec. 4.2, Eq. 9)
def test_basis_eckart_young_and_energy_ratio():
    rng = np.random.default_rng(11)
    L, d, r = 60, 90, 17
    spec = np.linspace(3.0, 0.1, 60)
    X, s = ai.planted_matrix(rng, L, d, spec, 0.0)          # full planted spectrum, known exactly
    U_r, X_r, sig, sall = oracle.principal_basis(X, r, return_all_sigma=True)
    assert np.allclose(sig, s[:r], rtol=1e-12)
    assert np.abs(U_r.T @ U_r - np.eye(r)).max() < 1e-13
    # Eckart-Young closed form of the optimum of Eq. 9
    res2 = np.linalg.norm(X - U_r @ X_r) ** 2
    assert np.isclose(res2, (s[r:] ** 2).sum(), rtol=1e-11)
    # energy ratio |X'|_F^2 / |X|_F^2 (Fig. 5)
    assert np.isclose(np.linalg.norm(X_r) ** 2 / np.linalg.norm(X) ** 2,
                      (s[:r] ** 2).sum() / (s ** 2).sum(), rtol=1e-12)
    # X' = [sigma_i v_i]: rows mutually orthogonal with norms sigma_i
    G = X_r @ X_r.T
    assert np.allclose(G, np.diag(s[:r] ** 2), atol=1e-11)
    assert np.allclose(X_r, U_r.T @ X, atol=1e-12)


def test_basis_brute_force_rank_one_tiny():
    """r = 1 on tiny inputs: no unit vector u does better than the oracle's (Eq. 9)."""
    rng = np.random.default_rng(3)
    for (L, d) in [(2, 3), (3, 3), (3, 4)]:
        X = rng.standard_normal((L, d))
        U_r, X_r, sig = oracle.principal_basis(X, 1)
        best = np.linalg.norm(X - U_r @ X_r)
        # dense grid over the unit sphere of R^L (L <= 3): for fixed u the best X' is u^T X
        worst_gap = np.inf
        if L == 2:
            cand = [np.array([math.cos(t), math.sin(t)]) for t in np.linspace(0, math.pi, 4001)]
        else:
            cand = []
            for t in np.linspace(0, math.pi, 241):
                for p in np.linspace(0, math.pi, 241):
                    cand.append(np.array([math.sin(t) * math.cos(p), math.sin(t) * math.sin(p), math.cos(t)]))
        for u in cand:
            res = np.linalg.norm(X - np.outer(u, u @ X))
            worst_gap = min(worst_gap, res - best)
        assert worst_gap > -1e-12            # nothing beats it
        assert worst_gap < 1e-3              # and the grid gets close to it


def test_basis_exact_recovery_and_eq6():
    X, s = ai.exact_rank(50, 70, 9, dtype="f64", seed=21)
    rng = np.random.default_rng(2)
    W = [ai.gaussian_weight(rng, 70, 32) for _ in range(3)]
    for r in (9, 14):                      # r >= rank: X = U X' exactly (Eq. 5)
        U_r, X_r, sig = oracle.principal_basis(X, r)
        assert np.abs(U_r @ X_r - X).max() < 1e-12 * s[0]
        assert np.abs(U_r.T @ U_r - np.eye(r)).max() < 1e-12
        for w in W:                        # Q,K,V = U {Q',K',V'} (Eq. 6)
            assert np.abs(U_r @ (X_r @ w) - X @ w).max() < 1e-12 * s[0]
        if r > 9:                          # rows of X' beyond the rank are zero
            assert np.abs(X_r[9:]).max() < 1e-12 * s[0]


def test_basis_sign_convention():
    rng = np.random.default_rng(8)
    X = rng.standard_normal((30, 40))
    U_r, X_r, _ = oracle.principal_basis(X, 10)
    assert np.all(U_r.sum(axis=0) >= 0)
    U2, X2, _ = oracle.principal_basis(-X, 10)      # negating X flips v, not the convention on u
    assert np.allclose(U2, U_r, atol=1e-12) and np.allclose(X2, -X_r, atol=1e-12)
    # fallback rule: columns of U summing to ~0. X = [a; -a] stacked makes every u antisymmetric.
    A = rng.standard_normal((6, 9))
    Xa = np.concatenate([A, -A], axis=0)
    U3, X3, s3 = oracle.principal_basis(Xa, 4)
    assert np.abs(U3.sum(axis=0)).max() < 1e-12
    for a in range(4):
        assert X3[a, np.argmax(np.abs(X3[a]))] > 0


def test_basis_invalid_rank():
    X = np.ones((4, 6))
    with pytest.raises(ValueError):
        oracle.principal_basis(X, 5)
    with pytest.raises(ValueError):
        oracle.principal_basis(X, 0)


# ------------------------------------------------------------------ attention (Eq. 1, 6, 7, 8)
def _textbook_attention(X, WQ, WK, WV, heads):
    """Independent statement of Eq. 1-2 with heads as column blocks."""
    Q, K, V = X @ WQ, X @ WK, X @ WV
    dh = Q.shape[1] // heads
    out = np.zeros_like(Q)
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        S = Q[:, sl] @ K[:, sl].T / math.sqrt(dh)
        P = np.exp(S - S.max(axis=1, keepdims=True))
        P /= P.sum(axis=1, keepdims=True)
        out[:, sl] = P @ V[:, sl]
    return out


def test_attention_reduces_to_textbook():
    rng = np.random.default_rng(4)
    L, d, dp, heads = 24, 20, 16, 4
    X = rng.standard_normal((L, d))
    WQ, WK, WV = (ai.gaussian_weight(rng, d, dp) for _ in range(3))
    ref = _textbook_attention(X, WQ, WK, WV, heads)
    O = oracle.attention(None, np.eye(L), X, WQ, WK, WV, heads)        # U = I, X' = X, r = L
    assert np.abs(O - ref).max() < 1e-13
    O2 = oracle.attention(X, np.eye(L), X, WQ, WK, WV, heads, q_mode=1)
    assert np.abs(O2 - ref).max() < 1e-13
    # full-rank basis (r = L): K = U K' is a rotation of the keys, not the keys themselves, so
    # the softmax result differs in general, but the FULL-query mode on an orthogonal U with
    # a scale override must still follow Eq. 1 on the rotated keys:
    U_r, X_r, _ = oracle.principal_basis(X, min(L, d))
    O3 = oracle.attention(X, U_r, X_r, WQ, WK, WV, heads, q_mode=1, scale=0.3)
    Kp, Vp, Q = X_r @ WK, X_r @ WV, X @ WQ
    dh = dp // heads
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        S = 0.3 * Q[:, sl] @ Kp[:, sl].T
        P = np.exp(S - S.max(1, keepdims=True)); P /= P.sum(1, keepdims=True)
        assert np.abs(O3[:, sl] - P @ Vp[:, sl]).max() < 1e-13


def test_attention_single_key_and_sign_dependence():
    rng = np.random.default_rng(6)
    L, d, dp, heads = 12, 10, 8, 2
    X = rng.standard_normal((L, d))
    WQ, WK, WV = (ai.gaussian_weight(rng, d, dp) for _ in range(3))
    U_r, X_r, _ = oracle.principal_basis(X, 1)
    O = oracle.attention(None, U_r, X_r, WQ, WK, WV, heads)
    assert np.allclose(O, np.tile(X_r @ WV, (L, 1)), atol=1e-13)     # softmax over one key is 1
    Of = oracle.attention(None, -U_r, -X_r, WQ, WK, WV, heads)      # flipped sign: same X, other O
    assert np.allclose(Of, -O, atol=1e-13)


def test_attention_invariants():
    rng = np.random.default_rng(9)
    L, d, dp, heads, r = 30, 26, 12, 3, 7
    X = rng.standard_normal((L, d))
    WQ, WK, WV = (ai.gaussian_weight(rng, d, dp) for _ in range(3))
    U_r, X_r, _ = oracle.principal_basis(X, r)
    O = oracle.attention(None, U_r, X_r, WQ, WK, WV, heads)
    Vp = X_r @ WV
    # each output row is a convex combination of the rows of V' (head by head)
    assert np.all(O <= Vp.max(axis=0) + 1e-12) and np.all(O >= Vp.min(axis=0) - 1e-12)
    # permuting the components leaves O unchanged
    perm = rng.permutation(r)
    Op = oracle.attention(None, U_r[:, perm], X_r[perm], WQ, WK, WV, heads)
    assert np.abs(Op - O).max() < 1e-13
    # shifting all keys of a head by a vector c adds q.c to every score of a row: O unchanged.
    # (X_r -> X_r + 1 t^T shifts every K' row by t W_K.) Values are kept fixed through W_V = 0 part.
    # a zero row of X' is a key with score 0 and value 0 (weight exp(0 - max)):
    Uz = np.concatenate([U_r, np.zeros((L, 1))], axis=1)
    Xz = np.concatenate([X_r, np.zeros((1, d))], axis=0)
    Oz = oracle.attention(None, Uz, Xz, WQ, WK, WV, heads)
    dh = dp // heads
    Q = U_r @ (X_r @ WQ); Kp = X_r @ WK
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        S = Q[:, sl] @ Kp[:, sl].T / math.sqrt(dh)
        S = np.concatenate([S, np.zeros((L, 1))], axis=1)
        P = np.exp(S - S.max(1, keepdims=True)); P /= P.sum(1, keepdims=True)
        assert np.abs(Oz[:, sl] - P[:, :r] @ Vp[:, sl]).max() < 1e-13


def test_linearised_identity_and_taylor_order():
    """Eq. 7-8: for exact-rank X, q K^T V = q K'^T V' for any orthonormal basis, and the
    first-order expansion of exp is accurate to second order in the logit scale."""
    X, s = ai.exact_rank(20, 28, 5, dtype="f64", seed=33)
    rng = np.random.default_rng(1)
    WQ, WK, WV = (ai.gaussian_weight(rng, 28, 10) for _ in range(3))
    U_r, X_r, _ = oracle.principal_basis(X, 5)
    Q, K, V = X @ WQ, X @ WK, X @ WV
    Kp, Vp = X_r @ WK, X_r @ WV
    assert np.abs(Q @ K.T @ V - Q @ Kp.T @ Vp).max() < 1e-10 * np.abs(Q @ K.T @ V).max()
    errs = []
    for eps in (1e-2, 1e-3):
        q = eps * Q[3] / np.abs(Q[3] @ K.T).max()
        full = np.exp(q @ K.T) @ V
        lin = (np.ones(20) @ U_r + q @ Kp.T) @ Vp           # (1.U + q K'^T) V'
        errs.append(np.abs(full - lin).max())
    assert errs[1] < errs[0] * 2e-2                        # ~100x smaller for 10x smaller logits


# ------------------------------------------------------------------ low-rank linear, norm
def test_lowrank_linear_pins():
    rng = np.random.default_rng(12)
    L, d, dout, r = 18, 22, 14, 6
    X = rng.standard_normal((L, d))
    W = ai.gaussian_weight(rng, d, dout); Wg = ai.gaussian_weight(rng, d, dout)
    b = rng.standard_normal(dout)
    assert np.abs(oracle.lowrank_linear(np.eye(L), X, W) - X @ W).max() < 1e-13     # U = I
    U_r, X_r, _ = oracle.principal_basis(X, r)
    Y = oracle.lowrank_linear(U_r, X_r, W)
    assert np.abs(Y - (U_r @ U_r.T @ X) @ W).max() < 1e-12                          # projector form
    Xe, _ = ai.exact_rank(L, d, 4, dtype="f64", seed=5)
    Ue, Xre, _ = oracle.principal_basis(Xe, 4)
    assert np.abs(oracle.lowrank_linear(Ue, Xre, W, bias=b) - (Xe @ W + b)).max() < 1e-12
    # GELU (erf form): known values and against the error function directly
    Z = U_r @ X_r @ W + b
    Yg = oracle.lowrank_linear(U_r, X_r, W, bias=b, act="gelu")
    from scipy.special import erf
    assert np.abs(Yg - 0.5 * Z * (1 + erf(Z / math.sqrt(2)))).max() < 1e-13
    one = oracle.lowrank_linear(np.eye(1), np.array([[1.0]]), np.array([[1.0]]), act="gelu")
    assert abs(one[0, 0] - 0.8413447460685429) < 1e-15          # Phi(1)
    # SwiGLU
    Ys = oracle.lowrank_linear(U_r, X_r, W, W_gate=Wg, act="swiglu")
    Gt = U_r @ X_r @ Wg
    assert np.abs(Ys - Gt / (1 + np.exp(-Gt)) * (U_r @ X_r @ W)).max() < 1e-13
    with pytest.raises(ValueError):
        oracle.lowrank_linear(U_r, X_r, W, act="swiglu")


def test_norm_pins():
    rng = np.random.default_rng(13)
    X = rng.standard_normal((5, 16)) * 3 + 1
    R = rng.standard_normal((5, 16))
    Y = oracle.norm(X, kind="rms", eps=0.0)
    assert np.allclose((Y ** 2).mean(axis=1), 1.0, atol=1e-13)
    assert np.allclose(Y * np.sqrt((X ** 2).mean(1, keepdims=True)), X, atol=1e-13)
    Yl = oracle.norm(X, residual=R, kind="layer", eps=0.0)
    assert np.allclose(Yl.mean(axis=1), 0.0, atol=1e-13) and np.allclose(Yl.var(axis=1), 1.0, atol=1e-12)
    Z = X + R
    assert np.allclose(Yl, (Z - Z.mean(1, keepdims=True)) / Z.std(1, keepdims=True), atol=1e-12)
    Ye = oracle.norm(np.zeros((1, 4)), kind="rms", eps=1e-5)
    assert np.all(Ye == 0)


# ------------------------------------------------------------------ Algorithm 1, Eq. 4
def test_alternating_svd_pins():
    rng = np.random.default_rng(14)
    a = rng.standard_normal(9); b = rng.standard_normal(12)
    U, Xp = oracle.alternating_svd(np.outer(a, b), 1, rng.standard_normal((1, 12)), inner=2)
    assert np.allclose(np.abs(U[:, 0]), np.abs(a) / np.linalg.norm(a), atol=1e-13)   # rank one: exact
    assert np.allclose(U @ Xp, np.outer(a, b), atol=1e-12)
    # well separated spectrum and many inner rounds: converges to the SVD (sigma fused into v)
    X, s = ai.planted_matrix(rng, 20, 30, [100.0, 10.0, 1.0], 0.0, frob2=10101.0)
    U, Xp = oracle.alternating_svd(X, 3, rng.standard_normal((3, 30)), inner=40)
    assert np.allclose(np.linalg.norm(Xp, axis=1), s, rtol=1e-9)
    assert np.abs(U.T @ U - np.eye(3)).max() < 1e-8
    # two rounds (the paper's setting): residual never increases as components are added
    Xn = X + 0.1 * rng.standard_normal(X.shape)
    v0 = rng.standard_normal((6, 30))
    res = [np.linalg.norm(Xn - np.matmul(*oracle.alternating_svd(Xn, k, v0[:k], inner=2))) for k in range(1, 7)]
    assert all(res[i + 1] <= res[i] + 1e-12 for i in range(5))
    assert res[-1] >= math.sqrt((np.linalg.svd(Xn, compute_uv=False)[6:] ** 2).sum()) - 1e-12   # Eckart-Young bound


def test_svd_entropy_pins():
    assert abs(oracle.svd_entropy(np.ones(8)) - 3.0) < 1e-14      # n equal values: log2 n
    assert abs(oracle.svd_entropy(np.array([5.0, 0, 0]))) < 1e-14
    s = np.array([3.0, 1.0])
    assert abs(oracle.svd_entropy(s) + math.log2((9 + 1) / 16.0)) < 1e-14


# ------------------------------------------------------------------ workloads: recipe checks
def test_workload_one_matches_recipe():
    w = ai.bert_base_fp32()
    X = w.seqs[0].X
    assert X.shape == (512, 768) and w.heads == 12 and w.seqs[0].r == 128
    assert np.all(X == X.astype(np.float32).astype(np.float64))
    sv = np.linalg.svd(X, compute_uv=False)
    assert sv[0] > 1000 * sv[40] and sv[40] < 0.6       # steep planted part, then the 0.01*N noise bulk
    assert set(w.weights) == {"W_Q", "W_K", "W_V", "W_O"}
    assert abs(w.weights["W_Q"].var() * 768 - 1.0) < 0.02


def test_bf16_rounding_is_exact_and_idempotent():
    rng = np.random.default_rng(0)
    a = rng.standard_normal(1000).astype(np.float32)
    b = ai.round_to_bf16(a)
    assert np.all(ai.round_to_bf16(b) == b)
    assert np.all((b.view(np.uint32) & 0xFFFF) == 0)
    assert np.abs(b - a).max() <= np.abs(a).max() * 2.0 ** -8
    import torch
    assert np.all(torch.from_numpy(a).to(torch.bfloat16).float().numpy() == b)


# ------------------------------------------------------------------ rotary positions (Sec. 4.2)
def _naive_rope(M, heads, pos, base):
    """Independent restatement: complex multiplication of consecutive coordinate pairs by e^{i pos theta_j}."""
    L, dp = M.shape
    dh = dp // heads
    out = np.empty_like(M)
    theta = base ** (-2.0 * np.arange(dh // 2) / dh)
    for h in range(heads):
        blk = M[:, h * dh:(h + 1) * dh]
        z = (blk[:, 0::2] + 1j * blk[:, 1::2]) * np.exp(1j * np.outer(pos, theta))
        out[:, h * dh + 0:(h + 1) * dh:2] = z.real
        out[:, h * dh + 1:(h + 1) * dh:2] = z.imag
    return out


def _naive_attention(Q, K, V, heads, scale):
    L, dp = Q.shape
    dh = dp // heads
    O = np.empty((L, dp))
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        S = Q[:, sl] @ K[:, sl].T * scale
        P = np.exp(S - S.max(axis=1, keepdims=True))
        P /= P.sum(axis=1, keepdims=True)
        O[:, sl] = P @ V[:, sl]
    return O


def test_attention_rope_pins():
    rng = np.random.default_rng(123)
    L, d, heads, dh = 24, 20, 2, 8
    dp = heads * dh
    X = rng.standard_normal((L, d))
    WQ, WK, WV = (rng.standard_normal((d, dp)) / math.sqrt(d) for _ in range(3))
    pos = rng.integers(0, 50, L)
    # (1) U = I, r = L: textbook rotary attention on the full keys, written independently
    I = np.eye(L)
    got = oracle.attention_rope(X, I, X, WQ, WK, WV, heads, positions=pos, rope_base=100.0)
    want = _naive_attention(_naive_rope(X @ WQ, heads, pos, 100.0), _naive_rope(X @ WK, heads, pos, 100.0), X @ WV,
                            heads, 1 / math.sqrt(dh))
    assert np.abs(got - want).max() < 1e-12
    # (2) with U = I the result depends on relative positions only: a common shift changes nothing
    got2 = oracle.attention_rope(X, I, X, WQ, WK, WV, heads, positions=pos + 17, rope_base=100.0)
    assert np.abs(got2 - got).max() < 1e-10
    # (3) all positions zero: no rotation, equals the plain principal-key attention for any basis
    U, Xr, _ = oracle.principal_basis(X, 6)
    a = oracle.attention_rope(X, U, Xr, WQ, WK, WV, heads, positions=np.zeros(L, dtype=int))
    b = oracle.attention(X, U, Xr, WQ, WK, WV, heads)
    assert np.abs(a - b).max() < 1e-12
    # (4) truncated basis: the principal keys are U^T applied to the rotated keys, checked by composing the pieces
    Kp = U.T @ _naive_rope(U @ (Xr @ WK), heads, np.arange(L), 10000.0)
    Qr = _naive_rope(U @ (Xr @ WQ), heads, np.arange(L), 10000.0)
    want = _naive_attention(Qr, Kp, Xr @ WV, heads, 1 / math.sqrt(dh))
    got = oracle.attention_rope(X, U, Xr, WQ, WK, WV, heads)          # default positions 0..L-1, base 10000
    assert np.abs(got - want).max() < 1e-12
    # (5) exact-query option rotates X W_Q
    got = oracle.attention_rope(X, U, Xr, WQ, WK, WV, heads, q_mode=1)
    want = _naive_attention(_naive_rope(X @ WQ, heads, np.arange(L), 10000.0), Kp, Xr @ WV, heads, 1 / math.sqrt(dh))
    assert np.abs(got - want).max() < 1e-12
    # odd head width is rejected
    with pytest.raises(ValueError):
        oracle.attention_rope(X, U, Xr, WQ[:, :6], WK[:, :6], WV[:, :6], 2)
