"""Helpers shared by the GPU parity tests: tensor conversion, error metric, basis invariants."""
import math

import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2}          # max relative error bars for O and Y (max|G-R| / max|R|)


def tdtype(dtype):
    return torch.float32 if dtype == "f32" else torch.bfloat16


def to_dev(a, dtype, ld_multiple=8):
    """numpy (float64 holding values of `dtype`) -> CUDA tensor; rows padded so that ld % 8 == 0."""
    a = np.asarray(a, dtype=np.float64)
    rows, cols = a.shape
    ld = (cols + ld_multiple - 1) // ld_multiple * ld_multiple
    t = torch.zeros((rows, ld), dtype=tdtype(dtype), device="cuda")
    t[:, :cols] = torch.from_numpy(a).to(tdtype(dtype))
    return t[:, :cols]


def to_np(t):
    return t.detach().float().cpu().double().numpy()


def rel_err(G, R):
    den = np.abs(R).max()
    return float(np.abs(G - R).max() / (den if den > 0 else 1.0))


ORACLE_SVD_LIMIT = 512 * 1024      # entries: above this the oracle's Jacobi SVD takes minutes


def spectrum(X):
    """All singular values of X: from the oracle's own Jacobi SVD where that is affordable (up to 512 x 1024,
    i.e. workloads 1 and 2 and every small case), from LAPACK above that size (the oracle is pinned to LAPACK
    to 1e-12 on CPU, so the two agree; the larger workloads could not be checked at all otherwise)."""
    X = np.asarray(X, dtype=np.float64)
    if X.size <= ORACLE_SVD_LIMIT:
        import oracle
        return oracle.svd_jacobi(X)[1]
    return np.linalg.svd(X, compute_uv=False)


def basis_invariants(X, U, Xr, sig):
    """T1 quantities of one sequence (all float64 numpy)."""
    r = U.shape[1]
    s_true = spectrum(X)
    out = {}
    out["orth"] = float(np.abs(U.T @ U - np.eye(r)).max())
    out["xr_vs_utx"] = float(np.abs(Xr - U.T @ X).max() / s_true[0])
    # quality of the subspace alone: project X on an exactly orthonormalised copy of U
    Qu, _ = np.linalg.qr(U)
    res_sub = math.sqrt(max(np.linalg.norm(X) ** 2 - np.linalg.norm(Qu.T @ X) ** 2, 0.0))
    opt = math.sqrt(float((s_true[r:] ** 2).sum()))
    out["opt"] = opt
    out["res_sub"] = res_sub
    out["res_ratio"] = res_sub / opt if opt > 1e-12 * s_true[0] else 1.0 + res_sub / s_true[0]
    out["normX"] = float(np.linalg.norm(X))
    out["res_pair"] = float(np.linalg.norm(X - U @ Xr))
    G = Xr @ Xr.T
    dg = np.sqrt(np.maximum(np.diag(G), 0))
    den = np.outer(dg, dg)
    den[den < (1e-12 * s_true[0]) ** 2] = np.inf
    off = np.abs(G - np.diag(np.diag(G))) / den
    out["offdiag"] = float(off.max())
    out["energy_rel"] = float(abs(np.linalg.norm(Xr) ** 2 - (s_true[:r] ** 2).sum()) / (s_true ** 2).sum())
    rn = np.linalg.norm(Xr, axis=1)
    out["sigma_vs_rows"] = float(np.abs(sig - rn).max() / s_true[0])
    out["sorted"] = bool(np.all(np.diff(sig) <= 1e-6 * s_true[0]))
    out["sigma_rel"] = np.abs(sig - s_true[:r]) / s_true[0]
    out["s_true"] = s_true
    return out


def residual_ok(res_sub, opt, norm_x, dtype, tol):
    """Subspace residual against the Eckart-Young optimum. The range finder reaches (1 + tol) * opt;
    a basis stored in bf16 additionally tilts every direction by its entry rounding (relative
    2^-9), which costs up to (2^-9 |X|_F)^2 of captured energy whatever the algorithm."""
    eps = 2.0 ** -9 if dtype == "bf16" else 2.0 ** -22
    return res_sub ** 2 <= ((1.0 + tol) * opt) ** 2 + (eps * norm_x) ** 2
