"""ctypes front end of the CPU oracle (oracle/atp_oracle.c).

Test infrastructure only: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg. The CUDA library never imports or calls it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "atp_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) into oracle/liboracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-fvisibility=hidden",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_svd_entropy.restype = ctypes.c_double
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _c(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def svd_jacobi(X):
    """Eq. 3: X = U diag(S) Vt by one-sided Jacobi. Returns (U, S, Vt, sweeps)."""
    X = _c(X)
    L, d = X.shape
    n = min(L, d)
    U = np.empty((L, n)); S = np.empty(n); Vt = np.empty((n, d))
    sweeps = _load().oracle_svd_jacobi(_p(X), L, d, _p(U), _p(S), _p(Vt))
    return U, S, Vt, int(sweeps)


def svd_jacobi_capped(X, max_rounds):
    """The same Jacobi iteration stopped after `max_rounds` rounds (a round rotates n/2 disjoint pairs, a sweep
    is n-1 rounds): for timing a bounded part of a large decomposition. Returns the number of rounds run; the
    unfinished factors are discarded."""
    X = _c(X)
    L, d = X.shape
    n = min(L, d)
    U = np.empty((L, n)); S = np.empty(n); Vt = np.empty((n, d))
    done = ctypes.c_long(0)
    _load().oracle_svd_jacobi_capped(_p(X), L, d, _p(U), _p(S), _p(Vt), ctypes.c_long(int(max_rounds)), ctypes.byref(done))
    return int(done.value)


def project_rows(X, U_r, nrows=None):
    """Leading `nrows` rows of X_r = U_r^T X (all r by default)."""
    X = _c(X); U_r = _c(U_r)
    L, d = X.shape
    r = U_r.shape[1]
    nrows = r if nrows is None else int(nrows)
    X_r = np.empty((nrows, d))
    _load().oracle_project_rows(_p(X), _p(U_r), L, d, r, nrows, _p(X_r))
    return X_r


def principal_basis(X, r, return_all_sigma=False):
    """Eq. 5 / Sec. 4.2: (U_r, X_r, sigma) of the exact truncated SVD, canonical signs."""
    X = _c(X)
    L, d = X.shape
    U_r = np.empty((L, r)); X_r = np.empty((r, d)); sig = np.empty(r)
    sall = np.empty(min(L, d))
    rc = _load().oracle_principal_basis(_p(X), L, d, int(r), _p(U_r), _p(X_r), _p(sig), _p(sall))
    if rc < 0:
        raise ValueError("invalid rank")
    return (U_r, X_r, sig, sall) if return_all_sigma else (U_r, X_r, sig)


def attention(X, U_r, X_r, W_Q, W_K, W_V, heads, q_mode=0, scale=0.0):
    """Eq. 6 + attention on r principal keys (Eq. 1 with K', V')."""
    U_r = _c(U_r); X_r = _c(X_r); W_Q = _c(W_Q); W_K = _c(W_K); W_V = _c(W_V); X = _c(X)
    L, r = U_r.shape
    d = X_r.shape[1]
    dp = W_Q.shape[1]
    O = np.empty((L, dp))
    rc = _load().oracle_attention(_p(X), _p(U_r), _p(X_r), _p(W_Q), _p(W_K), _p(W_V),
                                  L, d, dp, r, int(heads), int(q_mode), ctypes.c_double(scale), _p(O))
    if rc < 0:
        raise ValueError("invalid attention arguments")
    return O


def attention_rope(X, U_r, X_r, W_Q, W_K, W_V, heads, positions=None, rope_base=10000.0, q_mode=0, scale=0.0):
    """Attention on principal keys with rotary positions (Sec. 4.2): K = U_r K' rotated row by row,
    K'_rot = U_r^T K_rot are the principal keys; queries rotated; positions default to 0..L-1."""
    U_r = _c(U_r); X_r = _c(X_r); W_Q = _c(W_Q); W_K = _c(W_K); W_V = _c(W_V); X = _c(X)
    L, r = U_r.shape
    d = X_r.shape[1]
    dp = W_Q.shape[1]
    O = np.empty((L, dp))
    pos = None if positions is None else np.ascontiguousarray(positions, dtype=np.int32)
    rc = _load().oracle_attention_rope(_p(X), _p(U_r), _p(X_r), _p(W_Q), _p(W_K), _p(W_V),
                                       L, d, dp, r, int(heads), int(q_mode), ctypes.c_double(scale),
                                       None if pos is None else pos.ctypes.data_as(ctypes.c_void_p),
                                       ctypes.c_double(rope_base), _p(O))
    if rc < 0:
        raise ValueError("invalid attention arguments")
    return O


ACT = {None: 0, "none": 0, "gelu": 1, "swiglu": 2}


def lowrank_linear(U_r, X_r, W, bias=None, W_gate=None, act=None):
    """Y = act(U_r (X_r W) + bias); SwiGLU gates with silu(U_r X_r W_gate)."""
    U_r = _c(U_r); X_r = _c(X_r); W = _c(W); bias = _c(bias); W_gate = _c(W_gate)
    L, r = U_r.shape
    d_in, d_out = W.shape
    Y = np.empty((L, d_out))
    rc = _load().oracle_lowrank_linear(_p(U_r), _p(X_r), _p(W), _p(bias), _p(W_gate), ACT[act],
                                       L, r, d_in, d_out, _p(Y))
    if rc < 0:
        raise ValueError("invalid linear arguments")
    return Y


def norm(X, residual=None, kind="rms", eps=1e-5):
    """Norm box of Fig. 3 (unit gain), optional residual added first."""
    X = _c(X); residual = _c(residual)
    L, d = X.shape
    Y = np.empty((L, d))
    _load().oracle_norm(_p(X), _p(residual), 0 if kind == "rms" else 1, ctypes.c_double(eps), L, d, _p(Y))
    return Y


def alternating_svd(X, r, v0, inner=2):
    """Algorithm 1: rank-1 alternating fits with deflation. Returns (U, Xp)."""
    X = _c(X); v0 = _c(v0)
    L, d = X.shape
    U = np.empty((L, r)); Xp = np.empty((r, d))
    _load().oracle_alternating_svd(_p(X), L, d, int(r), _p(v0), int(inner), _p(U), _p(Xp))
    return U, Xp


def svd_entropy(sigma) -> float:
    """Eq. 4 with log base 2."""
    sigma = _c(sigma)
    return float(_load().oracle_svd_entropy(_p(sigma), sigma.shape[0]))


def layer_forward(X, weights, r, heads, ffn=None, input_norm=None, post_norm="layer", stages=None):
    """One ATP layer (Fig. 3) for a single sequence, composed from the functions above: Norm,
    basis, attention on r principal keys, then output projection and FeedForward, each linear layer
    applied to the principal basis of its own input (same r). `stages` (a dict) receives the
    intermediate results when given. Returns the layer output."""
    st = {} if stages is None else stages
    Xin = norm(X, kind=input_norm) if input_norm else np.asarray(X, dtype=np.float64)
    U, Xr, _ = principal_basis(Xin, r)
    O = attention(Xin, U, Xr, weights["W_Q"], weights["W_K"], weights["W_V"], heads)
    st.update(Xin=Xin, U=U, Xr=Xr, O=O)
    if "W_O" not in weights:
        return O
    Uo, Or, _ = principal_basis(O, r)
    A = lowrank_linear(Uo, Or, weights["W_O"])
    st.update(A=A)
    if not ffn:
        return A
    H = norm(X, residual=A, kind=post_norm)
    Uh, Hr, _ = principal_basis(H, r)
    if ffn == "gelu":
        F = lowrank_linear(Uh, Hr, weights["W_1"], act="gelu")
        Uf, Fr, _ = principal_basis(F, r)
        Y = lowrank_linear(Uf, Fr, weights["W_2"])
    else:
        F = lowrank_linear(Uh, Hr, weights["W_up"], W_gate=weights["W_gate"], act="swiglu")
        Uf, Fr, _ = principal_basis(F, r)
        Y = lowrank_linear(Uf, Fr, weights["W_down"])
    st.update(H=H, F=F, Y=Y)
    return Y


def stack_forward(X, layer_weights, r, heads, ffn=None, input_norm=None, post_norm="layer", stages=None):
    """A chain of ATP layers for a single sequence (Sec. 4.2: the next encoder/decoder layer follows the same
    procedure and first attains the principal components of the previous layer's output; Fig. 3). Layer l maps
    X_l to Y_l = FFN(H_l), H_l = Norm(X_l + A_l) (layer_forward); the block is closed the post-norm way,
    X_{l+1} = Norm(H_l + Y_l). Layers without a FeedForward pass their output on unchanged. `stages` (a list)
    receives one dict of intermediates per layer. Returns the input of the layer after the last one."""
    x = np.asarray(X, dtype=np.float64)
    for wts in layer_weights:
        st = {}
        y = layer_forward(x, wts, r, heads, ffn=ffn, input_norm=input_norm, post_norm=post_norm, stages=st)
        x = norm(st["H"], residual=y, kind=post_norm) if ffn else y
        if stages is not None:
            st["X_next"] = x
            stages.append(st)
    return x
