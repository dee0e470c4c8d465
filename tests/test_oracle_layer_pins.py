"""Pins of the oracle's layer and stack compositions (Fig. 3, Sec. 4.2 closing paragraph), CPU only.

The single stages are pinned in test_oracle_pins.py; here the order of the stages, the operands of the
residual connections, the kinds of the Norm boxes and the roles of the FeedForward weights are checked
against dense numpy formulas. At full rank r = min(L, d) every basis is exact (U_r X_r = X), so every
low-rank linear layer must equal the dense product of its input.
"""
import math

import numpy as np
import pytest

import atp_inputs as ai
import oracle


def _rms(x, eps=1e-5):
    return x / np.sqrt((x * x).mean(axis=1, keepdims=True) + eps)


def _ln(x, eps=1e-5):
    m = x.mean(axis=1, keepdims=True)
    v = ((x - m) ** 2).mean(axis=1, keepdims=True)
    return (x - m) / np.sqrt(v + eps)


def _gelu(x):
    return 0.5 * x * (1.0 + np.vectorize(math.erf)(x / math.sqrt(2.0)))


def _silu(x):
    return x / (1.0 + np.exp(-x))


def _weights(rng, d, dff, ffn):
    w = {k: rng.standard_normal((d, d)) / math.sqrt(d) for k in ("W_Q", "W_K", "W_V", "W_O")}
    if ffn == "gelu":
        w["W_1"] = rng.standard_normal((d, dff)) / math.sqrt(d)
        w["W_2"] = rng.standard_normal((dff, d)) / math.sqrt(dff)
    elif ffn == "swiglu":
        w["W_up"] = rng.standard_normal((d, dff)) / math.sqrt(d)
        w["W_gate"] = rng.standard_normal((d, dff)) / math.sqrt(d)
        w["W_down"] = rng.standard_normal((dff, d)) / math.sqrt(dff)
    return w


@pytest.mark.parametrize("ffn,input_norm,post_norm", [("gelu", None, "layer"), ("swiglu", "rms", "rms"), ("gelu", "layer", "rms")])
def test_layer_at_full_rank_is_the_dense_layer_after_attention(ffn, input_norm, post_norm):
    rng = np.random.default_rng(11)
    L, d, dff, heads = 12, 12, 12, 2          # L = d = dff: every stage's input has min(L, d) = 12 = r
    X = rng.standard_normal((L, d)) * 1.7 + 0.3
    w = _weights(rng, d, dff, ffn)
    st = {}
    Y = oracle.layer_forward(X, w, L, heads, ffn=ffn, input_norm=input_norm, post_norm=post_norm, stages=st)
    nrm = {"rms": _rms, "layer": _ln}
    Xin = nrm[input_norm](X) if input_norm else X
    assert np.allclose(st["Xin"], Xin, atol=1e-12)
    # the attention stage is pinned on its own; everything after it has a dense closed form at full rank
    A = st["O"] @ w["W_O"]
    assert np.allclose(st["A"], A, atol=1e-9)
    H = nrm[post_norm](X + A)                                  # residual from the layer input, before its Norm
    assert np.allclose(st["H"], H, atol=1e-9)
    if ffn == "gelu":
        F = _gelu(H @ w["W_1"]); Yd = F @ w["W_2"]
    else:
        F = _silu(H @ w["W_gate"]) * (H @ w["W_up"]); Yd = F @ w["W_down"]
    assert np.allclose(st["F"], F, atol=1e-9)
    assert np.allclose(Y, Yd, atol=1e-8)
    if input_norm:                                             # a residual taken after the Norm would differ
        assert not np.allclose(nrm[post_norm](Xin + A), H, atol=1e-3)


def test_layer_equals_its_pinned_stages_below_full_rank_and_short_forms():
    rng = np.random.default_rng(12)
    L, d, dff, heads, r = 20, 16, 24, 4, 5
    X, _ = ai.planted_matrix(rng, L, d, 0.6 ** np.arange(8), 0.05)
    w = _weights(rng, d, dff, "swiglu")
    st = {}
    Y = oracle.layer_forward(X, w, r, heads, ffn="swiglu", input_norm="rms", post_norm="rms", stages=st)
    Xin = oracle.norm(X, kind="rms")
    U, Xr, _ = oracle.principal_basis(Xin, r)
    O = oracle.attention(Xin, U, Xr, w["W_Q"], w["W_K"], w["W_V"], heads)
    assert np.array_equal(st["O"], O)
    Uo, Or, _ = oracle.principal_basis(O, r)
    A = oracle.lowrank_linear(Uo, Or, w["W_O"])
    H = oracle.norm(X, residual=A, kind="rms")
    Uh, Hr, _ = oracle.principal_basis(H, r)
    F = oracle.lowrank_linear(Uh, Hr, w["W_up"], W_gate=w["W_gate"], act="swiglu")
    Uf, Fr, _ = oracle.principal_basis(F, r)
    assert np.array_equal(Y, oracle.lowrank_linear(Uf, Fr, w["W_down"]))
    # the low-rank linear layers see the projector of their own input: A = (Uo Uo^T O) W_O, F from (Uh Uh^T H)
    assert np.allclose(A, (Uo @ (Uo.T @ O)) @ w["W_O"], atol=1e-10)
    Hp = Uh @ (Uh.T @ H)
    assert np.allclose(F, _silu(Hp @ w["W_gate"]) * (Hp @ w["W_up"]), atol=1e-10)
    # short forms: without W_O the layer returns O, without a FeedForward it returns A
    wq = {k: w[k] for k in ("W_Q", "W_K", "W_V")}
    assert np.array_equal(oracle.layer_forward(X, wq, r, heads, input_norm="rms"), O)
    wo = dict(wq, W_O=w["W_O"])
    assert np.array_equal(oracle.layer_forward(X, wo, r, heads, input_norm="rms"), A)


def test_stack_closes_the_block_and_chains_layers():
    rng = np.random.default_rng(13)
    L, d, dff, heads, r = 18, 12, 16, 2, 6
    X, _ = ai.planted_matrix(rng, L, d, 0.7 ** np.arange(6), 0.05)
    ws = [_weights(rng, d, dff, "gelu"), _weights(rng, d, dff, "gelu")]
    st1 = {}
    y1 = oracle.layer_forward(X, ws[0], r, heads, ffn="gelu", post_norm="layer", stages=st1)
    x1 = _ln(st1["H"] + y1)                                    # X_{l+1} = Norm(H_l + Y_l)
    one = oracle.stack_forward(X, ws[:1], r, heads, ffn="gelu", post_norm="layer")
    assert np.allclose(one, x1, atol=1e-10)
    st2 = {}
    y2 = oracle.layer_forward(x1, ws[1], r, heads, ffn="gelu", post_norm="layer", stages=st2)
    x2 = _ln(st2["H"] + y2)
    log = []
    two = oracle.stack_forward(X, ws, r, heads, ffn="gelu", post_norm="layer", stages=log)
    assert np.allclose(two, x2, atol=1e-9)
    assert len(log) == 2 and np.allclose(log[0]["X_next"], x1, atol=1e-10)
    # the second layer's basis is taken of the first layer's closed output, not of the raw input
    assert not np.allclose(log[1]["Xin"], X, atol=1e-3)
    # layers without a FeedForward hand their output on unchanged
    wo = [{k: w[k] for k in ("W_Q", "W_K", "W_V", "W_O")} for w in ws]
    a1 = oracle.layer_forward(X, wo[0], r, heads)
    a2 = oracle.layer_forward(a1, wo[1], r, heads)
    assert np.allclose(oracle.stack_forward(X, wo, r, heads), a2, atol=1e-12)


def test_capped_jacobi_runs_the_rounds_it_is_given_and_projection_helper():
    rng = np.random.default_rng(14)
    X = rng.standard_normal((30, 22))
    assert oracle.svd_jacobi_capped(X, 5) == 5                 # 21 rounds per sweep: stops inside the first
    full_rounds = oracle.svd_jacobi_capped(X, 10 ** 6)         # converges long before the cap
    sweeps = oracle.svd_jacobi(X)[3]
    assert full_rounds == sweeps * 21
    U, Xr, _ = oracle.principal_basis(X, 7)
    assert np.allclose(oracle.project_rows(X, U), U.T @ X, atol=1e-13)
    assert np.allclose(oracle.project_rows(X, U, 3), (U.T @ X)[:3], atol=1e-13)
