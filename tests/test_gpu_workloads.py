"""Parity on the five workloads (shapes, value distributions and layer composition of the
benchmark), through the same AtpLayer driver and launch configuration bench.py times.

Small and medium cases are compared element by element; at full size the oracle evaluates
sampled heads / output columns one by one (heads and output columns are independent, so slicing
the weights is exact), on the basis the GPU produced (stage parity).
"""
import math

import numpy as np
import pytest

import atp_inputs as ai
import oracle
from gpu_util import TOL, basis_invariants, rel_err, residual_ok, to_dev, to_np

pytestmark = pytest.mark.gpu
POST_NORM = {"gelu": "layer", "swiglu": "rms", None: "layer"}


@pytest.fixture(scope="module")
def ctx():
    import paper_2403_02352_b200 as atp
    c = atp.Context(0)
    yield c
    c.close()


def _layer(ctx, w, **kw):
    from paper_2403_02352_b200.layer import AtpLayer
    weights = {k: to_dev(v, w.dtype) for k, v in w.weights.items()}
    return AtpLayer(ctx, weights, w.lengths, w.ranks, w.heads, ffn=w.ffn, input_norm=w.input_norm,
                    post_norm=POST_NORM[w.ffn], **kw)


def _split(t, offs, b):
    return to_np(t[offs[b]:offs[b + 1]])


def _check_basis(stage, X, basis, ro, ko, b, r, dtype, ratio_tol=5e-2):
    U = to_np(basis[0][ro[b]:ro[b + 1]])[:, :r]
    Xr = to_np(basis[1][ko[b]:ko[b + 1]])
    sig = to_np(basis[2][ko[b]:ko[b + 1]].reshape(-1, 1)).ravel()
    inv = basis_invariants(X, U, Xr, sig)
    inv.pop("s_true"); inv.pop("sigma_rel")
    assert inv["orth"] <= (2e-2 if dtype == "bf16" else 2e-4), (stage, inv)
    assert residual_ok(inv["res_sub"], inv["opt"], inv["normX"], dtype, ratio_tol), (stage, inv)
    assert inv["offdiag"] <= (5e-2 if dtype == "bf16" else 1e-4), (stage, inv)
    assert inv["xr_vs_utx"] <= 8 * (2.0 ** -8 if dtype == "bf16" else 2.0 ** -23), (stage, inv)
    assert inv["sorted"], (stage, inv)
    return U, Xr


def _stage_parity_full_layer(ctx, w, sample_heads=None, sample_cols=None, sample_seqs=None):
    """Runs the layer on the GPU and checks every stage against the oracle evaluated on the GPU's
    own inputs to that stage (basis invariants for the bases, T2 for attention and linear layers).
    The GPU always runs the whole batch at full size; sample_heads / sample_cols / sample_seqs bound what the
    CPU oracle re-computes (heads, output columns and sequences are independent, so slicing is exact)."""
    layer = _layer(ctx, w)
    Xp, row_off, rank, rank_off = ai.pack(w.seqs)
    Xd = to_dev(Xp, w.dtype)
    layer.forward(Xd)
    ctx.poll()
    _check_layer_stages(layer, w, Xd, sample_heads, sample_cols, sample_seqs)
    return layer


def _check_layer_stages(layer, w, Xd, sample_heads=None, sample_cols=None, sample_seqs=None):
    row_off = np.concatenate([[0], np.cumsum(w.lengths)]).astype(int)
    rank_off = np.concatenate([[0], np.cumsum(w.ranks)]).astype(int)
    for t in (layer.O, layer.bX[0], layer.bX[1]):
        assert bool(np.isfinite(to_np(t[:8])).all())
    dt, tol = w.dtype, TOL[w.dtype]
    W = w.weights
    heads, dh = w.heads, W["W_Q"].shape[1] // w.heads
    hs = list(range(heads)) if sample_heads is None else sample_heads
    cols = slice(None) if sample_cols is None else sample_cols
    for b, s in enumerate(w.seqs):
        if sample_seqs is not None and b not in sample_seqs:
            continue
        r = s.r
        Xin = _split(layer.Xn if w.input_norm else Xd, row_off, b)
        Xraw = _split(Xd, row_off, b)
        if w.input_norm:
            assert rel_err(Xin, oracle.norm(Xraw, kind=w.input_norm)) <= (1e-5 if dt == "f32" else 8e-3)
        U, Xr = _check_basis("X", Xin, layer.bX, row_off, rank_off, b, r, dt)
        O = _split(layer.O, row_off, b)
        for h in hs:
            sl = slice(h * dh, (h + 1) * dh)
            ref = oracle.attention(None, U, Xr, W["W_Q"][:, sl], W["W_K"][:, sl], W["W_V"][:, sl], 1)
            assert rel_err(O[:, sl], ref) <= tol, (b, h)
        if "W_O" not in W:
            continue
        Uo, Or = _check_basis("O", O, layer.bO, row_off, rank_off, b, r, dt)
        A = _split(layer.A, row_off, b)
        assert rel_err(A[:, cols], oracle.lowrank_linear(Uo, Or, W["W_O"][:, cols])) <= tol
        if not w.ffn:
            continue
        H = _split(layer.H, row_off, b)
        assert rel_err(H, oracle.norm(Xraw, residual=A, kind=POST_NORM[w.ffn])) <= (1e-5 if dt == "f32" else 1.6e-2)
        Uh, Hr = _check_basis("H", H, layer.bH, row_off, rank_off, b, r, dt)
        F = _split(layer.F, row_off, b)
        if w.ffn == "gelu":
            assert rel_err(F[:, cols], oracle.lowrank_linear(Uh, Hr, W["W_1"][:, cols], act="gelu")) <= tol
            Wd = W["W_2"]
        else:
            assert rel_err(F[:, cols], oracle.lowrank_linear(Uh, Hr, W["W_up"][:, cols], W_gate=W["W_gate"][:, cols],
                                                             act="swiglu")) <= tol
            Wd = W["W_down"]
        Uf, Fr = _check_basis("F", F, layer.bF, row_off, rank_off, b, r, dt)
        Y = _split(layer.Y, row_off, b)
        assert rel_err(Y[:, cols], oracle.lowrank_linear(Uf, Fr, Wd[:, cols])) <= tol


def test_workload1_bert_base_fp32_full_size(ctx):
    _stage_parity_full_layer(ctx, ai.bert_base_fp32())


@pytest.mark.parametrize("r", [256, 128])
def test_workload2_bert_large_bf16_two_sequences_full_size(ctx, r):
    w = ai.bert_large_bf16(batch=2, r=r)
    _stage_parity_full_layer(ctx, w, sample_heads=[0, 7, 15], sample_cols=slice(0, 192))


def test_workload2_bert_large_bf16_full_batch_of_16(ctx):
    w = ai.bert_large_bf16(batch=16, r=256)
    _stage_parity_full_layer(ctx, w, sample_heads=[2, 11], sample_cols=slice(320, 448), sample_seqs=[0, 9, 15])


def test_workload3_llama_like_reduced(ctx):
    w = ai.llama7b_bf16(L=512, d=512, heads=4, r=128, k=48, d_ff=1376)
    _stage_parity_full_layer(ctx, w)


def test_workload3_llama7b_full_size_sampled(ctx):
    w = ai.llama7b_bf16(r=1024)
    _stage_parity_full_layer(ctx, w, sample_heads=[0, 17], sample_cols=slice(64, 192))


def test_workload3_llama7b_full_size_rank_2048_sampled(ctx):
    w = ai.llama7b_bf16(r=2048)                       # the configuration bench.py times by default
    _stage_parity_full_layer(ctx, w, sample_heads=[5, 28], sample_cols=slice(1024, 1152))


@pytest.mark.parametrize("L", [16384, 32768])
def test_workload4_long_context_sampled(ctx, L):
    w = ai.long_context_bf16(L=L, r=1024)
    import paper_2403_02352_b200 as atp
    s = w.seqs[0]
    d, r = w.d, 1024
    Xd = to_dev(s.X, "bf16")
    U, Xr, sig = atp.atp_principal_basis(ctx, Xd, [L], [r])
    Wd = {k: to_dev(v, "bf16") for k, v in w.weights.items()}
    O = atp.atp_attention(ctx, Xd, U, Xr, Wd["W_Q"], Wd["W_K"], Wd["W_V"], w.heads, [L], [r])
    ctx.poll()
    Un, Xrn, sn = to_np(U), to_np(Xr), to_np(sig.reshape(-1, 1)).ravel()
    # properties that hold at any size (the d x d Gram matrix gives the exact spectrum)
    ev = np.linalg.eigvalsh(s.X.T @ s.X)[::-1]
    sv = np.sqrt(np.maximum(ev, 0))
    assert np.abs(Un.T @ Un - np.eye(r)).max() <= 2e-2
    Qu, _ = np.linalg.qr(Un)
    res = math.sqrt(max((sv ** 2).sum() - np.linalg.norm(Qu.T @ s.X) ** 2, 0.0))
    assert residual_ok(res, math.sqrt((sv[r:] ** 2).sum()), np.linalg.norm(s.X), "bf16", 5e-2)
    assert np.all(np.diff(sn) <= 1e-6 * sv[0])
    assert np.abs(sn[:64] - sv[:64]).max() <= 1e-2 * sv[0]
    dh = d // w.heads
    rows = np.r_[0:64, L // 2 - 192:L // 2 - 128, L - 64:L]
    On = to_np(O)
    for h in (0, 31):
        sl = slice(h * dh, (h + 1) * dh)
        ref = oracle.attention(None, Un[rows], Xrn, w.weights["W_Q"][:, sl], w.weights["W_K"][:, sl], w.weights["W_V"][:, sl], 1)
        assert rel_err(On[rows][:, sl], ref) <= TOL["bf16"]


def test_workload5_serving_batch_ragged(ctx):
    w = ai.serving_batch_bf16(batch=8, L=1024)
    assert len(set(w.lengths)) > 1 and any(r % 8 for r in w.ranks)      # ragged lengths, unaligned ranks
    _stage_parity_full_layer(ctx, w, sample_heads=[3, 30])


def test_workload5_serving_batch_of_32_at_2048(ctx):
    w = ai.serving_batch_bf16(batch=32, L=2048)                          # every launch carries 32 sequences
    assert max(w.lengths) > 1024 and min(w.lengths) >= 1024
    _stage_parity_full_layer(ctx, w, sample_heads=[12], sample_seqs=[0, 17, 31])


def test_workload5_serving_single_sequence_at_2048(ctx):
    w = ai.serving_batch_bf16(batch=1, L=2048)
    _stage_parity_full_layer(ctx, w, sample_heads=[7, 25])
