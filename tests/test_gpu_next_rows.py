"""GPU parity of the two widened rows: Algorithm 1 (alternating rank-1 fits with deflation) and the
SVD entropy of Eq. 4, each against its oracle on the same seeded inputs (start vectors included)."""
import math

import numpy as np
import pytest
import torch

import atp_inputs as ai
import oracle
from gpu_util import TOL, rel_err, to_dev, to_np

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


def _planted(rng, L, d, k, dtype, noise=0.02):
    x, _ = ai.planted_matrix(rng, L, d, 0.85 ** np.arange(k), noise)
    return ai.finish(x, dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,d,r,inner", [(300, 200, 24, 2), (130, 513, 17, 2), (96, 64, 8, 5)])
def test_alternating_basis_vs_oracle(ctx, dtype, L, d, r, inner):
    rng = np.random.default_rng(40 + L + r)
    X = _planted(rng, L, d, 12, dtype)
    V0 = rng.standard_normal((r, d)).astype(np.float32).astype(np.float64)     # fp32-representable
    Uo, Xo = oracle.alternating_svd(X, r, V0, inner=inner)
    U, Xr = _atp().atp_alternating_basis(ctx, to_dev(X, dtype), to_dev(V0, "f32"), [L], [r], inner=inner)
    ctx.poll()
    # the reconstruction U X' is what the later stages consume; U and X' themselves are compared too
    assert rel_err(to_np(U) @ to_np(Xr), Uo @ Xo) <= TOL[dtype]
    assert rel_err(to_np(U), Uo) <= TOL[dtype] * (1 if dtype == "f32" else 2)
    assert rel_err(to_np(Xr), Xo) <= TOL[dtype]


def test_alternating_basis_ragged_batch_and_properties(ctx):
    rng = np.random.default_rng(77)
    lengths, ranks, d = [70, 0, 129, 33], [9, 0, 20, 4], 96
    Xs = [_planted(rng, L, d, 6, "f32") if L else np.zeros((0, d)) for L in lengths]
    V0 = rng.standard_normal((sum(ranks), d)).astype(np.float32).astype(np.float64)
    U, Xr = _atp().atp_alternating_basis(ctx, to_dev(np.concatenate(Xs), "f32"), to_dev(V0, "f32"), lengths, ranks)
    ctx.poll()
    U, Xr = to_np(U), to_np(Xr)
    ro = np.concatenate([[0], np.cumsum(lengths)]); ko = np.concatenate([[0], np.cumsum(ranks)])
    for b, (L, r) in enumerate(zip(lengths, ranks)):
        if L == 0:
            continue
        Uo, Xo = oracle.alternating_svd(Xs[b], r, V0[ko[b]:ko[b + 1]], inner=2)
        assert rel_err(U[ro[b]:ro[b + 1], :r], Uo) <= 1e-4
        assert rel_err(Xr[ko[b]:ko[b + 1]], Xo) <= 1e-4
        # columns of U have unit norm; the residual does not grow with the number of components
        assert np.abs(np.linalg.norm(U[ro[b]:ro[b + 1], :r], axis=0) - 1).max() < 1e-5
        res = [np.linalg.norm(Xs[b] - U[ro[b]:ro[b + 1], :k] @ Xr[ko[b]:ko[b] + k]) for k in range(1, r + 1)]
        assert all(res[i + 1] <= res[i] * (1 + 1e-6) for i in range(len(res) - 1))


def test_alternating_basis_rank_one_is_exact(ctx):
    rng = np.random.default_rng(5)
    a, b = rng.standard_normal(60), rng.standard_normal(40)
    X = ai.finish(np.outer(a, b), "f32")
    V0 = rng.standard_normal((1, 40)).astype(np.float32).astype(np.float64)
    U, Xr = _atp().atp_alternating_basis(ctx, to_dev(X, "f32"), to_dev(V0, "f32"), [60], [1])
    ctx.poll()
    assert rel_err(to_np(U) @ to_np(Xr), X) <= 1e-5


def test_svd_entropy_vs_oracle(ctx):
    rng = np.random.default_rng(9)
    groups = [np.ones(8), np.array([5.0, 0.0, 0.0]), 0.9 ** np.arange(300), rng.random(1000) + 0.01, np.zeros(4), np.zeros(0)]
    groups = [g.astype(np.float32).astype(np.float64) for g in groups]
    sigma = torch.from_numpy(np.concatenate(groups).astype(np.float32)).cuda()
    mu, rk = _atp().atp_svd_entropy(ctx, sigma, [len(g) for g in groups])
    ctx.poll()
    mu, rk = mu.cpu().numpy(), rk.cpu().numpy()
    for i, g in enumerate(groups):
        want = oracle.svd_entropy(g) if len(g) else 0.0
        assert abs(mu[i] - want) <= 1e-5 * max(1.0, abs(want))
        if g.sum() > 0:
            # the integer is decided in fp64 on both sides; skip a value within 1e-6 of an integer boundary
            x = 2.0 ** want
            if abs(x - round(x)) > 1e-6:
                assert rk[i] == math.ceil(x)
        else:
            assert rk[i] == 0
    assert rk[0] == 8 and rk[1] == 1


def test_svd_entropy_of_a_full_spectrum_from_the_basis_call(ctx):
    rng = np.random.default_rng(21)
    L, d = 96, 64
    X = _planted(rng, L, d, 10, "f32", noise=0.05)
    _, _, sig = _atp().atp_principal_basis(ctx, to_dev(X, "f32"), [L], [min(L, d)])
    mu, rk = _atp().atp_svd_entropy(ctx, sig, [min(L, d)])
    ctx.poll()
    s = oracle.svd_jacobi(X)[1]
    want = oracle.svd_entropy(s)
    assert abs(float(mu[0]) - want) <= 1e-4 * max(1.0, want)


# ------------------------------------------------------------------ rotary positions (Sec. 4.2)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("q_mode", ["lowrank", "full"])
@pytest.mark.parametrize("L,d,heads,dh,r", [(150, 128, 2, 64, 45), (70, 96, 3, 32, 70), (257, 256, 2, 128, 129)])
def test_attention_with_rotary_positions_on_oracle_basis(ctx, dtype, q_mode, L, d, heads, dh, r):
    rng = np.random.default_rng(900 + L + r)
    X = _planted(rng, L, d, 10, dtype)
    dp = heads * dh
    W = [ai.finish(ai.gaussian_weight(rng, d, dp), dtype) for _ in range(3)]
    U, Xr, _ = oracle.principal_basis(X, r)
    U, Xr = ai.finish(U, dtype), ai.finish(Xr, dtype)
    pos = rng.integers(0, 4000, L).astype(np.int32)
    want = oracle.attention_rope(X, U, Xr, W[0], W[1], W[2], heads, positions=pos, rope_base=10000.0,
                                 q_mode=1 if q_mode == "full" else 0)
    got = _atp().atp_attention(ctx, to_dev(X, dtype), to_dev(U, dtype), to_dev(Xr, dtype), *(to_dev(w, dtype) for w in W),
                               heads, [L], [r], q_mode=q_mode, rope_base=10000.0, positions=torch.from_numpy(pos).cuda())
    ctx.poll()
    assert rel_err(to_np(got), want) <= TOL[dtype]


def test_rotary_positions_default_to_row_index_per_sequence_and_zero_positions_are_plain_attention(ctx):
    rng = np.random.default_rng(31)
    lengths, ranks, d, heads, dh = [40, 0, 75], [10, 0, 20], 64, 2, 32
    dp = heads * dh
    Xs = [_planted(rng, L, d, 6, "f32") if L else np.zeros((0, d)) for L in lengths]
    W = [ai.finish(ai.gaussian_weight(rng, d, dp), "f32") for _ in range(3)]
    bases = [oracle.principal_basis(x, r)[:2] if len(x) else (np.zeros((0, 0)), np.zeros((0, d))) for x, r in zip(Xs, ranks)]
    maxr = max(ranks)
    Upack = np.zeros((sum(lengths), maxr)); row = 0
    for (U, _), L, r in zip(bases, lengths, ranks):
        Upack[row:row + L, :r] = U; row += L
    Xrpack = np.concatenate([b[1] for b in bases])
    args = (to_dev(np.concatenate(Xs), "f32"), to_dev(Upack, "f32"), to_dev(Xrpack, "f32"), *(to_dev(w, "f32") for w in W))
    got = to_np(_atp().atp_attention(ctx, *args, heads, lengths, ranks, rope_base=500.0))
    zero = to_np(_atp().atp_attention(ctx, *args, heads, lengths, ranks, rope_base=500.0,
                                      positions=torch.zeros(sum(lengths), dtype=torch.int32, device="cuda")))
    plain = to_np(_atp().atp_attention(ctx, *args, heads, lengths, ranks))
    ctx.poll()
    assert rel_err(zero, plain) <= 1e-6
    row = 0
    for x, (U, Xr), L, r in zip(Xs, bases, lengths, ranks):
        if L:
            want = oracle.attention_rope(x, U, Xr, W[0], W[1], W[2], heads, rope_base=500.0)     # positions 0..L-1
            assert rel_err(got[row:row + L], want) <= 1e-4
        row += L


# ------------------------------------------------------------------ a chain of layers
def test_stack_of_layers_equals_manual_chaining_and_options_reach_the_attention(ctx):
    from paper_2403_02352_b200.layer import AtpLayer, AtpStack
    atp = _atp()
    rng = np.random.default_rng(404)
    lengths, ranks, d, heads, dff = [96, 64], [24, 16], 64, 2, 128
    X = to_dev(np.concatenate([_planted(rng, L, d, 8, "f32") for L in lengths]), "f32")

    def weights():
        w = {k: to_dev(ai.finish(ai.gaussian_weight(rng, d, d), "f32"), "f32") for k in ("W_Q", "W_K", "W_V", "W_O")}
        w["W_1"] = to_dev(ai.finish(ai.gaussian_weight(rng, d, dff), "f32"), "f32")
        w["W_2"] = to_dev(ai.finish(ai.gaussian_weight(rng, dff, d), "f32"), "f32")
        return w

    ws = [weights(), weights()]
    for kw in (dict(), dict(q_mode="full", rope_base=10000.0)):
        stack = AtpStack(ctx, ws, lengths, ranks, heads, ffn="gelu", **kw)
        out = stack.forward(X).clone()
        x = X
        for w in ws:
            layer = AtpLayer(ctx, w, lengths, ranks, heads, ffn="gelu", **kw)
            y = layer.forward(x)
            x = atp.atp_input_norm(ctx, layer.H, y, kind="layer")
        ctx.poll()
        assert torch.isfinite(out).all()
        assert torch.equal(out, x)                 # same calls, same order: bit-identical
    plain = AtpStack(ctx, ws, lengths, ranks, heads, ffn="gelu").forward(X)
    assert not torch.equal(plain, out)             # the options changed the result


# ------------------------------------------------------------------ basis without host read-back, in a CUDA graph
def test_basis_without_host_sync_matches_and_can_be_captured(ctx):
    atp = _atp()
    rng = np.random.default_rng(77)
    lengths, ranks, d = [160, 96], [40, 24], 128
    X = to_dev(np.concatenate([_planted(rng, L, d, 12, "bf16") for L in lengths]), "bf16")
    U0, X0, s0 = atp.atp_principal_basis(ctx, X, lengths, ranks)
    U1, X1, s1 = atp.atp_principal_basis(ctx, X, lengths, ranks, no_host_sync=True, max_sweeps=16)
    ctx.poll()
    assert torch.equal(U0, U1) and torch.equal(X0, X1) and torch.equal(s0, s1)
    # the same call recorded by a stream capture and replayed on fresh outputs
    out = (torch.zeros_like(U0), torch.zeros_like(X0), torch.zeros_like(s0))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        ctx.use_current_stream()
        atp.atp_principal_basis(ctx, X, lengths, ranks, no_host_sync=True, max_sweeps=16, out=out, auto_workspace=False)
        torch.cuda.synchronize()
        for t in out:
            t.zero_()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            ctx.use_current_stream()
            atp.atp_principal_basis(ctx, X, lengths, ranks, no_host_sync=True, max_sweeps=16, out=out, auto_workspace=False)
        g.replay()
        torch.cuda.synchronize()
    ctx.use_current_stream()
    ctx.poll()
    assert torch.equal(out[0], U0) and torch.equal(out[1], X0) and torch.equal(out[2], s0)
