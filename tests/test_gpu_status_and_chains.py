"""Device-side status paths, end-to-end parity on gap inputs shaped like the workloads (T3), and a chain of
layers against the oracle's stack (stage parity on the bases the GPU produced)."""
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


# ------------------------------------------------------------------ status word
def test_sweep_limit_raises_not_converged_once_and_leaves_the_context_usable(ctx):
    atp = _atp()
    from paper_2403_02352_b200 import binding as B
    rng = np.random.default_rng(5)
    X, _ = ai.planted_matrix(rng, 256, 192, 0.9 ** np.arange(24), 0.05)       # noisy: r cuts through the bulk
    Xd = to_dev(ai.finish(X, "bf16"), "bf16")
    U, Xr, sig = atp.atp_principal_basis(ctx, Xd, [256], [96], max_sweeps=1)
    with pytest.raises(atp.AtpError) as e:
        ctx.poll()
    assert e.value.code == B.ERR_NOT_CONVERGED
    ctx.poll()                                                                # reading the status cleared it
    assert torch.isfinite(U.float()).all() and torch.isfinite(Xr.float()).all()
    U2, Xr2, _ = atp.atp_principal_basis(ctx, Xd, [256], [96])                # default budget: converges
    ctx.poll()
    assert np.abs(to_np(U2).T @ to_np(U2) - np.eye(96)).max() <= 2e-2


def test_bounded_wait_that_runs_out_raises_timeout(ctx):
    atp = _atp()
    from paper_2403_02352_b200 import binding as B
    ctx.selftest_wait_timeout()               # a barrier between CTAs whose partner does not exist, short limit
    with pytest.raises(atp.AtpError) as e:
        ctx.poll()
    assert e.value.code == B.ERR_TIMEOUT
    ctx.poll()
    rng = np.random.default_rng(6)            # the next persistent kernel must not see a stale abort flag
    X, _ = ai.planted_matrix(rng, 128, 96, 0.8 ** np.arange(8), 0.0)
    Xd = to_dev(ai.finish(X, "f32"), "f32")
    U, Xr, _ = atp.atp_principal_basis(ctx, Xd, [128], [8])
    ctx.poll()
    assert rel_err(to_np(U) @ to_np(Xr), X) <= 1e-4


def test_non_finite_input_raises_range(ctx):
    atp = _atp()
    from paper_2403_02352_b200 import binding as B
    rng = np.random.default_rng(7)
    X = rng.standard_normal((128, 96))
    X[17, 5] = np.inf
    Xd = torch.from_numpy(X).to(torch.bfloat16).cuda()
    atp.atp_principal_basis(ctx, Xd, [128], [16])
    with pytest.raises(atp.AtpError) as e:
        ctx.poll()
    assert e.value.code == B.ERR_RANGE
    ctx.poll()


# ------------------------------------------------------------------ T3 on gap inputs shaped like the workloads
def _gap_case(name):
    """The workload's recipe with the noise switched off and r = the planted rank: distinct singular values, a
    gap at r, so that the basis is unique up to the sign rule and end-to-end parity is well posed."""
    if name == "bert_base_fp32":
        return ai.bert_base_fp32(noise=0.0, r=32, k=32)
    if name == "bert_large_bf16":
        return ai.bert_large_bf16(batch=2, noise=0.0, r=64, k=64)
    if name == "llama_like_bf16":
        return ai.llama7b_bf16(L=512, d=512, heads=4, r=48, k=48, d_ff=1376, noise=0.0)
    if name == "long_context_like_bf16":
        return ai.long_context_bf16(L=2048, d=512, heads=4, r=64, k=64, noise=0.0)
    return ai.serving_batch_bf16(batch=3, L=512, d=512, heads=4, noise=0.0, kmin=32, kmax=64)


@pytest.mark.parametrize("name", ["bert_base_fp32", "bert_large_bf16", "llama_like_bf16", "long_context_like_bf16",
                                  "serving_like_bf16"])
def test_end_to_end_on_gap_inputs_of_each_workload(ctx, name):
    atp = _atp()
    w = _gap_case(name)
    dt = w.dtype
    Xp, row_off, rank, rank_off = ai.pack(w.seqs)
    Xd = to_dev(Xp, dt)
    Wd = {k: to_dev(v, dt) for k, v in w.weights.items()}
    ranks = list(w.ranks)
    if name == "serving_like_bf16":            # r_b = L_b / 4 by recipe; the gap sits at the planted rank
        ranks = [len(s.planted_sigma) for s in w.seqs]
    Xin = Xd
    if w.input_norm:
        Xin = atp.atp_input_norm(ctx, Xd, None, kind=w.input_norm)
    U, Xr, sig = atp.atp_principal_basis(ctx, Xin, w.lengths, ranks, power_iters=4)
    O = atp.atp_attention(ctx, Xin, U, Xr, Wd["W_Q"], Wd["W_K"], Wd["W_V"], w.heads, w.lengths, ranks)
    ctx.poll()
    ko = np.concatenate([[0], np.cumsum(ranks)]).astype(int)
    worst_o, worst_p, agree, total = 0.0, 0.0, 0, 0
    for b, s in enumerate(w.seqs):
        r = ranks[b]
        xin = to_np(Xin[row_off[b]:row_off[b + 1]])
        Uo, Xo, so = oracle.principal_basis(xin, r)
        Ug, Xg = to_np(U[row_off[b]:row_off[b + 1]])[:, :r], to_np(Xr[ko[b]:ko[b + 1]])
        worst_p = max(worst_p, rel_err(Ug @ Xg, Uo @ Xo))
        # sign agreement per component (the sign rule is the same on both sides)
        dots = np.einsum("ij,ij->j", Ug, Uo)
        agree += int((dots > 0).sum()); total += r
        Oo = oracle.attention(xin, Uo, Xo, w.weights["W_Q"], w.weights["W_K"], w.weights["W_V"], w.heads)
        worst_o = max(worst_o, rel_err(to_np(O[row_off[b]:row_off[b + 1]]), Oo))
    print(f"T3 {name}: err(U_r X_r) {worst_p:.2e}  err(O) {worst_o:.2e}  signs {agree}/{total}")
    assert agree == total
    # U_r X_r is sign- and rotation-free: storage precision. O multiplies the basis error by logits of order
    # 10^2 before the exponential, so its end-to-end bar is looser than the stage bar (tolerances).
    assert worst_p <= (1e-5 if dt == "f32" else 2e-2)
    assert worst_o <= (2e-3 if dt == "f32" else 1e-1)


# ------------------------------------------------------------------ a chain of layers against the oracle
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_two_layer_stack_stage_parity_against_the_oracle(ctx, dtype):
    from paper_2403_02352_b200.layer import AtpStack
    from test_gpu_workloads import _check_layer_stages
    atp = _atp()
    rng = np.random.default_rng(21)
    L, d, dff, heads, r = 160, 64, 128, 2, 24
    lengths, ranks = [L, 96], [r, 16]
    Xs = [ai.finish(ai.planted_matrix(rng, n, d, 0.8 ** np.arange(10), 0.03)[0], dtype) for n in lengths]

    def weights():
        w = {k: ai.finish(ai.gaussian_weight(rng, d, d), dtype) for k in ("W_Q", "W_K", "W_V", "W_O")}
        w["W_1"] = ai.finish(ai.gaussian_weight(rng, d, dff), dtype)
        w["W_2"] = ai.finish(ai.gaussian_weight(rng, dff, d), dtype)
        return w

    ws = [weights(), weights()]
    wd = [{k: to_dev(v, dtype) for k, v in w.items()} for w in ws]
    stack = AtpStack(ctx, wd, lengths, ranks, heads, ffn="gelu", post_norm="layer")
    Xd = to_dev(np.concatenate(Xs), dtype)
    out = stack.forward(Xd)
    ctx.poll()
    assert torch.isfinite(out.float()).all()
    row_off = np.concatenate([[0], np.cumsum(lengths)]).astype(int)
    x_in = Xd
    for l, layer in enumerate(stack.layers):
        # every stage of layer l against the oracle evaluated on the GPU's own input to that stage
        seqs = [ai.Seq(to_np(x_in[row_off[b]:row_off[b + 1]]), ranks[b], None) for b in range(2)]
        wl = ai.Workload("stack", dtype, d, heads, seqs, ws[l], "gelu", dff, None)
        _check_layer_stages(layer, wl, x_in)
        # block closing X_{l+1} = Norm(H_l + Y_l) (Sec. 4.2: the next layer takes the previous layer's output)
        for b in range(2):
            sl = slice(row_off[b], row_off[b + 1])
            want = oracle.norm(to_np(layer.H[sl]), residual=to_np(layer.Y[sl]), kind="layer")
            assert rel_err(to_np(stack.Xnext[l][sl]), want) <= (1e-5 if dtype == "f32" else 1.6e-2)
        x_in = stack.Xnext[l]
    assert torch.equal(out, stack.Xnext[-1])
    # and the oracle's own stack composes the same stages: on an input it can follow end to end (fp32, a gap at
    # r, distinct singular values) the two agree within the end-to-end bar of a single layer, compounded
    if dtype == "f32":
        Xg = ai.finish(ai.planted_matrix(rng, L, d, 0.7 ** np.arange(r), 0.0)[0], "f32")
        wo = [{k: w[k] for k in ("W_Q", "W_K", "W_V")} for w in ws[:1]]
        ref = oracle.stack_forward(Xg, wo, r, heads)
        st1 = AtpStack(ctx, [{k: wd[0][k] for k in ("W_Q", "W_K", "W_V")}], [L], [r], heads)
        got = st1.forward(to_dev(Xg, "f32"))
        ctx.poll()
        assert rel_err(to_np(got), ref) <= 2e-3
