"""The allocation-free entry point against the regular one.

atp_lowrank_linear_static serves callers that are not allowed to allocate device memory (code
embedded in another program's memory pool, latency-critical loops): it takes no context and no
workspace and keeps its intermediate in a fixed buffer inside the library. This test calls it
through the C ABI twice in a row, with different inputs, and checks each result against
atp_lowrank_linear on the same inputs. The file name makes pytest collect it last, so a run that
stops at the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

import atp_inputs as ai
from gpu_util import TOL, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_static_entry_point_matches_regular_one_twice(dtype):
    import paper_2403_02352_b200 as atp
    from paper_2403_02352_b200 import binding as B
    ctx = atp.Context(0)
    rng = np.random.default_rng(123)
    cases = [([150, 61], [40, 17], 96, 200, "gelu", True), ([203], [64], 128, 72, None, False)]
    for lengths, ranks, d_in, d_out, act, with_bias in cases:          # two calls in a row share the buffer
        rows, tr = sum(lengths), sum(ranks)
        U = to_dev(ai.finish(rng.standard_normal((rows, max(ranks))) / 8, dtype), dtype)
        Xr = to_dev(ai.finish(rng.standard_normal((tr, d_in)), dtype), dtype)
        W = to_dev(ai.finish(ai.gaussian_weight(rng, d_in, d_out), dtype), dtype)
        bias = torch.from_numpy(rng.standard_normal(d_out).astype(np.float32)).cuda() if with_bias else None
        ref = atp.atp_lowrank_linear(ctx, U, Xr, W, lengths, ranks, bias=bias, act=act)
        ctx.poll()
        out = torch.full_like(ref, float("nan"))
        atp.atp_lowrank_linear_static(U, Xr, W, lengths, ranks, out, bias=bias, act=act)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        assert rel_err(to_np(out), to_np(ref)) <= TOL[dtype]
    # The point of the entry point: a call takes no device memory. Repeat the last call (its kernels are loaded by
    # now, so the driver has no code to bring in) and compare the allocator's and the driver's counts around it.
    import gc
    gc.collect()                      # tensors of earlier tests must not be released in the middle of the measurement
    torch.cuda.synchronize()
    before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    atp.atp_lowrank_linear_static(U, Xr, W, lengths, ranks, out, bias=bias, act=act)
    torch.cuda.synchronize()
    after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    assert after[0] <= before[0] and after[1] <= before[1], ("the call took memory from the allocator", before, after)
    assert after[2] >= before[2], ("the call took device memory from the driver", before, after)
    assert rel_err(to_np(out), to_np(ref)) <= TOL[dtype]
    # beyond the fixed buffer: refused on the host, nothing launched
    big_r, big_out = 1024, B.STATIC_SCRATCH_BYTES // 4 // 1024 + 8
    U = torch.zeros((1024, big_r), device="cuda"); Xr = torch.zeros((big_r, 8), device="cuda")
    W = torch.zeros((8, big_out), device="cuda"); Y = torch.zeros((1024, big_out), device="cuda")
    with pytest.raises(atp.AtpError) as e:
        atp.atp_lowrank_linear_static(U, Xr, W, [1024], [big_r], Y)
    assert e.value.code == B.ERR_STATIC_SCRATCH_LIMIT
    with pytest.raises(atp.AtpError):
        atp.atp_lowrank_linear_static(U, Xr, W, [1024], [big_r], Y, act="swiglu")
    ctx.close()
