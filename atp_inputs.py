"""Seeded synthetic inputs for the ATP prefill hot path.

This module only draws random numbers and assembles matrices with a planted
low-rank part; it holds none of the method's arithmetic (no basis extraction,
no attention, no low-rank linear algebra beyond building the inputs) so that
both the CPU oracle's tests and the GPU tests can share it.

The inputs stand in for hidden states of BERT / Llama-2 style models on the
text-classification and question-answering workloads the paper evaluates
(Table 2 gives the model shapes): those datasets and weights are not
available offline, so each workload is a random matrix with a planted
low-rank component plus i.i.d. Gaussian noise, of the shape, rank fraction
and spectrum decay named by the workload list below.

Values meant for a bf16 run are rounded to bf16 once, here; both sides start
from exactly those values (held as float64 arrays whose entries are
bf16-representable).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import numpy as np


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16, returned as float32 holding bf16 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).reshape(a.shape)


def _orthonormal(rng: np.random.Generator, n: int, k: int) -> np.ndarray:
    q, _ = np.linalg.qr(rng.standard_normal((n, k)))
    return q


def planted_matrix(rng, L: int, d: int, spectrum: Sequence[float], noise_std: float,
                   frob2: Optional[float] = None):
    """X = U_p diag(s) V_p^T + noise, with explicitly orthonormal planted factors.

    Returns (X, s) where s holds the planted singular values after scaling the
    planted part to squared Frobenius norm `frob2` (default L*d: unit-RMS entries).
    With noise_std == 0 the singular values of X are exactly s (closed form).
    """
    s = np.asarray(spectrum, dtype=np.float64)
    k = s.shape[0]
    up = _orthonormal(rng, L, k)
    vp = _orthonormal(rng, d, k)
    if frob2 is None:
        frob2 = float(L) * float(d)
    s = s * math.sqrt(frob2 / float((s ** 2).sum()))
    x = (up * s) @ vp.T
    if noise_std > 0:
        x = x + noise_std * rng.standard_normal((L, d))
    return x, s


def gaussian_weight(rng, d_in: int, d_out: int) -> np.ndarray:
    """i.i.d. N(0, 1/d_in) weights, laid out d_in x d_out (so that X @ W matches Eq. 2)."""
    return rng.standard_normal((d_in, d_out)) / math.sqrt(d_in)


@dataclasses.dataclass
class Seq:
    X: np.ndarray          # L x d, float64 holding values of the workload dtype
    r: int
    planted_sigma: np.ndarray


@dataclasses.dataclass
class Workload:
    name: str
    dtype: str             # "f32" or "bf16"
    d: int
    heads: int
    seqs: List[Seq]
    weights: dict          # name -> d_in x d_out array
    ffn: Optional[str]     # None, "gelu", "swiglu"
    d_ff: int
    input_norm: Optional[str]   # None or "rms"

    @property
    def lengths(self):
        return [s.X.shape[0] for s in self.seqs]

    @property
    def ranks(self):
        return [s.r for s in self.seqs]

    @property
    def tokens(self):
        return int(sum(self.lengths))


def finish(x, dtype):
    """Round once to the workload dtype; keep as float64 for the oracle."""
    if dtype == "bf16":
        return round_to_bf16(x).astype(np.float64)
    if dtype == "f64":
        return np.asarray(x, dtype=np.float64)
    return np.asarray(x, dtype=np.float32).astype(np.float64)


def _weights(rng, d, dtype, ffn, d_ff, names=("W_Q", "W_K", "W_V", "W_O")):
    w = {n: finish(gaussian_weight(rng, d, d), dtype) for n in names}
    if ffn == "gelu":
        w["W_1"] = finish(gaussian_weight(rng, d, d_ff), dtype)
        w["W_2"] = finish(gaussian_weight(rng, d_ff, d), dtype)
    elif ffn == "swiglu":
        w["W_gate"] = finish(gaussian_weight(rng, d, d_ff), dtype)
        w["W_up"] = finish(gaussian_weight(rng, d, d_ff), dtype)
        w["W_down"] = finish(gaussian_weight(rng, d_ff, d), dtype)
    return w


def bert_base_fp32(L=512, d=768, heads=12, r=128, k=32, noise=0.01, seed=0) -> Workload:
    """Workload 1: X = A.B + noise.N, singular values of A scaled by 0.8^i, fp32."""
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((L, k))
    b = rng.standard_normal((k, d))
    u, s, vt = np.linalg.svd(a, full_matrices=False)      # input construction only
    a = (u * (s * 0.8 ** np.arange(k))) @ vt
    x = a @ b + noise * rng.standard_normal((L, d))
    w = _weights(rng, d, "f32", None, 0)
    return Workload("bert_base_fp32", "f32", d, heads,
                    [Seq(finish(x, "f32"), r, s * 0.8 ** np.arange(k))], w, None, 0, None)


def bert_large_bf16(batch=16, L=512, d=1024, heads=16, r=256, k=64, noise=0.02,
                    d_ff=4096, seed=2000) -> Workload:
    """Workload 2: planted rank-64 part with 0.9^i spectrum + N(0, 0.02^2), bf16, GELU FFN."""
    rng = np.random.default_rng(seed + r)
    seqs = []
    for _ in range(batch):
        x, s = planted_matrix(rng, L, d, 0.9 ** np.arange(k), noise)
        seqs.append(Seq(finish(x, "bf16"), r, s))
    w = _weights(rng, d, "bf16", "gelu", d_ff)
    return Workload(f"bert_large_bf16_r{r}", "bf16", d, heads, seqs, w, "gelu", d_ff, None)


def llama7b_bf16(L=4096, d=4096, heads=32, r=1024, k=256, noise=0.01, d_ff=11008,
                 seed=3000) -> Workload:
    """Workload 3: planted rank-256 power-law (i^-1.2) part + N(0, 0.01^2), bf16, RMSNorm, SwiGLU."""
    rng = np.random.default_rng(seed + r)
    x, s = planted_matrix(rng, L, d, np.arange(1, k + 1) ** -1.2, noise)
    w = _weights(rng, d, "bf16", "swiglu", d_ff)
    return Workload(f"llama7b_bf16_r{r}", "bf16", d, heads, [Seq(finish(x, "bf16"), r, s)],
                    w, "swiglu", d_ff, "rms")


def long_context_bf16(L=16384, d=4096, heads=32, r=1024, k=512, noise=0.01, seed=4000) -> Workload:
    """Workload 4: attention only, planted rank-512 (1/i) part + N(0, 0.01^2), fixed r."""
    rng = np.random.default_rng(seed + L)
    x, s = planted_matrix(rng, L, d, 1.0 / np.arange(1, k + 1), noise)
    w = _weights(rng, d, "bf16", None, 0, names=("W_Q", "W_K", "W_V"))
    return Workload(f"long_context_bf16_L{L}", "bf16", d, heads, [Seq(finish(x, "bf16"), r, s)],
                    w, None, 0, None)


def serving_batch_bf16(batch=8, L=1024, d=4096, heads=32, noise=0.01, kmin=32, kmax=256,
                       seed=5000) -> Workload:
    """Workload 5: ragged lengths uniform in [L/2, L], r_b = L_b // 4, planted rank uniform
    in [kmin, kmax] with a spectrum falling 100x across the planted part, + N(0, 0.01^2)."""
    rng = np.random.default_rng(seed + 10 * batch + L)
    seqs = []
    for _ in range(batch):
        lb = int(rng.integers(L // 2, L + 1))
        kb = int(rng.integers(kmin, kmax + 1))
        rho = 10.0 ** (-2.0 / max(kb - 1, 1))
        x, s = planted_matrix(rng, lb, d, rho ** np.arange(kb), noise)
        seqs.append(Seq(finish(x, "bf16"), lb // 4, s))
    w = _weights(rng, d, "bf16", None, 0, names=("W_Q", "W_K", "W_V"))
    return Workload(f"serving_b{batch}_L{L}", "bf16", d, heads, seqs, w, None, 0, None)


def exact_rank(L, d, k, dtype="f32", decay=0.8, seed=7):
    """Exact-rank-k matrix with distinct, geometrically decaying singular values (no noise)."""
    rng = np.random.default_rng(seed)
    x, s = planted_matrix(rng, L, d, decay ** np.arange(k), 0.0)
    return finish(x, dtype), s


def pack(seqs: Sequence[Seq]):
    """Packed varlen layout: rows of all sequences stacked; returns (X, row_off, rank, rank_off)."""
    row_off = np.zeros(len(seqs) + 1, dtype=np.int32)
    rank_off = np.zeros(len(seqs) + 1, dtype=np.int32)
    for i, s in enumerate(seqs):
        row_off[i + 1] = row_off[i] + s.X.shape[0]
        rank_off[i + 1] = rank_off[i] + s.r
    x = np.concatenate([s.X for s in seqs], axis=0)
    rank = np.array([s.r for s in seqs], dtype=np.int32)
    return x, row_off, rank, rank_off
