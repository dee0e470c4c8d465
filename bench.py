#!/usr/bin/env python
"""Benchmark of the ATP prefill hot path on B200: one "step" is one pass of the whole layer
(Norm -> basis -> attention on r principal keys -> output projection and FFN through the low-rank
representation) over one batch of synthetic sequences.

    python bench.py --gpus 1 --steps K --warmup W [--workload NAME] [--rank R]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

Prints one JSON line (rank 0). With N > 1 ranks (torchrun) every rank processes its own batch of
independent sequences (no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
import atp_inputs as ai  # noqa: E402

WORKLOADS = {
    # name: (builder, kwargs, layer composition)
    "bert_large_bf16": dict(build=lambda r, seed: ai.bert_large_bf16(r=r or 256, seed=seed), default_rank=256),
    "bert_base_fp32": dict(build=lambda r, seed: ai.bert_base_fp32(r=r or 128, seed=seed - 2000), default_rank=128),
    "llama7b_bf16": dict(build=lambda r, seed: ai.llama7b_bf16(r=r or 2048, seed=seed + 1000), default_rank=2048),
    "long_context_bf16": dict(build=lambda r, seed: ai.long_context_bf16(r=r or 1024, seed=seed + 2000), default_rank=1024),
    "serving_bf16": dict(build=lambda r, seed: ai.serving_batch_bf16(seed=seed + 3000), default_rank=0),
}
POST_NORM = {"gelu": "layer", "swiglu": "rms", None: "layer"}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        m = json.load(open(p))
        return dict(hbm_gbs=m["hbm_gbs"], bf16_tflops=m["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 148 SMs x 128 FMA lanes x 2 flop x max SM clock


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return None
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


ALT_INNER = 2        # rounds per component of Algorithm 1, as the paper runs it

# DRAM bytes (read + write) of one launch of the dominant kernels, from one ncu pass on the same command
# (profiles/ncu_metrics_llama7b_bf16_r2048.md); other workloads / kernels: no capture, null.
NCU_DRAM_BYTES_PER_LAUNCH = {("llama7b_bf16", 2048, "jacobi_persistent"): 33.7e6,
                             ("llama7b_bf16", 2048, "orth_persistent"): 67.2e6}


def alt_start_vectors(w, seed):
    """The Gaussian start vectors of Algorithm 1 (one row per component), part of the seeded input."""
    rng = np.random.default_rng(seed + 7)
    return [rng.standard_normal((s.r, w.d)).astype(np.float32) for s in w.seqs]


def workload_config(w, world, extraction="randomized"):
    ranks = w.ranks
    layer = "basis+attention" + ("+W_O" if "W_O" in w.weights else "") + ("+FFN" if w.ffn else "")
    if extraction == "alternating":
        layer = f"attention block: Algorithm 1 extraction (inner {ALT_INNER}) + attention"
    return {"workload": w.name + ("_alg1" if extraction == "alternating" else ""), "batch": len(w.lengths),
            "tokens_per_step_per_gpu": w.tokens, "d": w.d,
            "heads": w.heads, "rank": ranks[0] if len(set(ranks)) == 1 else "L_b/4",
            "ffn": w.ffn, "d_ff": w.d_ff, "input_norm": w.input_norm, "extraction": extraction,
            "layer": layer,
            "l2": "flushed between steps (256 MiB memset), rotating input copies",
            "parallelism": f"dp{world} (independent sequences per rank)"}


def oracle_step(w, seq_index, extraction="randomized", v0=None):
    import oracle
    s = w.seqs[seq_index]
    if extraction == "alternating":
        U, Xp = oracle.alternating_svd(s.X, s.r, v0[seq_index].astype(np.float64), inner=ALT_INNER)
        return oracle.attention(s.X, U, Xp, w.weights["W_Q"], w.weights["W_K"], w.weights["W_V"], w.heads)
    return oracle.layer_forward(s.X, w.weights, s.r, w.heads, ffn=w.ffn, input_norm=w.input_norm,
                                post_norm=POST_NORM[w.ffn])


SAMPLE_ROUNDS = 12       # Jacobi rounds timed per decomposition shape in a bounded oracle sample
SAMPLE_HEADS = 2         # heads of the oracle attention timed in a bounded sample
SAMPLE_COLS = 128        # output columns of each oracle linear layer timed in a bounded sample


def oracle_sample(w, seq_index, extraction="randomized", v0=None, state=None):
    """Seconds the CPU oracle needs for one sequence of the workload (one layer pass).

    Small sequences (min(L, d) <= 1024) are run in full. For larger ones a full pass would take hours (a
    one-sided Jacobi SVD of 4096 columns is ~10^13 flops), so every stage is timed on a bounded part whose cost
    is proportional to a loop count of the oracle, and scaled to the full count:
      * Jacobi SVD: SAMPLE_ROUNDS rounds (a round rotates n/2 disjoint pairs; a sweep is n-1 rounds), scaled to
        `sweeps` sweeps, the number the oracle needs to converge on a 384 x 384 corner of the same input;
      * X_r = U_r^T X: its first 64 rows of r;   attention: SAMPLE_HEADS heads of all;
      * linear layers: SAMPLE_COLS output columns of d_out.
    Returns (seconds, description, extrapolated?). `state` caches the sweep count between calls."""
    import oracle
    s = w.seqs[seq_index]
    L, d = s.X.shape
    what = "full layer" if extraction == "randomized" else "attention block"
    if min(L, d) <= 1024 or extraction == "alternating":
        t0 = time.perf_counter()
        oracle_step(w, seq_index, extraction, v0)
        return time.perf_counter() - t0, f"one sequence in full ({L} tokens), {what}", False
    state = state if state is not None else {}
    W, r, heads = w.weights, s.r, w.heads
    X = np.asarray(s.X, dtype=np.float64)
    if "sweeps" not in state:
        state["sweeps"] = oracle.svd_jacobi(X[:384, :384])[3]
    sweeps = state["sweeps"]

    def timed(fn):
        t0 = time.perf_counter()
        fn()
        return time.perf_counter() - t0

    def svd_seconds(M):
        nvec = min(M.shape)
        per_sweep = nvec - 1 + (nvec & 1)
        dt = timed(lambda: oracle.svd_jacobi_capped(M, SAMPLE_ROUNDS))
        return dt * sweeps * per_sweep / SAMPLE_ROUNDS

    total = 0.0
    Xin = oracle.norm(X, kind=w.input_norm) if w.input_norm else X
    if w.input_norm:
        total += timed(lambda: oracle.norm(X, kind=w.input_norm))
    t_svd_x = svd_seconds(Xin)
    # stand-ins of the right shape for the stages after the (unfinished) decomposition: their cost does not
    # depend on the values
    if "U" not in state:
        rng = np.random.default_rng(5)
        state["U"] = np.linalg.qr(rng.standard_normal((L, r)))[0]
        state["F"] = rng.standard_normal((L, w.d_ff)) if w.ffn else None
        state["Fr"] = rng.standard_normal((r, w.d_ff)) if w.ffn else None
    U = state["U"]
    t_proj = timed(lambda: oracle.project_rows(Xin, U, 64)) * r / 64
    Xr = U.T @ Xin
    n_basis = 1
    dh = W["W_Q"].shape[1] // heads
    c = SAMPLE_HEADS * dh
    t_attn = timed(lambda: oracle.attention(Xin, U, Xr, W["W_Q"][:, :c], W["W_K"][:, :c], W["W_V"][:, :c], SAMPLE_HEADS)) * heads / SAMPLE_HEADS
    total += t_svd_x + t_proj + t_attn
    if "W_O" in W:
        n_basis += 1
        total += t_svd_x + t_proj          # basis of O: same shape as X
        total += timed(lambda: oracle.lowrank_linear(U, Xr, W["W_O"][:, :SAMPLE_COLS])) * W["W_O"].shape[1] / SAMPLE_COLS
    if w.ffn:
        n_basis += 2
        total += timed(lambda: oracle.norm(X, residual=Xin, kind=POST_NORM[w.ffn]))
        total += t_svd_x + t_proj          # basis of H
        if w.ffn == "gelu":
            W1, W2 = W["W_1"], W["W_2"]
            total += timed(lambda: oracle.lowrank_linear(U, Xr, W1[:, :SAMPLE_COLS], act="gelu")) * W1.shape[1] / SAMPLE_COLS
        else:
            W1, W2 = W["W_up"], W["W_down"]
            total += timed(lambda: oracle.lowrank_linear(U, Xr, W1[:, :SAMPLE_COLS], W_gate=W["W_gate"][:, :SAMPLE_COLS],
                                                         act="swiglu")) * W1.shape[1] / SAMPLE_COLS
        F = state["F"]
        total += svd_seconds(F)
        total += timed(lambda: oracle.project_rows(F, U, 64)) * r / 64
        Fr = state["Fr"]
        total += timed(lambda: oracle.lowrank_linear(U, Fr, W2[:, :SAMPLE_COLS])) * W2.shape[1] / SAMPLE_COLS
    desc = (f"one sequence ({L} tokens), {what}, extrapolated from bounded parts: {SAMPLE_ROUNDS} Jacobi rounds per "
            f"decomposition shape scaled to {sweeps} sweeps (the count on a 384x384 corner of the input) x {n_basis} "
            f"decompositions, 64 of {r} rows of U_r^T X, {SAMPLE_HEADS} of {heads} heads, {SAMPLE_COLS} output columns "
            f"per linear layer")
    return total, desc, True


def run_reference(args):
    """The CPU oracle as it stands, on the host cores; each step is one sequence of the workload (a bounded,
    extrapolated sample of it when the sequence is too large to finish, see oracle_sample)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = WORKLOADS[args.workload]["build"](args.rank, args.seed)
    nseq = len(w.seqs)
    v0 = alt_start_vectors(w, args.seed) if args.extraction == "alternating" else None
    state = {}
    for i in range(args.warmup):
        oracle_sample(w, i % nseq, args.extraction, v0, state)
    secs, toks, desc, extrap = 0.0, 0, "", False
    for i in range(args.steps):
        dt, desc, extrap = oracle_sample(w, i % nseq, args.extraction, v0, state)
        secs += dt
        toks += w.seqs[i % nseq].X.shape[0]
    val = toks / secs
    line = {"impl": "reference", "metric": "ATP layer prefill tokens/sec", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args.gpus, args.extraction),
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": desc, "extrapolated": extrap},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def stage_rooflines(w, stage_ms, pk, sbytes):
    """Per library call of the layer: algorithmic flops and bytes (the method's own counts: two passes over X for
    the extraction, the r-row projections, the L x r score and value contractions, the two chained products of a
    low-rank linear layer), the measured time, and both roofline fractions; `binds` names the larger ideal time."""
    out = {}
    if not stage_ms:
        return out
    d, dff = w.d, w.d_ff or 0
    Ls, rs = w.lengths, w.ranks
    sumL = sum(Ls)
    sLr = sum(L * r for L, r in zip(Ls, rs))
    sr = sum(rs)

    def basis(dd):
        return 4.0 * sLr * dd, (2.0 * sumL * dd + sLr + sr * dd) * sbytes

    def linear(din, dout, nw=1):
        return nw * (2.0 * sr * din * dout + 2.0 * sLr * dout), (nw * din * dout + sLr + sr * din + sumL * dout) * sbytes

    model = {"basis_X": basis(d), "basis_O": basis(d), "basis_H": basis(d), "basis_F": basis(dff),
             "attention": (6.0 * sr * d * d + 6.0 * sLr * d, (sLr + sr * d + 3.0 * d * d + sumL * d) * sbytes),
             "linear_WO": linear(d, d), "linear_ffn_in": linear(d, dff, 2 if w.ffn == "swiglu" else 1),
             "linear_ffn_out": linear(dff, d),
             "norm_in": (0.0, 2.0 * sumL * d * sbytes), "norm_post": (0.0, 3.0 * sumL * d * sbytes)}
    for name, ms in stage_ms.items():
        fl, by = model.get(name, (0.0, 0.0))
        sec = ms / 1e3
        t_tensor, t_hbm = fl / (pk["bf16_tflops"] * 1e12), by / (pk["hbm_gbs"] * 1e9)
        out[name] = {"ms": ms, "flops": fl, "bytes": by, "tflops": fl / sec / 1e12, "gbs": by / sec / 1e9,
                     "tensor_frac": t_tensor / sec, "hbm_frac": t_hbm / sec, "binds": "tensor" if t_tensor > t_hbm else "hbm"}
    return out


def run_kernel_linear(args):
    """Micro-benchmark of the low-rank linear layer (a5: T = X_r W, Y = U_r T, two tcgen05 GEMMs) through the
    public call, at the shapes of the default workload. One JSON line per shape: algorithmic TFLOP/s
    (2 r d_in d_out + 2 L r d_out flops over the CUDA-event time of a call, L2 flushed between calls) and the
    fraction of the measured sustained bf16 peak."""
    import torch
    import paper_2403_02352_b200 as atp
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = atp.Context(0)
    pk = peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    g = torch.Generator(device=dev); g.manual_seed(args.seed)
    L, r = 4096, (args.rank or 2048)
    for name, d_in, d_out in (("W_O", 4096, 4096), ("FFN up", 4096, 11008), ("FFN down", 11008, 4096)):
        U = (torch.randn(L, r, device=dev, generator=g) / math.sqrt(L)).to(torch.bfloat16)
        Xr = torch.randn(r, d_in, device=dev, generator=g).to(torch.bfloat16)
        W = (torch.randn(d_in, d_out, device=dev, generator=g) / math.sqrt(d_in)).to(torch.bfloat16)
        Y = torch.empty(L, d_out, device=dev, dtype=torch.bfloat16)
        for _ in range(max(args.warmup, 3)):
            atp.atp_lowrank_linear(ctx, U, Xr, W, [L], [r], out=Y)
        times = []
        for _ in range(args.steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); atp.atp_lowrank_linear(ctx, U, Xr, W, [L], [r], out=Y); e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ctx.poll()
        ms = float(np.median(times))
        flops = 2.0 * r * d_in * d_out + 2.0 * L * r * d_out
        tf = flops / ms / 1e9
        print(json.dumps({"kernel": "lowrank_linear (gemm_tc x 2)", "shape": name, "L": L, "r": r, "d_in": d_in, "d_out": d_out,
                          "ms": ms, "tflops": tf, "peak": pk["bf16_tflops"], "frac": tf / pk["bf16_tflops"],
                          "peak_source": pk["source"], "steps": args.steps, "l2": "flushed between calls"}))
    ctx.close()
    return 0



def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_bf16", choices=sorted(WORKLOADS))
    ap.add_argument("--rank", type=int, default=0, help="number of principal keys r (0: the workload's default)")
    ap.add_argument("--seed", type=int, default=2000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extraction", default="randomized", choices=["randomized", "alternating"],
                    help="alternating: time the attention block with the paper's Algorithm 1 as the extraction")
    ap.add_argument("--power-iters", type=int, default=-1)
    ap.add_argument("--jacobi-block", type=int, default=0)
    ap.add_argument("--jacobi-inner", type=int, default=0)
    ap.add_argument("--max-sweeps", type=int, default=0)
    ap.add_argument("--no-long-context", action="store_true", help="skip the T(32768)/T(16384) measurement")
    ap.add_argument("--kernel", default=None, choices=["linear"],
                    help="micro-benchmark of one stage instead of the layer: linear = the two GEMMs of a low-rank linear layer")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.kernel == "linear":
        return run_kernel_linear(args)

    import torch
    import paper_2403_02352_b200 as atp          # raises if libatp.so is missing: no fallback
    from paper_2403_02352_b200.layer import AtpLayer

    from paper_2403_02352_b200 import dist as pdist
    world, rank, local = pdist.env_ranks()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pdist.init("nccl", dev)
    args.warmup = max(args.warmup, 3)

    w = WORKLOADS[args.workload]["build"](args.rank, pdist.rank_seed(args.seed, rank))   # every rank: its own sequences
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16

    def dev_mat(a, pin=False):
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(tdt)
        return t.pin_memory() if pin else t.to(dev)

    weights = {k: dev_mat(v) for k, v in w.weights.items()}
    Xpacked, row_off, rank_arr, rank_off = ai.pack(w.seqs)
    lengths, ranks = w.lengths, w.ranks
    tokens = int(sum(lengths))
    x_bytes = Xpacked.size * (4 if w.dtype == "f32" else 2)
    # rotating input sets: the same sequences with rows cyclically shifted per set would change the
    # problem; instead each set is an independent copy placed at a different address, and the L2 is
    # flushed between steps, so that no step finds its inputs or weights cached.
    nsets = max(2, min(8, int(300e6 // max(x_bytes, 1)) + 1))
    Xsets = [dev_mat(Xpacked) for _ in range(nsets)]
    Xhost = dev_mat(Xpacked, pin=True)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    ctx = atp.Context(local)
    layer = AtpLayer(ctx, weights, lengths, ranks, w.heads, ffn=w.ffn, input_norm=w.input_norm,
                     post_norm=POST_NORM[w.ffn], power_iters=args.power_iters,
                     basis_kwargs=dict(jacobi_block=args.jacobi_block, jacobi_inner=args.jacobi_inner,
                                       max_sweeps=args.max_sweeps))
    out_rows, out_cols = None, None

    if args.extraction == "alternating":
        V0 = torch.from_numpy(np.concatenate(alt_start_vectors(w, pdist.rank_seed(args.seed, rank)))).to(dev)
        bufs = {}

        def step(i):
            X = Xsets[i % nsets]
            if "U" not in bufs:
                bufs["U"], bufs["Xr"] = atp.atp_alternating_basis(ctx, X, V0, lengths, ranks, inner=ALT_INNER)
            else:
                atp.atp_alternating_basis(ctx, X, V0, lengths, ranks, inner=ALT_INNER, out=(bufs["U"], bufs["Xr"]))
            bufs["O"] = atp.atp_attention(ctx, X, bufs["U"], bufs["Xr"], weights["W_Q"], weights["W_K"], weights["W_V"],
                                          w.heads, lengths, ranks, out=bufs.get("O"))
            return bufs["O"]
    else:
        def step(i):
            return layer.forward(Xsets[i % nsets])

    for i in range(args.warmup):
        y = step(i)
    ctx.poll()
    out_shape = tuple(y.shape)
    Yhost = torch.empty(out_shape, dtype=tdt).pin_memory()

    def barrier():
        torch.cuda.synchronize()
        pdist.barrier()
        torch.cuda.synchronize()

    # ---- device-timed region: K steps, CUDA events per step, L2 flushed between steps
    sampler = ClockSampler(local) if rank == 0 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = ctx.launches
    barrier()
    if sampler:
        sampler.start()
    for i in range(args.steps):
        flush.zero_()
        evs[i][0].record()
        step(i)
        evs[i][1].record()
    barrier()
    clocks = sampler.stop() if sampler else None
    launches = (ctx.launches - launches0)
    ctx.poll()
    ms = pdist.max_over_ranks(sum(a.elapsed_time(b) for a, b in evs), dev)
    value = pdist.aggregate_tokens_per_s(tokens, args.steps, ms, world)

    # ---- end to end: pinned host input -> device, layer, result -> host, every step
    xd = torch.empty_like(Xsets[0])
    e2e_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        flush.zero_()
        e2e_ev[i][0].record()
        xd.copy_(Xhost, non_blocking=True)
        yy = layer.forward(xd)
        Yhost.copy_(yy, non_blocking=True)
        e2e_ev[i][1].record()
    barrier()
    ms_e2e = pdist.max_over_ranks(sum(a.elapsed_time(b) for a, b in e2e_ev), dev)
    e2e = {"value": pdist.aggregate_tokens_per_s(tokens, args.steps, ms_e2e, world), "unit": "tokens/s",
           "h2d_bytes_per_step": int(x_bytes), "d2h_bytes_per_step": int(Yhost.numel() * Yhost.element_size())}

    if rank != 0:
        pdist.finish()
        return

    # ---- per-stage times: an event pair around every library call of the layer (separate pass)
    pk = peaks()
    sbytes = 4 if w.dtype == "f32" else 2
    stage_ms = {}
    nstage = 3
    if args.extraction == "randomized":
        for i in range(nstage):
            flush.zero_()
            evl = []
            layer.forward(Xsets[i % nsets], stage_events=evl)
            torch.cuda.synchronize()
            for name, a, b in evl:
                stage_ms[name] = stage_ms.get(name, 0.0) + a.elapsed_time(b) / nstage
    stages = stage_rooflines(w, stage_ms, pk, sbytes)

    # ---- per-kernel times (event pair around every launch; separate pass, not the timed one)
    ctx.profile_start()
    nprof = 2
    for i in range(nprof):
        flush.zero_()
        step(i)
    prof = ctx.profile_stop()
    total_ms = sum(v["ms"] for v in prof.values()) or 1.0
    dom_name, dom = max(prof.items(), key=lambda kv: kv[1]["ms"])

    def rate(name, rec):
        per_launch_s = rec["ms"] / 1e3 / max(rec["launches"], 1)
        fl, by = rec["flops"] / max(rec["launches"], 1), rec["bytes"] / max(rec["launches"], 1)
        if name.startswith("gemm_tc") or name.startswith("attn_tc"):
            return "tensor", fl / per_launch_s / 1e12, pk["bf16_tflops"], "TFLOP/s"
        if fl > 0:
            return "alu", fl / per_launch_s / 1e12, FP32_ALU_TFLOPS, "TFLOP/s"
        return "hbm", by / per_launch_s / 1e9, pk["hbm_gbs"], "GB/s"

    kernels = {k: {"launches": v["launches"] // nprof, "ms_per_step": v["ms"] / nprof, "share": v["ms"] / total_ms,
                   "bound": rate(k, v)[0], "executed": rate(k, v)[1], "executed_frac": rate(k, v)[1] / rate(k, v)[2],
                   "unit": rate(k, v)[3]} for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])}
    # The dominant kernel is a part of the basis extraction; its roofline entry is the extraction's ALGORITHMIC work
    # (bytes (2 L d + L r + r d) s and flops 4 L d r per call, summed over the calls of a step) over the time this
    # kernel takes per step, against the measured HBM copy bandwidth, with the tensor-peak fraction beside it.
    ext_bytes = sum(v["bytes"] for k, v in stages.items() if k.startswith("basis"))
    ext_flops = sum(v["flops"] for k, v in stages.items() if k.startswith("basis"))
    dom_s = dom["ms"] / nprof / 1e3
    in_extraction = not (dom_name.startswith("attn") or dom_name in ("norm", "rope"))
    if in_extraction and ext_bytes > 0:
        achieved = ext_bytes / dom_s / 1e9
        roofline = {"kernel": dom_name, "bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / pk["hbm_gbs"], "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((args.workload, ranks[0], dom_name)),
                    "tensor_frac": ext_flops / dom_s / 1e12 / pk["bf16_tflops"],
                    "work": "algorithmic bytes / flops of the extraction calls of a step over this kernel's time per step"}
    else:
        bound, achieved, peak, unit = rate(dom_name, dom)
        roofline = {"kernel": dom_name, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                    "frac": achieved / peak, "traffic": None}
    roofline.update({"peak_source": pk["source"], "share_of_step": dom["ms"] / total_ms, "launches_per_step": dom["launches"] // nprof,
                     "stages": stages, "kernels": kernels})

    # ---- long context: T(32768) / T(16384) of the attention block (basis + attention), linear-in-L claim of Fig. 4
    per_workload = None
    if not args.no_long_context and world == 1 and args.workload == "llama7b_bf16":
        per_workload = {}
        del layer, Xsets, xd
        torch.cuda.empty_cache()
        for Llong in (16384, 32768):
            wl = ai.long_context_bf16(L=Llong, r=1024, seed=args.seed + 2000)
            wts = {k: dev_mat(v) for k, v in wl.weights.items()}
            Xl = dev_mat(ai.pack(wl.seqs)[0])
            ll = AtpLayer(ctx, wts, wl.lengths, wl.ranks, wl.heads, ffn=None, input_norm=None)
            for _ in range(2):
                ll.forward(Xl)
            evl = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(3)]
            for a, b in evl:
                flush.zero_()
                a.record()
                ll.forward(Xl)
                b.record()
            torch.cuda.synchronize()
            ctx.poll()
            msl = sum(a.elapsed_time(b) for a, b in evl) / len(evl)
            per_workload[f"long_context_bf16_L{Llong}"] = {"ms_per_step": msl, "tokens_per_s": Llong / msl * 1e3, "rank": 1024,
                                                           "layer": "basis+attention"}
            del ll, Xl, wts, wl
            torch.cuda.empty_cache()
        per_workload["T32768_over_T16384"] = (per_workload["long_context_bf16_L32768"]["ms_per_step"] /
                                              per_workload["long_context_bf16_L16384"]["ms_per_step"])

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (about 10-30 s)
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        import oracle
        v0_cpu = alt_start_vectors(w, args.seed) if args.extraction == "alternating" else None
        t0 = time.perf_counter()
        n, toks, secs, desc, extrap, state = 0, 0, 0.0, "", False, {}
        if min(w.seqs[0].X.shape) > 1024:
            oracle_sample(w, 0, args.extraction, v0_cpu, state)      # untimed: page in the oracle's buffers
        while n < len(w.seqs) and (time.perf_counter() - t0 < 15.0 or n == 0):
            dt, desc, extrap = oracle_sample(w, n, args.extraction, v0_cpu, state)
            secs += dt
            toks += w.seqs[n].X.shape[0]
            n += 1
        cpu = {"value": toks / secs, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"{n} of {len(w.seqs)} sequences; each: {desc}; wall time of the sample {time.perf_counter() - t0:.1f} s",
               "extrapolated": extrap}

    line = {"metric": "ATP layer prefill tokens/sec", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_config(w, world, args.extraction),
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu}
    if per_workload:
        line["per_workload"] = per_workload
    print(json.dumps(line), flush=True)
    pdist.finish()


if __name__ == "__main__":
    main()
