"""ctypes binding of include/atp.h. Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libatp.so")

OK, ERR_INVALID_ARG, ERR_INVALID_RANK, ERR_UNSUPPORTED_DTYPE, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, \
    ERR_NOT_CONVERGED, ERR_TIMEOUT, ERR_RANGE, ERR_STATIC_SCRATCH_LIMIT = range(10)
STATIC_SCRATCH_BYTES = 8 << 20
F32, BF16 = 0, 1
OP_BASIS, OP_ATTENTION, OP_LINEAR, OP_NORM, OP_ALTERNATING = 0, 1, 2, 3, 4
Q_LOWRANK, Q_FULL = 0, 1
ACT = {None: 0, "none": 0, "gelu": 1, "swiglu": 2}
NORM = {"rms": 0, "layer": 1}

exported_symbols = (
    "atp_create", "atp_destroy", "atp_set_stream", "atp_workspace_bytes", "atp_set_workspace",
    "atp_input_norm", "atp_principal_basis", "atp_attention", "atp_lowrank_linear",
    "atp_poll_device_status", "atp_launch_count", "atp_status_string", "atp_profile_start", "atp_profile_stop",
    "atp_lowrank_linear_static", "atp_alternating_basis", "atp_svd_entropy",
    "atp_basis_workspace_bytes", "atp_selftest_wait_timeout", "atp_selftest_per_device_once",
)


class AtpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (atp_status {code})")


class Mat(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64)]


class Seqs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("row_off", C.POINTER(C.c_int32)), ("rank", C.POINTER(C.c_int32)),
                ("rank_off", C.POINTER(C.c_int32))]


class BasisOpts(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("oversample", C.c_int32), ("power_iters", C.c_int32),
                ("max_sweeps", C.c_int32), ("seed", C.c_uint64), ("jacobi_block", C.c_int32), ("jacobi_inner", C.c_int32), ("groups", C.c_int32),
                ("no_host_sync", C.c_int32)]


class AttnOpts(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("q_mode", C.c_int32), ("scale", C.c_float), ("rope_base", C.c_float),
                ("positions", C.c_void_p)]


class LinearOpts(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("act", C.c_int32), ("bias", C.c_void_p), ("W_gate", C.POINTER(Mat))]


def library_path() -> str:
    return _LIB_PATH


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2403_02352_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(_LIB_PATH)
    lib.atp_status_string.restype = C.c_char_p
    lib.atp_launch_count.restype = C.c_int64
    lib.atp_launch_count.argtypes = [C.c_void_p]
    lib.atp_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    lib.atp_destroy.argtypes = [C.c_void_p]
    lib.atp_set_stream.argtypes = [C.c_void_p, C.c_void_p]
    lib.atp_set_workspace.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
    lib.atp_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.POINTER(Seqs), C.c_int64, C.c_int64, C.c_int,
                                        C.POINTER(C.c_size_t)]
    lib.atp_basis_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(Seqs), C.c_int64, C.c_int, C.POINTER(BasisOpts),
                                              C.POINTER(C.c_size_t)]
    lib.atp_selftest_wait_timeout.argtypes = [C.c_void_p]
    lib.atp_selftest_per_device_once.restype = C.c_int
    lib.atp_poll_device_status.argtypes = [C.c_void_p]
    lib.atp_profile_start.argtypes = [C.c_void_p]
    lib.atp_profile_stop.argtypes = [C.c_void_p, C.c_char_p, C.c_size_t, C.POINTER(C.c_size_t)]
    lib.atp_input_norm.argtypes = [C.c_void_p, C.POINTER(Mat), C.POINTER(Mat), C.c_int, C.c_float, C.POINTER(Mat)]
    lib.atp_alternating_basis.argtypes = [C.c_void_p, C.POINTER(Mat), C.POINTER(Seqs), C.POINTER(Mat), C.c_int,
                                          C.POINTER(Mat), C.POINTER(Mat)]
    lib.atp_svd_entropy.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32), C.c_int32, C.c_void_p, C.c_void_p]
    lib.atp_principal_basis.argtypes = [C.c_void_p, C.POINTER(Mat), C.POINTER(Seqs), C.POINTER(BasisOpts),
                                        C.POINTER(Mat), C.POINTER(Mat), C.c_void_p]
    lib.atp_attention.argtypes = [C.c_void_p, C.POINTER(Mat), C.POINTER(Mat), C.POINTER(Mat), C.POINTER(Mat),
                                  C.POINTER(Mat), C.POINTER(Mat), C.c_int, C.POINTER(Seqs), C.POINTER(AttnOpts),
                                  C.POINTER(Mat)]
    lib.atp_lowrank_linear.argtypes = [C.c_void_p, C.POINTER(Mat), C.POINTER(Mat), C.POINTER(Mat), C.POINTER(Seqs),
                                       C.POINTER(LinearOpts), C.POINTER(Mat)]
    lib.atp_lowrank_linear_static.argtypes = [C.c_void_p, C.POINTER(Mat), C.POINTER(Mat), C.POINTER(Mat),
                                              C.POINTER(Seqs), C.POINTER(LinearOpts), C.POINTER(Mat)]
    return lib


lib = _load()


def status_string(code: int) -> str:
    return lib.atp_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != OK:
        raise AtpError(code, where)


def mat(t: Optional[torch.Tensor]) -> Optional[Mat]:
    """Describe a 2-D row-major torch tensor (device memory stays owned by the tensor)."""
    if t is None:
        return None
    if t.dim() != 2 or t.stride(1) != 1 and t.shape[1] > 1:
        raise ValueError("expected a 2-D tensor with unit stride along columns")
    if t.dtype == torch.float32:
        dt = F32
    elif t.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise AtpError(ERR_UNSUPPORTED_DTYPE, "mat")
    ld = t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0))
    return Mat(t.data_ptr(), dt, t.shape[0], t.shape[1], ld)


class SeqDesc:
    """Host arrays of a packed batch (kept alive for the duration of a call)."""

    def __init__(self, lengths: Sequence[int], ranks: Sequence[int]):
        self.lengths = [int(x) for x in lengths]
        self.ranks = [int(x) for x in ranks]
        if len(self.lengths) != len(self.ranks):
            raise ValueError("lengths and ranks differ in size")
        n = len(self.lengths)
        self.row_off = np.zeros(n + 1, dtype=np.int32)
        self.rank_off = np.zeros(n + 1, dtype=np.int32)
        self.row_off[1:] = np.cumsum(self.lengths)
        self.rank_off[1:] = np.cumsum(self.ranks)
        self.rank = np.asarray(self.ranks, dtype=np.int32)
        p32 = C.POINTER(C.c_int32)
        self.c = Seqs(n, self.row_off.ctypes.data_as(p32), self.rank.ctypes.data_as(p32),
                      self.rank_off.ctypes.data_as(p32))

    @property
    def total_rows(self):
        return int(self.row_off[-1])

    @property
    def total_rank(self):
        return int(self.rank_off[-1])


class Context:
    """Owns an atp_ctx and a workspace tensor that grows on demand."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("libatp needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self._h = C.c_void_p()
        _check(lib.atp_create(C.byref(self._h), device), "atp_create")
        self._ws = None
        self.use_current_stream()

    def close(self):
        if self._h:
            lib.atp_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def use_current_stream(self):
        s = torch.cuda.current_stream(self.device)
        _check(lib.atp_set_stream(self._h, C.c_void_p(s.cuda_stream)), "atp_set_stream")

    def workspace_bytes(self, op: int, seqs: SeqDesc, d: int, d_out: int, dtype: int) -> int:
        out = C.c_size_t(0)
        _check(lib.atp_workspace_bytes(self._h, op, C.byref(seqs.c), d, d_out, dtype, C.byref(out)), "atp_workspace_bytes")
        return int(out.value)

    def ensure_workspace(self, nbytes: int):
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(int(nbytes), dtype=torch.uint8, device=self.device)
            _check(lib.atp_set_workspace(self._h, C.c_void_p(self._ws.data_ptr()), self._ws.numel()), "atp_set_workspace")

    def set_workspace(self, t: Optional[torch.Tensor]):
        self._ws = t
        if t is None:
            _check(lib.atp_set_workspace(self._h, None, 0), "atp_set_workspace")
        else:
            _check(lib.atp_set_workspace(self._h, C.c_void_p(t.data_ptr()), t.numel() * t.element_size()), "atp_set_workspace")

    def selftest_wait_timeout(self):
        """Enqueues a kernel whose barrier cannot complete; the next poll() raises ATP_ERR_TIMEOUT."""
        self.ensure_workspace(256)
        _check(lib.atp_selftest_wait_timeout(self._h), "atp_selftest_wait_timeout")

    def poll(self):
        """Synchronise and raise if a kernel recorded a device-side condition."""
        _check(lib.atp_poll_device_status(self._h), "device status")

    def profile_start(self):
        _check(lib.atp_profile_start(self._h), "atp_profile_start")

    def profile_stop(self):
        """Returns {kernel name: dict(launches, ms, flops, bytes)} for the launches since profile_start."""
        buf = C.create_string_buffer(1 << 16)
        _check(lib.atp_profile_stop(self._h, buf, len(buf), None), "atp_profile_stop")
        out = {}
        for line in buf.value.decode().splitlines():
            name, n, ms, fl, by = line.split()
            out[name] = dict(launches=int(n), ms=float(ms), flops=float(fl), bytes=float(by))
        return out

    @property
    def launches(self) -> int:
        return int(lib.atp_launch_count(self._h))


def _padded(shape, like: torch.Tensor) -> torch.Tensor:
    """Uninitialised (rows x cols) tensor whose leading dimension is a multiple of 8 elements."""
    rows, cols = shape
    return torch.empty((rows, (cols + 7) // 8 * 8), dtype=like.dtype, device=like.device)[:, :cols]


def _dt(t: torch.Tensor) -> int:
    return F32 if t.dtype == torch.float32 else BF16


def atp_input_norm(ctx: Context, X, residual=None, kind="rms", eps=1e-5, out=None):
    Y = torch.empty_like(X) if out is None else out
    mx, my = mat(X), mat(Y)
    mr = mat(residual)
    _check(lib.atp_input_norm(ctx._h, C.byref(mx), C.byref(mr) if mr else None, NORM[kind], eps, C.byref(my)), "atp_input_norm")
    return Y


def atp_principal_basis(ctx: Context, X, lengths, ranks, oversample=-1, power_iters=-1, max_sweeps=0, seed=0,
                        out=None, auto_workspace=True, jacobi_block=0, jacobi_inner=0, groups=0, no_host_sync=False):
    """(U_r, X_r, sigma) for a packed batch; see include/atp.h."""
    sd = SeqDesc(lengths, ranks)
    d = X.shape[1]
    maxr = max(sd.ranks) if sd.ranks else 0
    if out is None:
        ldu = (maxr + 7) // 8 * 8
        U = torch.zeros((sd.total_rows, ldu), dtype=X.dtype, device=X.device)[:, :maxr]
        Xr = torch.empty((sd.total_rank, (d + 7) // 8 * 8), dtype=X.dtype, device=X.device)[:, :d]
        sig = torch.empty(sd.total_rank, dtype=torch.float32, device=X.device)
    else:
        U, Xr, sig = out
    opts = BasisOpts(C.sizeof(BasisOpts), oversample, power_iters, max_sweeps, seed, jacobi_block, jacobi_inner, groups,
                     1 if no_host_sync else 0)
    if auto_workspace:
        need = C.c_size_t(0)
        _check(lib.atp_basis_workspace_bytes(ctx._h, C.byref(sd.c), d, _dt(X), C.byref(opts), C.byref(need)),
               "atp_basis_workspace_bytes")
        ctx.ensure_workspace(int(need.value))
    mx, mu, mxr = mat(X), mat(U), mat(Xr)
    _check(lib.atp_principal_basis(ctx._h, C.byref(mx), C.byref(sd.c), C.byref(opts), C.byref(mu), C.byref(mxr),
                                   C.c_void_p(sig.data_ptr()) if sig is not None else None), "atp_principal_basis")
    return U, Xr, sig


def atp_attention(ctx: Context, X, U_r, X_r, W_Q, W_K, W_V, heads, lengths, ranks, q_mode="lowrank", scale=0.0,
                  out=None, auto_workspace=True, rope_base=0.0, positions=None):
    sd = SeqDesc(lengths, ranks)
    dp = W_Q.shape[1]
    O = _padded((sd.total_rows, dp), U_r) if out is None else out
    if auto_workspace:
        ctx.ensure_workspace(ctx.workspace_bytes(OP_ATTENTION, sd, X_r.shape[1], dp, _dt(X_r)))
    if positions is not None and (positions.dtype != torch.int32 or not positions.is_cuda or positions.numel() != sd.total_rows):
        raise ValueError("positions: CUDA int32 tensor with one entry per row")
    opts = AttnOpts(C.sizeof(AttnOpts), Q_FULL if q_mode == "full" else Q_LOWRANK, scale, rope_base,
                    C.c_void_p(positions.data_ptr()) if positions is not None else None)
    mx = mat(X)
    ms = [mat(t) for t in (U_r, X_r, W_Q, W_K, W_V, O)]
    _check(lib.atp_attention(ctx._h, C.byref(mx) if mx else None, C.byref(ms[0]), C.byref(ms[1]), C.byref(ms[2]),
                             C.byref(ms[3]), C.byref(ms[4]), heads, C.byref(sd.c), C.byref(opts), C.byref(ms[5])),
           "atp_attention")
    return O


def atp_lowrank_linear(ctx: Context, U_r, X_r, W, lengths, ranks, bias=None, act=None, W_gate=None, out=None,
                       auto_workspace=True):
    sd = SeqDesc(lengths, ranks)
    d_out = W.shape[1]
    Y = _padded((sd.total_rows, d_out), U_r) if out is None else out
    if auto_workspace:
        ctx.ensure_workspace(ctx.workspace_bytes(OP_LINEAR, sd, X_r.shape[1], d_out, _dt(X_r)))
    mg = mat(W_gate)
    opts = LinearOpts(C.sizeof(LinearOpts), ACT[act], C.c_void_p(bias.data_ptr()) if bias is not None else None,
                      C.pointer(mg) if mg else None)
    ms = [mat(t) for t in (U_r, X_r, W, Y)]
    _check(lib.atp_lowrank_linear(ctx._h, C.byref(ms[0]), C.byref(ms[1]), C.byref(ms[2]), C.byref(sd.c), C.byref(opts),
                                  C.byref(ms[3])), "atp_lowrank_linear")
    return Y


def atp_lowrank_linear_static(U_r, X_r, W, lengths, ranks, out, bias=None, act=None, stream=None):
    """Y = act(U_r (X_r W) + bias) through the entry point that allocates nothing: no context, no
    workspace; the intermediate lives in a fixed buffer inside the library (see include/atp.h for
    the size limit and the rules on overlapping calls). `out` must be supplied by the caller."""
    sd = SeqDesc(lengths, ranks)
    opts = LinearOpts(C.sizeof(LinearOpts), ACT[act], C.c_void_p(bias.data_ptr()) if bias is not None else None, None)
    ms = [mat(t) for t in (U_r, X_r, W, out)]
    s = torch.cuda.current_stream(U_r.device).cuda_stream if stream is None else stream
    with torch.cuda.device(U_r.device):
        _check(lib.atp_lowrank_linear_static(C.c_void_p(s), C.byref(ms[0]), C.byref(ms[1]), C.byref(ms[2]),
                                             C.byref(sd.c), C.byref(opts), C.byref(ms[3])), "atp_lowrank_linear_static")
    return out


def atp_alternating_basis(ctx: Context, X, V0, lengths, ranks, inner=2, out=None, auto_workspace=True):
    """Algorithm 1: (U, X') from alternating rank-1 fits with deflation; see include/atp.h."""
    sd = SeqDesc(lengths, ranks)
    d = X.shape[1]
    maxr = max(sd.ranks) if sd.ranks else 0
    if out is None:
        U = torch.zeros((sd.total_rows, (maxr + 7) // 8 * 8), dtype=X.dtype, device=X.device)[:, :maxr]
        Xr = torch.empty((sd.total_rank, (d + 7) // 8 * 8), dtype=X.dtype, device=X.device)[:, :d]
    else:
        U, Xr = out
    if auto_workspace:
        ctx.ensure_workspace(ctx.workspace_bytes(OP_ALTERNATING, sd, d, 0, _dt(X)))
    mx, mv, mu, mxr = mat(X), mat(V0), mat(U), mat(Xr)
    _check(lib.atp_alternating_basis(ctx._h, C.byref(mx), C.byref(sd.c), C.byref(mv), int(inner), C.byref(mu), C.byref(mxr)),
           "atp_alternating_basis")
    return U, Xr


def atp_svd_entropy(ctx: Context, sigma: torch.Tensor, counts: Sequence[int]):
    """(mu, rank) per group of singular values (Eq. 4, rank = ceil(2^mu)); `counts` = group sizes."""
    off = np.zeros(len(counts) + 1, dtype=np.int32)
    off[1:] = np.cumsum(np.asarray(counts, dtype=np.int64))
    mu = torch.empty(len(counts), dtype=torch.float32, device=sigma.device)
    rk = torch.empty(len(counts), dtype=torch.int32, device=sigma.device)
    _check(lib.atp_svd_entropy(ctx._h, C.c_void_p(sigma.data_ptr()), off.ctypes.data_as(C.POINTER(C.c_int32)), len(counts),
                               C.c_void_p(mu.data_ptr()), C.c_void_p(rk.data_ptr())), "atp_svd_entropy")
    return mu, rk
