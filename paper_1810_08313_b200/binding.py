"""ctypes binding of libls.so (include/ls.h).

Argument marshalling only: every arithmetic step runs inside the CUDA library.
torch is used for device memory and streams.  If the library cannot be built
or loaded this module raises; there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

LS_MAX_LAYERS = 8
LS_MAX_REPLICAS = 64

LS_OK = 0
LS_ERR_INVALID_ARG = -1
LS_ERR_BAD_HANDLE = -2
LS_ERR_STATE_SIZE = -3
LS_ERR_NO_DATASET = -4
LS_ERR_ROW_RANGE = -5
LS_ERR_CUDA = -6
LS_ERR_UNSUPPORTED = -7
LS_ERR_OVERFLOW = -8
LS_ERR_DEVICE_TIMEOUT = -9
LS_ERR_TOO_LARGE = -10
LS_ERR_EXCHANGE = -11

LOSS = {"softmax_ce": 0, "mse_half": 1}
GEMM = {"fp32": 0, "bf16": 1}
MOMENTUM_MODE = {"average": 0, "keep": 1, "reset": 2, "block": 3}
KERNEL_CLASSES = ("fwd", "loss", "dx", "dw", "bias", "avg")


class AdacommOpts(C.Structure):
    _fields_ = [("gamma", C.c_double), ("slack", C.c_int32), ("n_decay", C.c_int32), ("decay_at", C.c_void_p),
                ("decay_factor", C.c_double)]


class ModelSpec(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32),
        ("dims", C.c_int32 * (LS_MAX_LAYERS + 1)),
        ("loss", C.c_int32),
        ("has_bias", C.c_int32),
        ("gemm_dtype", C.c_int32),
        ("momentum_mode", C.c_int32),
        ("weight_decay", C.c_float),
        ("block_momentum", C.c_float),
    ]


# int exchange(void* ctx, const float* partial_dev, float* gathered_dev, size_t bytes, int n_gpus)
EXCHANGE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_int)


class LsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib().ls_strerror(code).decode()} ({code})")


_LIB = None


def _lib():
    global _LIB
    if _LIB is not None:
        return _LIB
    path = _build.build()          # compiles with nvcc when missing or stale; raises on failure
    lib = C.CDLL(path)
    vp, i64, f32 = C.c_void_p, C.c_int64, C.c_float
    P = C.POINTER
    sig = {
        "ls_strerror": (C.c_char_p, [C.c_int]),
        "ls_param_count": (C.c_int, [P(ModelSpec), P(i64)]),
        "ls_state_bytes": (C.c_int, [C.c_int, P(ModelSpec), C.c_int, P(C.c_size_t)]),
        "ls_create": (C.c_int, [P(vp), C.c_int, P(ModelSpec), f32, f32, C.c_int, vp, C.c_size_t, vp]),
        "ls_destroy": (C.c_int, [vp]),
        "ls_sync": (C.c_int, [vp]),
        "ls_selftest_wait_timeout": (C.c_int, [vp, i64]),
        "ls_last_cuda_error": (C.c_int, [vp]),
        "ls_set_lr": (C.c_int, [vp, f32]),
        "ls_set_params": (C.c_int, [vp, vp]),
        "ls_set_state": (C.c_int, [vp, C.c_int, vp, vp]),
        "ls_get_state": (C.c_int, [vp, C.c_int, vp, vp]),
        "ls_state_view": (C.c_int, [vp, P(vp), P(vp), P(i64)]),
        "ls_bind_dataset": (C.c_int, [vp, vp, vp, i64]),
        "ls_local_steps": (C.c_int, [vp, C.c_int, vp, vp]),
        "ls_local_steps_avg": (C.c_int, [vp, C.c_int, vp, vp]),
        "ls_local_steps_host": (C.c_int, [vp, C.c_int, vp, vp, vp]),
        "ls_average": (C.c_int, [vp]),
        "ls_average_flat": (C.c_int, [vp, C.c_int, i64, i64, vp]),
        "ls_block_average_flat": (C.c_int, [vp, vp, vp, C.c_int, i64, i64, C.c_float, C.c_float, vp]),
        "ls_set_block_state": (C.c_int, [vp, vp, vp]),
        "ls_run_timed": (C.c_int, [vp, i64, C.c_int, C.c_double, i64, vp, vp, vp, i64, vp, vp, vp, vp, vp, i64, vp, vp]),
        "ls_delay": (C.c_int, [C.c_double, C.c_int, C.c_int, vp]),
        "ls_speedup": (C.c_int, [C.c_double, C.c_int, vp]),
        "ls_error_bound": (C.c_int, [C.c_double] * 6 + [C.c_int, C.c_int, C.c_double, C.c_double, vp]),
        "ls_tau_star": (C.c_int, [C.c_double] * 7 + [vp]),
        "ls_simulate_runtime": (C.c_int, [C.c_int, C.c_int, i64, C.c_double, C.c_double, C.c_uint64, C.c_int, vp, vp]),
        "ls_philox4x32_10": (C.c_int, [vp, vp, vp]),
        "ls_get_block_state": (C.c_int, [vp, vp, vp]),
        "ls_eval_loss": (C.c_int, [vp, C.c_int, i64, i64, P(f32)]),
        "adacomm_next_tau": (C.c_int, [C.c_double, C.c_double, C.c_int]),
        "ls_run": (C.c_int, [vp, i64, C.c_int, C.c_int, i64, vp, vp, vp, i64, P(i64), vp, vp, vp, i64, P(i64),
                             P(f32)]),
        "ls_launch_count": (C.c_int, [vp, P(i64)]),
        "adacomm_next_tau_refined": (C.c_int, [C.c_double, C.c_double, C.c_int, C.c_int, C.c_double, C.c_int,
                                               C.c_double, C.c_double, C.c_int]),
        "ls_run_refined": (C.c_int, [vp, i64, C.c_int, C.c_int, i64, vp, vp, P(AdacommOpts), vp, i64, P(i64), vp, vp,
                                     vp, i64, P(i64), P(f32)]),
        "ls_get_lr": (C.c_int, [vp, P(f32)]),
        "ls_linear_loss_static": (C.c_int, [vp, vp, vp, vp, i64, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]),
        "ls_shard_buffer_floats": (C.c_int, [vp, P(i64)]),
        "ls_set_shard": (C.c_int, [vp, C.c_int, C.c_int, vp, vp, EXCHANGE_FN, vp]),
        "ls_shard_partial_sum": (C.c_int, [vp, vp]),
        "ls_shard_average": (C.c_int, [vp, vp, C.c_int, C.c_int]),
        "ls_partial_sum_flat": (C.c_int, [vp, C.c_int, i64, i64, vp, vp]),
        "ls_combine_partials_flat": (C.c_int, [vp, C.c_int, i64, C.c_int, i64, vp, C.c_int, i64, vp]),
        "ls_profile_begin": (C.c_int, [vp, C.c_uint32, C.c_int]),
        "ls_profile_end": (C.c_int, [vp, P(C.c_double), P(i64)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _LIB = lib
    return lib


def library_path() -> str:
    _lib()
    return _build.LIB_PATH


def _check(code: int, where: str):
    if code != LS_OK:
        raise LsError(code, where)


def make_spec(dims: Sequence[int], loss: str = "softmax_ce", has_bias: bool = True, gemm_dtype: str = "fp32",
              momentum_mode: str = "average", weight_decay: float = 0.0, block_momentum: float = 0.0) -> ModelSpec:
    s = ModelSpec()
    if not (2 <= len(dims) <= LS_MAX_LAYERS + 1):
        raise ValueError("1..8 layers")
    s.n_layers = len(dims) - 1
    for i, d in enumerate(dims):
        s.dims[i] = int(d)
    s.loss = LOSS[loss]
    s.has_bias = int(bool(has_bias))
    s.gemm_dtype = GEMM[gemm_dtype]
    s.momentum_mode = MOMENTUM_MODE[momentum_mode]
    s.weight_decay = float(weight_decay)
    s.block_momentum = float(block_momentum)
    return s


def param_count(spec: ModelSpec) -> int:
    n = C.c_int64()
    _check(_lib().ls_param_count(C.byref(spec), C.byref(n)), "ls_param_count")
    return n.value


def state_bytes(m: int, spec: ModelSpec, batch: int) -> int:
    n = C.c_size_t()
    _check(_lib().ls_state_bytes(m, C.byref(spec), batch, C.byref(n)), "ls_state_bytes")
    return n.value


def adacomm_next_tau(F_t: float, F_0: float, tau_0: int) -> int:
    r = _lib().adacomm_next_tau(float(F_t), float(F_0), int(tau_0))
    if r < 0:
        raise LsError(r, "adacomm_next_tau")
    return r


def adacomm_next_tau_refined(F_t: float, F_0: float, tau_0: int, tau_prev: int, gamma: float = 0.5, slack: int = 0,
                             lr_0: float = 1.0, lr_l: float = 1.0, lr_changed: bool = False) -> int:
    r = _lib().adacomm_next_tau_refined(float(F_t), float(F_0), int(tau_0), int(tau_prev), float(gamma), int(slack),
                                        float(lr_0), float(lr_l), int(bool(lr_changed)))
    if r < 0:
        raise LsError(r, "adacomm_next_tau_refined")
    return r


def _stream_ptr(stream) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def average_flat(buf, m: int, P: int, stride: Optional[int] = None, stream=None) -> None:
    """Average m float32 vectors of P elements held in the CUDA tensor `buf`
    (vector j starts at element j*stride) in place."""
    import torch
    if not (buf.is_cuda and buf.dtype == torch.float32 and buf.is_contiguous()):
        raise ValueError("buf must be a contiguous float32 CUDA tensor")
    stride = int(P if stride is None else stride)
    if buf.numel() < (m - 1) * stride + P:
        raise ValueError("buf too small")
    _check(_lib().ls_average_flat(buf.data_ptr(), int(m), int(P), stride, _stream_ptr(stream)), "ls_average_flat")


def partial_sum_flat(buf, m: int, P: int, out, stride: Optional[int] = None, stream=None) -> None:
    """out[0..P) = sum of the m vectors of buf (vector j at j*stride) in index order, fp32 (ls_partial_sum_flat)."""
    stride = int(P if stride is None else stride)
    _check(_lib().ls_partial_sum_flat(buf.data_ptr(), int(m), int(P), stride, out.data_ptr(), _stream_ptr(stream)),
           "ls_partial_sum_flat")


def combine_partials_flat(partials, G: int, part_stride: int, m_total: int, P: int, dst, m_local: int,
                          dst_stride: Optional[int] = None, stream=None) -> None:
    """Every one of the m_local vectors of dst = (partials[0] + ... + partials[G-1], in that order) / m_total
    (ls_combine_partials_flat)."""
    dst_stride = int(P if dst_stride is None else dst_stride)
    _check(_lib().ls_combine_partials_flat(partials.data_ptr(), int(G), int(part_stride), int(m_total), int(P),
                                           dst.data_ptr(), int(m_local), dst_stride, _stream_ptr(stream)),
           "ls_combine_partials_flat")


def block_average_flat(buf, anchor, u, m: int, P: int, lr: float, beta: float, stride: Optional[int] = None,
                       stream=None) -> None:
    """Block-momentum averaging step (Section 5.3) on raw CUDA tensors: buf as for average_flat, anchor and u
    float32 vectors of P elements (the period-start model and the global buffer), all updated in place."""
    import torch
    for t in (buf, anchor, u):
        if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            raise ValueError("contiguous float32 CUDA tensors expected")
    stride = int(P if stride is None else stride)
    if buf.numel() < (m - 1) * stride + P or anchor.numel() < P or u.numel() < P:
        raise ValueError("buffer too small")
    _check(_lib().ls_block_average_flat(buf.data_ptr(), anchor.data_ptr(), u.data_ptr(), int(m), int(P), stride,
                                        float(lr), float(beta), _stream_ptr(stream)), "ls_block_average_flat")


# ---- runtime model (host only; Sections 2-4) ----------------------------------------------------------
DELAY_SCALING = {"constant": 0, "log2": 1, "tree": 2, "linear": 3}


def delay(D0: float, m: int, scaling: str = "tree") -> float:
    out = C.c_double()
    _check(_lib().ls_delay(float(D0), int(m), DELAY_SCALING[scaling], C.byref(out)), "ls_delay")
    return out.value


def speedup(alpha: float, tau: int) -> float:
    out = C.c_double()
    _check(_lib().ls_speedup(float(alpha), int(tau), C.byref(out)), "ls_speedup")
    return out.value


def error_bound(T, F1, Finf, lr, L, sigma2, m, tau, Y, D) -> float:
    out = C.c_double()
    _check(_lib().ls_error_bound(float(T), float(F1), float(Finf), float(lr), float(L), float(sigma2), int(m), int(tau),
                                 float(Y), float(D), C.byref(out)), "ls_error_bound")
    return out.value


def tau_star(F1, Finf, D, lr, L, sigma2, T) -> float:
    out = C.c_double()
    _check(_lib().ls_tau_star(float(F1), float(Finf), float(D), float(lr), float(L), float(sigma2), float(T),
                              C.byref(out)), "ls_tau_star")
    return out.value


def simulate_runtime(m: int, tau: int, n_periods: int, y_mean: float, D: float, seed: int, exponential: bool = True):
    """(mean T_sync, mean T_P-Avg) per iteration over n_periods periods (Section 3.1)."""
    a, b = C.c_double(), C.c_double()
    _check(_lib().ls_simulate_runtime(int(m), int(tau), int(n_periods), float(y_mean), float(D), int(seed),
                                      int(bool(exponential)), C.byref(a), C.byref(b)), "ls_simulate_runtime")
    return a.value, b.value


def philox4x32_10(counter, key):
    c = (C.c_uint32 * 4)(*counter)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    _check(_lib().ls_philox4x32_10(c, k, o), "ls_philox4x32_10")
    return tuple(int(v) for v in o)


def linear_loss_static(W, bias, x, y, chunk_rows: int, chunk_loss, loss: str = "softmax_ce", stream=None) -> None:
    """Per-chunk mean loss of z = W x + b on the rows of x, computed by the library without allocating
    any memory (its scratch is a fixed array inside the library).  W [d_out][d_in], bias [d_out] or None,
    x [n_rows][d_in] float32, y int32 labels / float32 targets, chunk_loss float32 [n_rows // chunk_rows]:
    all CUDA tensors owned by the caller.  Calls that overlap on the GPU must be serialised."""
    _check(_lib().ls_linear_loss_static(W.data_ptr(), None if bias is None else bias.data_ptr(), x.data_ptr(),
                                        y.data_ptr(), int(x.shape[0]), int(x.shape[1]), int(W.shape[0]), LOSS[loss],
                                        int(chunk_rows), chunk_loss.data_ptr(), _stream_ptr(stream)),
           "ls_linear_loss_static")


class LocalSGD:
    """m replicas of a fully connected model on one GPU, trained by local SGD
    steps and periodic averaging.  Thin wrapper over the ls_* calls."""

    def __init__(self, m: int, dims: Sequence[int], loss: str = "softmax_ce", has_bias: bool = True,
                 gemm_dtype: str = "fp32", lr: float = 0.05, momentum: float = 0.0, batch: int = 32,
                 momentum_mode: str = "average", device: str = "cuda:0", stream=None, block_momentum: float = 0.0):
        import torch
        self._torch = torch
        self.lib = _lib()
        self.m, self.batch, self.dims = int(m), int(batch), tuple(int(d) for d in dims)
        self.gemm_dtype = gemm_dtype
        self.loss_kind = loss
        self.spec = make_spec(dims, loss, has_bias, gemm_dtype, momentum_mode, block_momentum=block_momentum)
        self.P = param_count(self.spec)
        nbytes = state_bytes(self.m, self.spec, self.batch)
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.state = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.state.data_ptr()
            self._state_ptr = (base + 255) // 256 * 256
            self.stream = stream if stream is not None else torch.cuda.current_stream()
            h = C.c_void_p()
            _check(self.lib.ls_create(C.byref(h), self.m, C.byref(self.spec), float(lr), float(momentum), self.batch,
                                      self._state_ptr, nbytes, int(self.stream.cuda_stream)), "ls_create")
        self.h = h
        self._x = self._y = None

    # -- life cycle -------------------------------------------------------
    def close(self):
        if getattr(self, "h", None) is not None and self.h.value:
            self.lib.ls_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sync(self):
        _check(self.lib.ls_sync(self.h), "ls_sync")

    def selftest_wait_timeout(self, limit_cycles: int = 2_000_000):
        """Enqueue the kernel whose bounded wait runs out (ls_selftest_wait_timeout); the next call that waits
        for the stream raises LsError(LS_ERR_DEVICE_TIMEOUT)."""
        _check(self.lib.ls_selftest_wait_timeout(self.h, int(limit_cycles)), "ls_selftest_wait_timeout")

    def set_lr(self, lr: float):
        _check(self.lib.ls_set_lr(self.h, float(lr)), "ls_set_lr")

    # -- state ------------------------------------------------------------
    def set_params(self, x1: np.ndarray):
        a = np.ascontiguousarray(x1, dtype=np.float32)
        if a.size != self.P:
            raise ValueError("x1 has the wrong size")
        _check(self.lib.ls_set_params(self.h, a.ctypes.data), "ls_set_params")

    def set_state(self, replica: int, params: Optional[np.ndarray] = None, momentum: Optional[np.ndarray] = None):
        p = None if params is None else np.ascontiguousarray(params, dtype=np.float32)
        v = None if momentum is None else np.ascontiguousarray(momentum, dtype=np.float32)
        for a in (p, v):
            if a is not None and a.size != self.P:
                raise ValueError("wrong size")
        _check(self.lib.ls_set_state(self.h, int(replica), None if p is None else p.ctypes.data,
                                     None if v is None else v.ctypes.data), "ls_set_state")

    def set_block_state(self, anchor: Optional[np.ndarray] = None, u: Optional[np.ndarray] = None):
        a = None if anchor is None else np.ascontiguousarray(anchor, dtype=np.float32)
        b = None if u is None else np.ascontiguousarray(u, dtype=np.float32)
        for t in (a, b):
            if t is not None and t.size != self.P:
                raise ValueError("wrong size")
        _check(self.lib.ls_set_block_state(self.h, None if a is None else a.ctypes.data,
                                           None if b is None else b.ctypes.data), "ls_set_block_state")

    def get_block_state(self):
        a = np.empty(self.P, dtype=np.float32)
        b = np.empty(self.P, dtype=np.float32)
        _check(self.lib.ls_get_block_state(self.h, a.ctypes.data, b.ctypes.data), "ls_get_block_state")
        return a, b

    def get_state(self, replica: int):
        p = np.empty(self.P, dtype=np.float32)
        v = np.empty(self.P, dtype=np.float32)
        _check(self.lib.ls_get_state(self.h, int(replica), p.ctypes.data, v.ctypes.data), "ls_get_state")
        return p, v

    def get_all(self):
        ps, vs = zip(*(self.get_state(i) for i in range(self.m)))
        return np.stack(ps), np.stack(vs)

    def state_view(self):
        """(params, momentum) as float32 CUDA tensors [m][stride] aliasing the state block."""
        torch = self._torch
        pp, vp, st = C.c_void_p(), C.c_void_p(), C.c_int64()
        _check(self.lib.ls_state_view(self.h, C.byref(pp), C.byref(vp), C.byref(st)), "ls_state_view")
        base = self.state.data_ptr()
        out = []
        for ptr in (pp.value, vp.value):
            off = ptr - base
            out.append(self.state[off:off + self.m * st.value * 4].view(torch.float32).view(self.m, st.value))
        return out[0], out[1]

    # -- data ---------------------------------------------------------------
    def bind_dataset(self, x, y):
        torch = self._torch
        want = torch.bfloat16 if self.gemm_dtype == "bf16" else torch.float32
        ywant = torch.int32 if self.loss_kind == "softmax_ce" else torch.float32
        if not (x.is_cuda and x.dtype == want and x.is_contiguous() and x.dim() == 2 and x.shape[1] == self.dims[0]):
            raise ValueError(f"x must be a contiguous CUDA {want} tensor [n_rows][{self.dims[0]}]")
        if not (y.is_cuda and y.dtype == ywant and y.is_contiguous() and y.numel() == x.shape[0]):
            raise ValueError(f"y must be a contiguous CUDA {ywant} tensor [n_rows]")
        self._x, self._y = x, y
        _check(self.lib.ls_bind_dataset(self.h, x.data_ptr(), y.data_ptr(), int(x.shape[0])), "ls_bind_dataset")

    # -- hot path -----------------------------------------------------------
    def local_steps(self, tau: int, row_offsets: np.ndarray, loss_out=None, average: bool = False):
        """tau local steps; average=True: followed by the averaging step (one whole period, ls_local_steps_avg)."""
        offs = np.ascontiguousarray(row_offsets, dtype=np.int64)
        if offs.size != tau * self.m:
            raise ValueError("row_offsets must be [tau][m]")
        lp = None
        if loss_out is not None:
            torch = self._torch
            if not (loss_out.is_cuda and loss_out.dtype == torch.float32 and loss_out.is_contiguous()
                    and loss_out.numel() >= tau * self.m):
                raise ValueError("loss_out must be a contiguous float32 CUDA tensor [tau][m]")
            lp = loss_out.data_ptr()
        if average:
            _check(self.lib.ls_local_steps_avg(self.h, int(tau), offs.ctypes.data, lp), "ls_local_steps_avg")
        else:
            _check(self.lib.ls_local_steps(self.h, int(tau), offs.ctypes.data, lp), "ls_local_steps")

    def local_steps_host(self, tau: int, x_host, y_host, loss_host):
        """x_host [tau][m][batch][d_in], y_host [tau][m][batch], loss_host float32 [tau][m]: CPU torch
        tensors (pinned for overlap)."""
        _check(self.lib.ls_local_steps_host(self.h, int(tau), x_host.data_ptr(), y_host.data_ptr(),
                                            loss_host.data_ptr()), "ls_local_steps_host")

    def average(self):
        _check(self.lib.ls_average(self.h), "ls_average")

    def eval_loss(self, replica: int, row_offset: int, n_rows: int) -> float:
        f = C.c_float()
        _check(self.lib.ls_eval_loss(self.h, int(replica), int(row_offset), int(n_rows), C.byref(f)), "ls_eval_loss")
        return float(f.value)

    def run(self, K: int, tau_0: int, row_offsets: np.ndarray, interval: int = 0, probe_rows: int = 0, loss_out=None):
        """K iterations of local steps + averaging in native code; AdaComm when interval > 0."""
        offs = np.ascontiguousarray(row_offsets, dtype=np.int64)
        if offs.size != K * self.m:
            raise ValueError("row_offsets must be [K][m]")
        max_p = int(K) + 1
        period_tau = np.zeros(max_p, dtype=np.int32)
        dk = np.zeros(max_p, dtype=np.int64)
        dF = np.zeros(max_p, dtype=np.float32)
        dt = np.zeros(max_p, dtype=np.int32)
        n_p, n_d, F0 = C.c_int64(), C.c_int64(), C.c_float()
        lp = None if loss_out is None else loss_out.data_ptr()
        _check(self.lib.ls_run(self.h, int(K), int(tau_0), int(interval), int(probe_rows), offs.ctypes.data, lp,
                               period_tau.ctypes.data, max_p, C.byref(n_p), dk.ctypes.data, dF.ctypes.data,
                               dt.ctypes.data, max_p, C.byref(n_d), C.byref(F0)), "ls_run")
        n_p, n_d = n_p.value, n_d.value
        return {"taus": period_tau[:n_p].tolist(), "decision_k": dk[:n_d].tolist(), "decision_F": dF[:n_d].copy(),
                "decision_tau": dt[:n_d].tolist(), "F_0": float(F0.value) if interval > 0 else None}

    def run_timed(self, K: int, tau_0: int, T0_ms: float, row_offsets: np.ndarray, probe_rows: int, loss_out=None):
        """K iterations with AdaComm decisions at wall-clock intervals of T0_ms (Section 4)."""
        offs = np.ascontiguousarray(row_offsets, dtype=np.int64)
        if offs.size != K * self.m:
            raise ValueError("row_offsets must be [K][m]")
        max_p = int(K) + 1
        period_tau = np.zeros(max_p, dtype=np.int32)
        dk = np.zeros(max_p, dtype=np.int64)
        dF = np.zeros(max_p, dtype=np.float32)
        dt = np.zeros(max_p, dtype=np.int32)
        dms = np.zeros(max_p, dtype=np.float64)
        n_p, n_d, F0 = C.c_int64(), C.c_int64(), C.c_float()
        lp = None if loss_out is None else loss_out.data_ptr()
        _check(self.lib.ls_run_timed(self.h, int(K), int(tau_0), float(T0_ms), int(probe_rows), offs.ctypes.data, lp,
                                     period_tau.ctypes.data, max_p, C.byref(n_p), dk.ctypes.data, dF.ctypes.data,
                                     dt.ctypes.data, dms.ctypes.data, max_p, C.byref(n_d), C.byref(F0)),
               "ls_run_timed")
        n_p, n_d = n_p.value, n_d.value
        return {"taus": period_tau[:n_p].tolist(), "decision_k": dk[:n_d].tolist(), "decision_F": dF[:n_d].copy(),
                "decision_tau": dt[:n_d].tolist(), "decision_ms": dms[:n_d].copy(), "F_0": float(F0.value)}

    def profile_begin(self, classes: Sequence[str] = KERNEL_CLASSES, layer: int = -1):
        mask = 0
        for c in classes:
            mask |= 1 << KERNEL_CLASSES.index(c)
        _check(self.lib.ls_profile_begin(self.h, mask, int(layer)), "ls_profile_begin")

    def profile_end(self):
        """{(class, layer): (total ms, launches)} for what ran since profile_begin()."""
        n = len(KERNEL_CLASSES) * LS_MAX_LAYERS
        ms = (C.c_double * n)()
        cnt = (C.c_int64 * n)()
        _check(self.lib.ls_profile_end(self.h, ms, cnt), "ls_profile_end")
        out = {}
        for ci, cname in enumerate(KERNEL_CLASSES):
            for l in range(LS_MAX_LAYERS):
                if cnt[ci * LS_MAX_LAYERS + l]:
                    out[(cname, l)] = (ms[ci * LS_MAX_LAYERS + l], cnt[ci * LS_MAX_LAYERS + l])
        return out

    def run_refined(self, K: int, tau_0: int, row_offsets: np.ndarray, interval: int, probe_rows: int,
                    gamma: float = 0.5, slack: int = 0, decay_at: Sequence[int] = (), decay_factor: float = 0.1,
                    loss_out=None):
        """ls_run_refined: AdaComm with the saturation decay and the learning-rate coupling (Section 4.3)."""
        offs = np.ascontiguousarray(row_offsets, dtype=np.int64)
        if offs.size != K * self.m:
            raise ValueError("row_offsets must be [K][m]")
        dec = np.ascontiguousarray(decay_at, dtype=np.int64)
        opts = AdacommOpts(float(gamma), int(slack), int(dec.size), dec.ctypes.data if dec.size else None,
                           float(decay_factor))
        max_p = int(K) + 1
        period_tau = np.zeros(max_p, dtype=np.int32)
        dk = np.zeros(max_p, dtype=np.int64)
        dF = np.zeros(max_p, dtype=np.float32)
        dt = np.zeros(max_p, dtype=np.int32)
        n_p, n_d, F0 = C.c_int64(), C.c_int64(), C.c_float()
        lp = None if loss_out is None else loss_out.data_ptr()
        _check(self.lib.ls_run_refined(self.h, int(K), int(tau_0), int(interval), int(probe_rows), offs.ctypes.data, lp,
                                       C.byref(opts), period_tau.ctypes.data, max_p, C.byref(n_p), dk.ctypes.data,
                                       dF.ctypes.data, dt.ctypes.data, max_p, C.byref(n_d), C.byref(F0)),
               "ls_run_refined")
        lr = C.c_float()
        _check(self.lib.ls_get_lr(self.h, C.byref(lr)), "ls_get_lr")
        n_p, n_d = n_p.value, n_d.value
        return {"taus": period_tau[:n_p].tolist(), "decision_k": dk[:n_d].tolist(), "decision_F": dF[:n_d].copy(),
                "decision_tau": dt[:n_d].tolist(), "F_0": float(F0.value), "lr": float(lr.value)}

    # -- one job on several GPUs ----------------------------------------------
    def shard_buffer_floats(self) -> int:
        n = C.c_int64()
        _check(self.lib.ls_shard_buffer_floats(self.h, C.byref(n)), "ls_shard_buffer_floats")
        return n.value

    def set_shard(self, n_gpus: int, m_total: int, partial=None, gathered=None, exchange=None):
        """ls_set_shard: this handle's replicas are one rank's share of a job of m_total replicas.  `exchange` is
        a Python callable (partial_ptr, gathered_ptr, nbytes, n_gpus) -> 0 on success; the buffers and the
        callback object are kept alive by this wrapper."""
        if n_gpus == 0:
            _check(self.lib.ls_set_shard(self.h, 0, 0, None, None, EXCHANGE_FN(0), None), "ls_set_shard")
            self._shard = None
            return
        cb = EXCHANGE_FN(0) if exchange is None else EXCHANGE_FN(lambda ctx, p, g, nbytes, n: int(exchange(p, g, nbytes, n)))
        _check(self.lib.ls_set_shard(self.h, int(n_gpus), int(m_total), partial.data_ptr(),
                                     None if gathered is None else gathered.data_ptr(), cb, None), "ls_set_shard")
        self._shard = (partial, gathered, cb)

    def shard_partial_sum(self, partial):
        _check(self.lib.ls_shard_partial_sum(self.h, partial.data_ptr()), "ls_shard_partial_sum")

    def shard_average(self, gathered, n_gpus: int, m_total: int):
        _check(self.lib.ls_shard_average(self.h, gathered.data_ptr(), int(n_gpus), int(m_total)), "ls_shard_average")

    def launch_count(self) -> int:
        n = C.c_int64()
        _check(self.lib.ls_launch_count(self.h, C.byref(n)), "ls_launch_count")
        return n.value
