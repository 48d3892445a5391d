"""ctypes binding of libcada.so: the same entry points as include/cada.h, argument marshalling only.

Every step of the method runs inside the library's CUDA kernels; this module moves pointers.
torch is used for device memory (workspace, data) and for the stream handle.  Loading fails
loudly if the shared library has not been built (``python -m paper_2012_15469_b200.build``):
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcada.so")

CADA_ABI_VERSION = 3
CADA_OK = 0
CADA_ERR_INVALID_ARG, CADA_ERR_UNSUPPORTED, CADA_ERR_WORKSPACE = -1, -2, -3
CADA_ERR_CUDA, CADA_ERR_NONFINITE, CADA_ERR_TIMEOUT = -4, -5, -6
CADA_MODEL_LOGISTIC, CADA_MODEL_SOFTMAX, CADA_MODEL_MLP2 = 0, 1, 2
CADA_RULE_CADA1, CADA_RULE_CADA2, CADA_RULE_LAG = 1, 2, 3
CADA_SERVER_AMSGRAD, CADA_SERVER_SGD = 0, 1
CADA_AGG_SLOTS, CADA_AGG_RECURSIVE = 0, 1
CADA_X_F32, CADA_X_BF16 = 0, 1
CADA_FLAG_NONFINITE, CADA_FLAG_BAD_INDEX, CADA_FLAG_TIMEOUT = 1, 2, 4
CADA_PATH_THREE_KERNELS, CADA_PATH_ONE_LAUNCH_GRID, CADA_PATH_ONE_LAUNCH_CLUSTER, CADA_PATH_SOFTMAX_CLUSTER = 0, 1, 2, 3
CADA_PATH_MLP_CLUSTER = 4
CADA_PATH_MLP_HIDDEN_SPLIT = 5
(CADA_BUF_THETA, CADA_BUF_H, CADA_BUF_VHAT, CADA_BUF_G, CADA_BUF_THETA_HAT, CADA_BUF_DELTA_STORED,
 CADA_BUF_THETA_TILDE, CADA_BUF_TAU, CADA_BUF_RING, CADA_BUF_GRAD_FRESH, CADA_BUF_INNOV_FRESH,
 CADA_BUF_LAST_LHS, CADA_BUF_LAST_MASK, CADA_BUF_UPLOADS_PER_WORKER, CADA_BUF_HIST_LHS,
 CADA_BUF_HIST_RHS, CADA_BUF_HIST_MASK, CADA_BUF_K, CADA_BUF_MLP_Z1, CADA_BUF_NABLA, CADA_BUF_MLP_DZ1,
 CADA_BUF_MLP_DZ2) = range(22)

EXPORTS = ["cada_workspace_bytes", "cada_create", "cada_step", "cada_step_host", "cada_set_indices",
           "cada_stats", "cada_read", "cada_write", "cada_profile", "cada_destroy", "cada_last_error",
           "cada_server_update_noalloc", "cada_eval", "cada_set_wait_limit", "cada_step_host_n",
           "cada_step_local", "cada_step_apply"]
CADA_NOALLOC_MAX_P = 1 << 22


class cada_config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("abi_version", C.c_uint32),
        ("model", C.c_int32), ("rule", C.c_int32),
        ("p", C.c_int64),
        ("M", C.c_int32), ("batch", C.c_int32),
        ("alpha", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
        ("c", C.c_float),
        ("d_max", C.c_int32), ("D", C.c_int32),
        ("lambda_", C.c_float),
        ("n_features", C.c_int32), ("n_classes", C.c_int32), ("n_hidden", C.c_int32),
        ("has_bias", C.c_int32), ("x_dtype", C.c_int32), ("history_capacity", C.c_int32),
        ("host_step_rows", C.c_int32), ("server", C.c_int32),
        ("ldx", C.c_int64),
        ("X", C.POINTER(C.c_void_p)), ("y", C.POINTER(C.c_void_p)),
        ("n_samples", C.POINTER(C.c_int64)),
        ("theta0", C.c_void_p),
        ("tau0", C.POINTER(C.c_int32)),
        ("seed", C.c_uint64),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("stream", C.c_void_p),
        ("aggregate", C.c_int32), ("alpha_K0", C.c_float),
        ("batch_m", C.POINTER(C.c_int32)),
        ("M_total", C.c_int32), ("m_first", C.c_int32), ("m_stride", C.c_int32), ("reserved0", C.c_int32),
    ]


class cada_stats_t(C.Structure):
    _fields_ = [
        ("k", C.c_int64), ("uploads_total", C.c_int64), ("uploads_forced", C.c_int64),
        ("uploads_rule", C.c_int64), ("near_ties", C.c_int64), ("kernel_launches", C.c_int64),
        ("last_rhs", C.c_double), ("last_step_sqnorm", C.c_double),
        ("grad_kernel_ms", C.c_double), ("grad_kernel_launches", C.c_int64), ("profiled_iterations", C.c_int64),
        ("status_flags", C.c_int32), ("path", C.c_int32),
    ]


_lib = None


def load_library() -> C.CDLL:
    """dlopen libcada.so and declare the prototypes; raises if the library is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2012_15469_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    H = C.c_void_p
    lib.cada_workspace_bytes.restype = C.c_size_t
    lib.cada_workspace_bytes.argtypes = [C.POINTER(cada_config)]
    lib.cada_create.restype = C.c_int
    lib.cada_create.argtypes = [C.POINTER(cada_config), C.POINTER(H)]
    lib.cada_step.restype = C.c_int
    lib.cada_step.argtypes = [H, C.c_int32]
    lib.cada_step_host.restype = C.c_int
    lib.cada_step_host.argtypes = [H, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.cada_step_local.restype = C.c_int
    lib.cada_step_local.argtypes = [H, C.c_void_p]
    lib.cada_step_apply.restype = C.c_int
    lib.cada_step_apply.argtypes = [H, C.c_void_p]
    lib.cada_step_host_n.restype = C.c_int
    lib.cada_step_host_n.argtypes = [H, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.cada_set_indices.restype = C.c_int
    lib.cada_set_indices.argtypes = [H, C.c_void_p, C.c_int32]
    lib.cada_stats.restype = C.c_int
    lib.cada_stats.argtypes = [H, C.POINTER(cada_stats_t)]
    lib.cada_read.restype = C.c_int
    lib.cada_read.argtypes = [H, C.c_int32, C.c_void_p, C.c_size_t]
    lib.cada_write.restype = C.c_int
    lib.cada_write.argtypes = [H, C.c_int32, C.c_void_p, C.c_size_t]
    lib.cada_profile.restype = C.c_int
    lib.cada_profile.argtypes = [H, C.c_int32]
    lib.cada_server_update_noalloc.restype = C.c_int
    lib.cada_server_update_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_float,
                                               C.c_float, C.c_float, C.c_float, C.c_void_p, C.c_void_p]
    lib.cada_set_wait_limit.restype = C.c_int
    lib.cada_set_wait_limit.argtypes = [H, C.c_int64]
    lib.cada_eval.restype = C.c_int
    lib.cada_eval.argtypes = [H, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.cada_destroy.restype = C.c_int
    lib.cada_destroy.argtypes = [H]
    lib.cada_last_error.restype = C.c_char_p
    lib.cada_last_error.argtypes = [H]
    _lib = lib
    return lib


class CadaError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"libcada error {code}: {message}")
        self.code = code


# -- thin wrappers with the C names ----------------------------------------------------------------

def cada_workspace_bytes(cfg: cada_config) -> int:
    return int(load_library().cada_workspace_bytes(C.byref(cfg)))


def cada_create(cfg: cada_config) -> C.c_void_p:
    lib = load_library()
    h = C.c_void_p()
    rc = lib.cada_create(C.byref(cfg), C.byref(h))
    if rc != CADA_OK:
        raise CadaError(rc, lib.cada_last_error(None).decode())
    return h


def _check(h, rc):
    if rc != CADA_OK:
        raise CadaError(rc, load_library().cada_last_error(h).decode())


def cada_step(h, n_iters: int) -> None:
    _check(h, load_library().cada_step(h, n_iters))


def cada_step_local(h, dev_sum_out_ptr: int) -> None:
    _check(h, load_library().cada_step_local(h, dev_sum_out_ptr or None))


def cada_step_apply(h, dev_sum_ptr: int) -> None:
    _check(h, load_library().cada_step_apply(h, dev_sum_ptr or None))


def cada_step_host(h, host_X_ptr: int, host_y_ptr: int, host_theta_out_ptr: int = 0, host_mask_out_ptr: int = 0) -> None:
    _check(h, load_library().cada_step_host(h, host_X_ptr, host_y_ptr, host_theta_out_ptr or None, host_mask_out_ptr or None))


def cada_step_host_n(h, n: int, host_X_ptr: int, host_y_ptr: int, host_theta_out_ptr: int = 0, host_mask_out_ptr: int = 0) -> None:
    _check(h, load_library().cada_step_host_n(h, n, host_X_ptr, host_y_ptr, host_theta_out_ptr or None, host_mask_out_ptr or None))


def cada_set_indices(h, dev_idx_ptr: int, n_iters: int) -> None:
    _check(h, load_library().cada_set_indices(h, dev_idx_ptr or None, n_iters))


def cada_stats(h) -> cada_stats_t:
    """The counters; ``.rc`` carries the call's status: CADA_OK, or CADA_ERR_TIMEOUT / CADA_ERR_NONFINITE when the device
    has raised that flag (the structure is filled in either case).  Any other status raises."""
    s = cada_stats_t()
    rc = load_library().cada_stats(h, C.byref(s))
    if rc not in (CADA_OK, CADA_ERR_TIMEOUT, CADA_ERR_NONFINITE):
        _check(h, rc)
    s.rc = rc
    return s


def cada_set_wait_limit(h, polls: int) -> None:
    _check(h, load_library().cada_set_wait_limit(h, polls))


def cada_read(h, which: int, dst: np.ndarray) -> np.ndarray:
    assert dst.flags["C_CONTIGUOUS"]
    _check(h, load_library().cada_read(h, which, dst.ctypes.data, dst.nbytes))
    return dst


def cada_write(h, which: int, src: np.ndarray) -> None:
    src = np.ascontiguousarray(src)
    _check(h, load_library().cada_write(h, which, src.ctypes.data, src.nbytes))


def cada_profile(h, enable: bool) -> None:
    _check(h, load_library().cada_profile(h, 1 if enable else 0))


def cada_server_update_noalloc(theta_ptr: int, h_ptr: int, vhat_ptr: int, nabla_ptr: int, p: int, alpha: float,
                               beta1: float, beta2: float, eps: float, step_sqnorm_out_ptr: int, stream_ptr: int) -> int:
    """Eqs. 2a-2c in place on device vectors, using only the library's built-in scratch (no allocation).
    Returns the status code; the caller owns every buffer."""
    return int(load_library().cada_server_update_noalloc(theta_ptr or None, h_ptr or None, vhat_ptr or None,
                                                         nabla_ptr or None, p, alpha, beta1, beta2, eps,
                                                         step_sqnorm_out_ptr or None, stream_ptr or None))


def cada_eval(h):
    """(loss of Eq. 1, accuracy) over all rows of all workers at the current iterate."""
    loss, acc = C.c_double(), C.c_double()
    _check(h, load_library().cada_eval(h, C.byref(loss), C.byref(acc)))
    return loss.value, acc.value


def cada_destroy(h) -> None:
    load_library().cada_destroy(h)


# -- convenience object: owns the torch workspace and keeps the data tensors alive ---------------

_BUF_SHAPES = {
    CADA_BUF_THETA: ("p", np.float32), CADA_BUF_H: ("p", np.float32), CADA_BUF_VHAT: ("p", np.float32),
    CADA_BUF_G: ("Mp", np.float32), CADA_BUF_THETA_HAT: ("Mp", np.float32),
    CADA_BUF_DELTA_STORED: ("Mp", np.float32), CADA_BUF_THETA_TILDE: ("p", np.float32),
    CADA_BUF_TAU: ("M", np.int32), CADA_BUF_RING: ("d", np.float64),
    CADA_BUF_GRAD_FRESH: ("Mp", np.float32), CADA_BUF_INNOV_FRESH: ("Mp", np.float32),
    CADA_BUF_LAST_LHS: ("M", np.float64), CADA_BUF_LAST_MASK: ("M", np.uint8),
    CADA_BUF_UPLOADS_PER_WORKER: ("M", np.int64), CADA_BUF_HIST_LHS: ("HM", np.float64),
    CADA_BUF_HIST_RHS: ("H", np.float64), CADA_BUF_HIST_MASK: ("HM", np.uint8), CADA_BUF_K: ("1", np.int64),
    CADA_BUF_MLP_Z1: ("Z1", np.float32), CADA_BUF_NABLA: ("p", np.float32),
    CADA_BUF_MLP_DZ1: ("Z1", np.float32), CADA_BUF_MLP_DZ2: ("Z2", np.float32),
}


class Cada:
    """A CADA run on the current CUDA device.

    ``X`` and ``y`` are lists of per-worker torch CUDA tensors ([n_m, ldx] features, [n_m]
    labels); ``theta0`` a CUDA float tensor [p].  Hyper-parameters carry the paper's names.
    """

    def __init__(self, *, model: int, rule: int, X: Sequence, y: Sequence, theta0, batch: int, alpha: float,
                 beta1: float, beta2: float, eps: float, c: float, d_max: int, D: int, lam: float = 0.0,
                 n_features: int, n_classes: int = 1, n_hidden: int = 0, has_bias: int = 0, seed: int = 0,
                 tau0: Optional[Sequence[int]] = None, history_capacity: int = 0, host_step: bool = False,
                 stream=None, server: int = 0, aggregate: int = 0, alpha_K0: float = 0.0,
                 batch_m: Optional[Sequence[int]] = None, M_total: int = 0, m_first: int = 0, m_stride: int = 0):
        import torch

        self._torch = torch
        M = len(X)
        self.M, self.batch, self.d_max, self.history_capacity = M, batch, d_max, history_capacity
        self.n_hidden, self.n_classes = n_hidden, n_classes
        self._keep = (list(X), list(y), theta0)
        bf16 = X[0].dtype == torch.bfloat16
        for t in list(X) + list(y) + [theta0]:
            assert t.is_cuda and t.is_contiguous()
        cfg = cada_config()
        cfg.struct_size = C.sizeof(cada_config)
        cfg.abi_version = CADA_ABI_VERSION
        cfg.model, cfg.rule = model, rule
        cfg.M, cfg.batch = M, batch
        cfg.alpha, cfg.beta1, cfg.beta2, cfg.eps = alpha, beta1, beta2, eps
        cfg.c = c
        cfg.d_max, cfg.D = d_max, D
        cfg.lambda_ = lam
        cfg.n_features, cfg.n_classes, cfg.n_hidden, cfg.has_bias = n_features, n_classes, n_hidden, has_bias
        cfg.x_dtype = CADA_X_BF16 if bf16 else CADA_X_F32
        cfg.history_capacity = history_capacity
        cfg.host_step_rows = batch if host_step else 0
        cfg.server = server
        cfg.aggregate, cfg.alpha_K0 = aggregate, alpha_K0
        cfg.M_total, cfg.m_first, cfg.m_stride = M_total, m_first, m_stride
        if batch_m is not None:
            self._batch_m = (C.c_int32 * M)(*[int(b) for b in batch_m])
            cfg.batch_m = C.cast(self._batch_m, C.POINTER(C.c_int32))
        cfg.ldx = X[0].shape[1]
        cfg.p = int(theta0.numel())
        self.p = cfg.p
        self._xptr = (C.c_void_p * M)(*[t.data_ptr() for t in X])
        self._yptr = (C.c_void_p * M)(*[t.data_ptr() for t in y])
        self._ns = (C.c_int64 * M)(*[int(t.shape[0]) for t in X])
        cfg.X = C.cast(self._xptr, C.POINTER(C.c_void_p))
        cfg.y = C.cast(self._yptr, C.POINTER(C.c_void_p))
        cfg.n_samples = C.cast(self._ns, C.POINTER(C.c_int64))
        cfg.theta0 = theta0.data_ptr()
        if tau0 is not None:
            self._tau0 = (C.c_int32 * M)(*[int(t) for t in tau0])
            cfg.tau0 = C.cast(self._tau0, C.POINTER(C.c_int32))
        cfg.seed = seed
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        cfg.stream = self.stream.cuda_stream
        need = cada_workspace_bytes(cfg)
        if need == 0:
            # let cada_create produce the message
            cfg.workspace, cfg.workspace_bytes = 0, 0
            cada_create(cfg)
            raise CadaError(CADA_ERR_INVALID_ARG, "invalid configuration")
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=theta0.device)
        base = self.workspace.data_ptr()
        cfg.workspace = (base + 255) // 256 * 256
        cfg.workspace_bytes = need
        self.workspace_bytes = need
        self.cfg = cfg
        self.handle = cada_create(cfg)
        self._idx_keep = None

    # mirrors of the C entry points
    def step(self, n_iters: int = 1) -> None:
        cada_step(self.handle, n_iters)

    def step_local(self, dev_sum_out) -> None:
        """Worker side for this handle's workers; their part of the server's sum goes to the CUDA float tensor [p]."""
        assert dev_sum_out.is_cuda and dev_sum_out.dtype == self._torch.float32 and dev_sum_out.numel() == self.p
        cada_step_local(self.handle, dev_sum_out.data_ptr())

    def step_apply(self, dev_sum) -> None:
        """Server side from the sum over ALL handles (CUDA float tensor [p])."""
        assert dev_sum.is_cuda and dev_sum.dtype == self._torch.float32 and dev_sum.numel() == self.p
        cada_step_apply(self.handle, dev_sum.data_ptr())

    def step_host(self, host_X, host_y, host_theta_out=None, host_mask_out=None) -> None:
        cada_step_host(self.handle, host_X.data_ptr(), host_y.data_ptr(),
                       host_theta_out.data_ptr() if host_theta_out is not None else 0,
                       host_mask_out.data_ptr() if host_mask_out is not None else 0)

    def step_host_n(self, n: int, host_X, host_y, host_theta_out=None, host_mask_out=None) -> None:
        """host_X [n, M, batch, ldx], host_y [n, M, batch] (pinned CPU tensors); outputs [n, p] and [n, M]."""
        cada_step_host_n(self.handle, n, host_X.data_ptr(), host_y.data_ptr(),
                         host_theta_out.data_ptr() if host_theta_out is not None else 0,
                         host_mask_out.data_ptr() if host_mask_out is not None else 0)

    def set_indices(self, dev_idx) -> None:
        """dev_idx: CUDA int32 tensor [n_iters, M, batch] (or None to return to the hashed stream)."""
        if dev_idx is None:
            cada_set_indices(self.handle, 0, 0)
            self._idx_keep = None
            return
        assert dev_idx.is_cuda and dev_idx.dtype == self._torch.int32 and dev_idx.is_contiguous()
        assert tuple(dev_idx.shape[1:]) == (self.M, self.batch)
        self._idx_keep = dev_idx
        cada_set_indices(self.handle, dev_idx.data_ptr(), int(dev_idx.shape[0]))

    def eval(self):
        return cada_eval(self.handle)

    def stats(self) -> cada_stats_t:
        return cada_stats(self.handle)

    def set_wait_limit(self, polls: int) -> None:
        cada_set_wait_limit(self.handle, polls)

    def profile(self, enable: bool) -> None:
        cada_profile(self.handle, enable)

    def _shape(self, which):
        kind, dt = _BUF_SHAPES[which]
        shp = {"p": (self.p,), "Mp": (self.M, self.p), "M": (self.M,), "d": (self.d_max,), "1": (1,),
               "HM": (self.history_capacity, self.M), "H": (self.history_capacity,),
               "Z1": (self.M, 2, self.batch, self.n_hidden), "Z2": (self.M, 2, self.batch, self.n_classes)}[kind]
        return shp, dt

    def read(self, which: int) -> np.ndarray:
        shp, dt = self._shape(which)
        return cada_read(self.handle, which, np.empty(shp, dtype=dt))

    def write(self, which: int, value: np.ndarray) -> None:
        shp, dt = self._shape(which)
        value = np.ascontiguousarray(value, dtype=dt).reshape(shp)
        cada_write(self.handle, which, value)

    def close(self) -> None:
        if self.handle is not None:
            cada_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
