"""ctypes wrapper around the CPU oracle (ssd_oracle.c).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline may import this package; the CUDA library and its Python binding never
do.  The wrapper only marshals numpy arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ssd_oracle.c")
_BUILD = os.path.join(_HERE, "_build")

STAGE_WARMUP, STAGE_DELAY = 0, 1
F_FIRST, F_REFRESH, F_PULL, F_COPY = 1, 2, 4, 8
VIEW_GLOBAL, VIEW_LOCAL, VIEW_DEVICE = 0, 1, 2

CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c99", "-fPIC", "-shared"]


def build(force: bool = False) -> None:
    """Compile the float32 oracle and its float64 shadow with gcc."""
    os.makedirs(_BUILD, exist_ok=True)
    for name, extra in (("libssd_oracle_f32.so", []), ("libssd_oracle_f64.so", ["-DORACLE_DOUBLE"])):
        out = os.path.join(_BUILD, name)
        if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(_SRC):
            tmp = out + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", *CFLAGS, *extra, "-o", tmp, _SRC])
            os.replace(tmp, out)


class _HP(C.Structure):
    _fields_ = [("K", C.c_int32), ("grad_bf16", C.c_int32), ("W", C.c_int64), ("k", C.c_int64),
                ("lr", C.c_float), ("m", C.c_float), ("wd", C.c_float),
                ("lr_loc", C.c_float), ("alpha", C.c_float), ("beta", C.c_float),
                ("rescale", C.c_float), ("T", C.c_int32), ("tensor_end", C.c_void_p),
                ("lr_mult", C.c_void_p), ("wd_mult", C.c_void_p), ("arena_index", C.c_void_p),
                ("local_sgd", C.c_int32)]


class _State(C.Structure):
    _fields_ = [("N", C.c_int64), ("w", C.c_void_p), ("mom", C.c_void_p),
                ("w_loc", C.POINTER(C.c_void_p)), ("pre", C.POINTER(C.c_void_p)),
                ("w_dev", C.POINTER(C.c_void_p)), ("iter", C.c_int64), ("loc_update", C.c_int64)]


_libs = {}


def _lib(double: bool):
    if double not in _libs:
        build()
        _libs[double] = bind(os.path.join(_BUILD, "libssd_oracle_f64.so" if double else "libssd_oracle_f32.so"),
                             double)
    return _libs[double]


def bind(path: str, double: bool):
    """Loads one build of ssd_oracle.c and declares its signatures."""
    lib = C.CDLL(path)
    lib.oracle_sync_scale.restype = C.c_double if double else C.c_float
    lib.oracle_sync_scale.argtypes = [C.POINTER(_HP)]
    lib.oracle_schedule.restype = None
    lib.oracle_schedule.argtypes = [C.c_int64, C.c_int64, C.c_int64,
                                    C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.oracle_server_update.restype = None
    lib.oracle_server_update.argtypes = [C.c_int64, C.POINTER(_HP), C.POINTER(C.c_void_p),
                                         C.c_void_p, C.c_void_p]
    lib.oracle_glu_update.restype = None
    lib.oracle_glu_update.argtypes = [C.c_int64, C.POINTER(_HP), C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]
    lib.oracle_step.restype = C.c_int32
    lib.oracle_step.argtypes = [C.POINTER(_State), C.POINTER(_HP), C.POINTER(C.c_void_p),
                                C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.oracle_real_bytes.restype = C.c_int32
    assert lib.oracle_real_bytes() == (8 if double else 4)
    return lib


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def _ptr_array(arrs: Sequence[np.ndarray]):
    return (C.c_void_p * len(arrs))(*[_ptr(a) for a in arrs])


class Hyper:
    """The hyper-parameters of Table 1 plus the GLU coefficients (Section 4.1 defaults:
    lr_loc = 4*lr, alpha = 2.0, beta = 0.5) and the schedule (W warm-up iterations, k delay steps)."""

    def __init__(self, K: int, lr: float, m: float, W: int, k: int, wd: float = 0.0,
                 lr_loc: Optional[float] = None, alpha: float = 2.0, beta: float = 0.5,
                 rescale: Optional[float] = None, grad_bf16: bool = False, local_sgd: bool = False):
        f32 = np.float32
        self.local_sgd = bool(local_sgd)        # workers update with plain SGD (Eq. 5) instead of GLU
        self.K, self.W, self.k = int(K), int(W), int(k)
        self.lr, self.m, self.wd = f32(lr), f32(m), f32(wd)
        self.lr_loc = f32(4.0) * f32(lr) if lr_loc is None else f32(lr_loc)
        self.alpha, self.beta = f32(alpha), f32(beta)
        self.rescale = f32(1.0 / K) if rescale is None else f32(rescale)
        self.grad_bf16 = bool(grad_bf16)
        self.tensor_end = self.lr_mult = self.wd_mult = self.arena_index = None

    def set_tensor_scales(self, tensor_end, lr_mult, wd_mult, arena_index=None) -> None:
        """Per-tensor multipliers: tensor t covers arena positions up to tensor_end[t] (exclusive,
        padding included).  arena_index maps local elements to arena positions for sampled runs."""
        self.tensor_end = np.ascontiguousarray(tensor_end, dtype=np.int64)
        self.lr_mult = np.ascontiguousarray(lr_mult, dtype=np.float32)
        self.wd_mult = np.ascontiguousarray(wd_mult, dtype=np.float32)
        assert self.tensor_end.shape == self.lr_mult.shape == self.wd_mult.shape
        self.arena_index = None if arena_index is None else np.ascontiguousarray(arena_index, dtype=np.int64)

    def c_struct(self) -> _HP:
        T = 0 if self.tensor_end is None else len(self.tensor_end)
        ptr = lambda a: None if a is None else a.ctypes.data
        return _HP(self.K, int(self.grad_bf16), self.W, self.k, float(self.lr), float(self.m),
                   float(self.wd), float(self.lr_loc), float(self.alpha), float(self.beta),
                   float(self.rescale), T, ptr(self.tensor_end), ptr(self.lr_mult), ptr(self.wd_mult),
                   ptr(self.arena_index), int(self.local_sgd))


def schedule(n: int, W: int, k: int):
    """(stage, flags) of 0-based iteration n."""
    st, fl = C.c_int32(), C.c_int32()
    _lib(False).oracle_schedule(n, W, k, C.byref(st), C.byref(fl))
    return st.value, fl.value


def sync_scale(hp: Hyper, double: bool = False) -> float:
    return _lib(double).oracle_sync_scale(C.byref(hp.c_struct()))


def _check_grad(g: np.ndarray, hp: Hyper, N: int) -> None:
    assert g.dtype == (np.uint16 if hp.grad_bf16 else np.float32) and g.shape == (N,)


def server_update(hp: Hyper, grads: Sequence[np.ndarray], w: np.ndarray, mom: np.ndarray) -> None:
    """In place on w and mom (float32 arrays, or float64 for the shadow build)."""
    double = w.dtype == np.float64
    N = w.shape[0]
    assert len(grads) == hp.K and mom.dtype == w.dtype and mom.shape == w.shape
    for g in grads:
        _check_grad(g, hp, N)
    _lib(double).oracle_server_update(N, C.byref(hp.c_struct()), _ptr_array(grads), _ptr(w), _ptr(mom))


def glu_update(hp: Hyper, grad: np.ndarray, w_loc: np.ndarray, pre: np.ndarray,
               w_dev: np.ndarray, w_server: Optional[np.ndarray], flags: int) -> None:
    """In place on w_loc, pre and (on pull) w_dev."""
    double = w_loc.dtype == np.float64
    N = w_loc.shape[0]
    _check_grad(grad, hp, N)
    for a in (pre, w_dev):
        assert a.dtype == w_loc.dtype and a.shape == w_loc.shape
    if flags & F_PULL:
        assert w_server is not None and w_server.dtype == w_loc.dtype
    _lib(double).oracle_glu_update(N, C.byref(hp.c_struct()), _ptr(grad), _ptr(w_loc), _ptr(pre),
                                   _ptr(w_dev), _ptr(w_server) if w_server is not None else None,
                                   flags)


class State:
    """Server state, K workers' state and the two counters, as numpy arrays."""

    def __init__(self, hp: Hyper, w0: np.ndarray, double: bool = False, fill: float = np.nan):
        dt = np.float64 if double else np.float32
        self.hp, self.double = hp, double
        self.N = int(w0.shape[0])
        self.w = w0.astype(dt).copy()
        self.mom = np.zeros(self.N, dt)
        # Algorithm 1 initialises every worker by pulling w_0.
        self.w_loc = [self.w.copy() for _ in range(hp.K)]
        self.pre = [np.full(self.N, fill, dt) for _ in range(hp.K)]
        self.w_dev = [np.full(self.N, fill, dt) for _ in range(hp.K)]
        self.iter = 0
        self.loc_update = 0
        self.view = VIEW_GLOBAL

    def step(self, grads: Sequence[np.ndarray]):
        """One iteration; returns (stage, flags)."""
        hp = self.hp
        assert len(grads) == hp.K
        for g in grads:
            _check_grad(g, hp, self.N)
        wl, pr, wd = _ptr_array(self.w_loc), _ptr_array(self.pre), _ptr_array(self.w_dev)
        st = _State(self.N, _ptr(self.w), _ptr(self.mom), wl, pr, wd, self.iter, self.loc_update)
        stage, view = C.c_int32(), C.c_int32()
        flags = _lib(self.double).oracle_step(C.byref(st), C.byref(hp.c_struct()), _ptr_array(grads),
                                              C.byref(stage), C.byref(view))
        self.iter, self.loc_update, self.view = st.iter, st.loc_update, view.value
        return stage.value, flags

    def worker_weights(self, i: int) -> np.ndarray:
        """The buffer worker i computes its next gradient on."""
        return (self.w, self.w_loc[i], self.w_dev[i])[self.view]
