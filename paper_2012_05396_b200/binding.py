"""ctypes binding of libssd_sgd.so: the same entry points as include/ssd_sgd.h.

Argument marshalling only.  Every step of the update path runs in the CUDA
library; there is no CPU or PyTorch fallback, and loading fails loudly when the
library has not been built (run `python -m paper_2012_05396_b200.build`).
torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libssd_sgd.so")

(SSD_OK, SSD_ERR_ARG, SSD_ERR_ALIGN, SSD_ERR_LAYOUT, SSD_ERR_STATE, SSD_ERR_CUDA, SSD_ERR_NOMEM,
 SSD_ERR_TOO_LARGE) = range(8)
SSD_STATIC_TABLE_MAX_TENSORS = 1024
SSD_F32, SSD_BF16 = 0, 1
SSD_LOCAL_GLU, SSD_LOCAL_SGD = 0, 1
SSD_STAGE_WARMUP, SSD_STAGE_DELAY = 0, 1
SSD_FLAG_FIRST, SSD_FLAG_REFRESH, SSD_FLAG_PULL, SSD_FLAG_COPY = 1, 2, 4, 8
SSD_VIEW_GLOBAL, SSD_VIEW_LOCAL, SSD_VIEW_DEVICE = 0, 1, 2
SSD_MAX_WORKERS = 32

EXPORTS = (
    "ssd_arena_numel", "ssd_init", "ssd_destroy", "ssd_tensor_offset", "ssd_schedule",
    "ssd_server_sync_update", "ssd_server_sync_update_static", "ssd_worker_glu_update", "ssd_worker_local_step", "ssd_advance",
    "ssd_step", "ssd_step_tensors", "ssd_step_host", "ssd_set_host_chunk", "ssd_set_host_pre_weight", "ssd_broadcast_weights", "ssd_worker_weights", "ssd_get_counters",
    "ssd_set_counters", "ssd_set_lr", "ssd_tensor_table_bytes", "ssd_set_tensor_scales", "ssd_get_hparams", "ssd_set_launch", "ssd_set_kernel_shape", "ssd_get_launch",
    "ssd_set_staging", "ssd_staging_error", "ssd_kernel_launches",
    "ssd_status_str", "ssd_last_cuda_error",
)


class ssd_layout(C.Structure):
    _fields_ = [("num_tensors", C.c_int32), ("numel", C.POINTER(C.c_int64))]


class ssd_hparams(C.Structure):
    _fields_ = [("K", C.c_int32), ("lr", C.c_float), ("momentum", C.c_float), ("wd", C.c_float),
                ("warmup_iters", C.c_int32), ("delay_k", C.c_int32), ("lr_local", C.c_float),
                ("alpha", C.c_float), ("beta", C.c_float), ("rescale", C.c_float),
                ("grad_dtype", C.c_int32), ("local_updater", C.c_int32)]


class ssd_buffers(C.Structure):
    _fields_ = [("w", C.c_void_p), ("mom", C.c_void_p), ("w_loc", C.POINTER(C.c_void_p)),
                ("pre", C.POINTER(C.c_void_p)), ("w_dev", C.POINTER(C.c_void_p))]


class SsdError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = f"{where}: {lib().ssd_status_str(status).decode()} (status {status})"
        super().__init__(msg + (f": {detail}" if detail else ""))


_lib = None


def lib():
    """The loaded library; raises if it is not built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2012_05396_b200.build`; there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        P = C.POINTER
        sigs = {
            "ssd_arena_numel": (i32, [P(ssd_layout), P(i64)]),
            "ssd_init": (i32, [P(vp), P(ssd_layout), P(ssd_hparams), P(ssd_buffers)]),
            "ssd_destroy": (None, [vp]),
            "ssd_tensor_offset": (i32, [vp, i32, P(i64)]),
            "ssd_schedule": (i32, [vp, i64, P(i32), P(i32)]),
            "ssd_server_sync_update": (i32, [vp, P(vp), vp]),
            "ssd_server_sync_update_static": (i32, [vp, P(vp), P(C.c_float), P(C.c_float), vp]),
            "ssd_worker_glu_update": (i32, [vp, i32, vp, i32, vp]),
            "ssd_worker_local_step": (i32, [vp, i32, vp, vp]),
            "ssd_advance": (i32, [vp]),
            "ssd_step": (i32, [vp, P(vp), vp]),
            "ssd_step_tensors": (i32, [vp, P(vp), i32, i32, vp]),
            "ssd_step_host": (i32, [vp, P(vp), P(vp), vp, vp]),
            "ssd_set_host_chunk": (i32, [vp, i64]),
            "ssd_set_host_pre_weight": (i32, [vp, vp, vp, i32]),
            "ssd_broadcast_weights": (i32, [vp, vp]),
            "ssd_worker_weights": (i32, [vp, i32, P(vp), P(i32)]),
            "ssd_get_counters": (i32, [vp, P(i64), P(i64), P(i32), P(i32)]),
            "ssd_set_counters": (i32, [vp, i64, i64]),
            "ssd_set_lr": (i32, [vp, C.c_float, C.c_float, vp]),
            "ssd_tensor_table_bytes": (i32, [vp, P(i64)]),
            "ssd_set_tensor_scales": (i32, [vp, P(C.c_float), P(C.c_float), vp, vp]),
            "ssd_get_hparams": (i32, [vp, P(ssd_hparams), P(C.c_float)]),
            "ssd_set_launch": (i32, [vp, i32, i32]),
            "ssd_set_kernel_shape": (i32, [vp, i32, i32]),
            "ssd_get_launch": (i32, [vp, P(i32), P(i32), P(i32), P(i32)]),
            "ssd_set_staging": (i32, [vp, i32]),
            "ssd_staging_error": (i32, [vp, P(i32)]),
            "ssd_kernel_launches": (i64, [vp]),
            "ssd_status_str": (C.c_char_p, [i32]),
            "ssd_last_cuda_error": (C.c_char_p, [vp]),
        }
        for name, (res, args) in sigs.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(x) -> Optional[int]:
    """Device or host address of a tensor / int / None."""
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return x.data_ptr()
    return int(x)


def _ptr_table(xs):
    if isinstance(xs, C.Array):            # already marshalled by pointer_table()
        return xs
    return (C.c_void_p * len(xs))(*[_ptr(x) for x in xs])


def pointer_table(tensors: Sequence):
    """Marshals a list of tensors / addresses once; the result can be passed wherever a list of
    gradient or staging buffers is expected, which saves the per-call conversion when the same
    buffers are used for many steps.  The caller keeps the tensors alive."""
    return _ptr_table(list(tensors))


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream
    return int(stream)


def _layout(numels: Sequence[int]):
    arr = (C.c_int64 * len(numels))(*[int(n) for n in numels])
    return ssd_layout(len(numels), arr), arr


def ssd_arena_numel(numels: Sequence[int]) -> int:
    lay, _keep = _layout(numels)
    out = C.c_int64()
    st = lib().ssd_arena_numel(C.byref(lay), C.byref(out))
    if st != SSD_OK:
        raise SsdError(st, "ssd_arena_numel")
    return out.value


def make_hparams(K: int, lr: float, momentum: float, warmup_iters: int, delay_k: int, wd: float = 0.0,
                 lr_local: float = math.nan, alpha: float = math.nan, beta: float = math.nan,
                 rescale: float = math.nan, grad_dtype: int = SSD_F32,
                 local_updater: int = SSD_LOCAL_GLU) -> ssd_hparams:
    return ssd_hparams(K, lr, momentum, wd, warmup_iters, delay_k, lr_local, alpha, beta, rescale,
                       grad_dtype, local_updater)


class Context:
    """Owner of one ssd_ctx handle.  Methods carry the names of the C entry points."""

    def __init__(self, numels: Sequence[int], hp: ssd_hparams, w, mom, w_loc: Optional[Sequence] = None,
                 pre: Optional[Sequence] = None, w_dev: Optional[Sequence] = None):
        self._h = C.c_void_p()
        self.K = hp.K
        self._keep = (w, mom, w_loc, pre, w_dev)                         # keep tensors alive
        lay, _arr = _layout(numels)
        tables = [None if t is None else _ptr_table(t) for t in (w_loc, pre, w_dev)]
        bufs = ssd_buffers(_ptr(w), _ptr(mom), *tables)
        st = lib().ssd_init(C.byref(self._h), C.byref(lay), C.byref(hp), C.byref(bufs))
        if st != SSD_OK:
            self._h = C.c_void_p()
            raise SsdError(st, "ssd_init")

    def _check(self, st: int, where: str):
        if st != SSD_OK:
            detail = lib().ssd_last_cuda_error(self._h).decode() if st == SSD_ERR_CUDA else ""
            raise SsdError(st, where, detail)

    def ssd_destroy(self):
        if self._h:
            lib().ssd_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.ssd_destroy()
        except Exception:
            pass

    def ssd_tensor_offset(self, tensor: int) -> int:
        out = C.c_int64()
        self._check(lib().ssd_tensor_offset(self._h, tensor, C.byref(out)), "ssd_tensor_offset")
        return out.value

    def ssd_schedule(self, it: int):
        stage, flags = C.c_int32(), C.c_int32()
        self._check(lib().ssd_schedule(self._h, it, C.byref(stage), C.byref(flags)), "ssd_schedule")
        return stage.value, flags.value

    def ssd_server_sync_update(self, grads: Sequence, stream=None):
        self._check(lib().ssd_server_sync_update(self._h, _ptr_table(grads), _stream(stream)),
                    "ssd_server_sync_update")

    def ssd_server_sync_update_static(self, grads: Sequence, lr_mult=None, wd_mult=None, stream=None):
        """Per-tensor server update whose table lives in the library's static device array: for
        callers that must not allocate device memory.  lr_mult / wd_mult: sequences of floats or None."""
        def arr(x):
            return None if x is None else (C.c_float * len(x))(*[float(v) for v in x])
        self._check(lib().ssd_server_sync_update_static(self._h, _ptr_table(grads), arr(lr_mult), arr(wd_mult),
                                                        _stream(stream)), "ssd_server_sync_update_static")

    def ssd_worker_glu_update(self, worker: int, grad, flags: int, stream=None):
        self._check(lib().ssd_worker_glu_update(self._h, worker, _ptr(grad), flags, _stream(stream)),
                    "ssd_worker_glu_update")

    def ssd_worker_local_step(self, worker: int, grad, stream=None):
        self._check(lib().ssd_worker_local_step(self._h, worker, _ptr(grad), _stream(stream)),
                    "ssd_worker_local_step")

    def ssd_advance(self):
        self._check(lib().ssd_advance(self._h), "ssd_advance")

    def ssd_step(self, grads: Sequence, stream=None):
        self._check(lib().ssd_step(self._h, _ptr_table(grads), _stream(stream)), "ssd_step")

    def ssd_step_tensors(self, grads: Sequence, first_tensor: int, num_tensors: int, stream=None):
        self._check(lib().ssd_step_tensors(self._h, _ptr_table(grads), first_tensor, num_tensors,
                                           _stream(stream)), "ssd_step_tensors")

    def ssd_step_host(self, host_grads: Optional[Sequence], staging: Sequence, host_w_out=None, stream=None):
        """host_grads None: the gradients are already in `staging` (device memory)."""
        self._check(lib().ssd_step_host(self._h, None if host_grads is None else _ptr_table(host_grads),
                                        _ptr_table(staging), _ptr(host_w_out), _stream(stream)), "ssd_step_host")

    def ssd_set_host_chunk(self, chunk_elems: int = 0):
        self._check(lib().ssd_set_host_chunk(self._h, chunk_elems), "ssd_set_host_chunk")

    def ssd_set_host_pre_weight(self, host_pre, device_slices, slots: int):
        """host_pre: pinned host tensor / address; device_slices: device tensor / address; (None, None, 0) = off."""
        self._host_pre = (host_pre, device_slices)       # keep the tensors alive
        self._check(lib().ssd_set_host_pre_weight(self._h, _ptr(host_pre), _ptr(device_slices), slots),
                    "ssd_set_host_pre_weight")

    def ssd_broadcast_weights(self, stream=None):
        self._check(lib().ssd_broadcast_weights(self._h, _stream(stream)), "ssd_broadcast_weights")

    def ssd_worker_weights(self, worker: int):
        """(device address, view code) of the weights worker `worker` computes on next."""
        p, v = C.c_void_p(), C.c_int32()
        self._check(lib().ssd_worker_weights(self._h, worker, C.byref(p), C.byref(v)), "ssd_worker_weights")
        return p.value, v.value

    def ssd_get_counters(self):
        """(iter, loc_update, next_stage, next_flags)"""
        it, lu, st, fl = C.c_int64(), C.c_int64(), C.c_int32(), C.c_int32()
        self._check(lib().ssd_get_counters(self._h, C.byref(it), C.byref(lu), C.byref(st), C.byref(fl)),
                    "ssd_get_counters")
        return it.value, lu.value, st.value, fl.value

    def ssd_set_counters(self, it: int, loc_update: int):
        self._check(lib().ssd_set_counters(self._h, it, loc_update), "ssd_set_counters")

    def ssd_set_lr(self, lr: float = math.nan, lr_local: float = math.nan, stream=None):
        self._check(lib().ssd_set_lr(self._h, lr, lr_local, _stream(stream)), "ssd_set_lr")

    def ssd_tensor_table_bytes(self) -> int:
        out = C.c_int64()
        self._check(lib().ssd_tensor_table_bytes(self._h, C.byref(out)), "ssd_tensor_table_bytes")
        return out.value

    def ssd_set_tensor_scales(self, lr_mult, wd_mult, device_table, stream=None):
        """lr_mult / wd_mult: sequences of floats or None; device_table: tensor / address / None."""
        def arr(x):
            return None if x is None else (C.c_float * len(x))(*[float(v) for v in x])
        self._table = device_table                       # keep the tensor alive
        self._check(lib().ssd_set_tensor_scales(self._h, arr(lr_mult), arr(wd_mult), _ptr(device_table),
                                                _stream(stream)), "ssd_set_tensor_scales")

    def ssd_get_hparams(self):
        hp, c = ssd_hparams(), C.c_float()
        self._check(lib().ssd_get_hparams(self._h, C.byref(hp), C.byref(c)), "ssd_get_hparams")
        return hp, c.value

    def ssd_set_launch(self, threads_per_block: int = 0, blocks_per_sm: int = 0):
        self._check(lib().ssd_set_launch(self._h, threads_per_block, blocks_per_sm), "ssd_set_launch")

    def ssd_set_kernel_shape(self, vector_elems: int = 0, batch: int = 0):
        self._check(lib().ssd_set_kernel_shape(self._h, vector_elems, batch), "ssd_set_kernel_shape")

    def ssd_get_launch(self):
        """(threads_per_block, blocks_per_sm, vector_elems, batch) overrides, 0 = default"""
        v = [C.c_int32() for _ in range(4)]
        self._check(lib().ssd_get_launch(self._h, *[C.byref(x) for x in v]), "ssd_get_launch")
        return tuple(x.value for x in v)

    def ssd_set_staging(self, stages: int = 0):
        self._check(lib().ssd_set_staging(self._h, stages), "ssd_set_staging")

    def ssd_staging_error(self) -> int:
        out = C.c_int32()
        self._check(lib().ssd_staging_error(self._h, C.byref(out)), "ssd_staging_error")
        return out.value

    def ssd_kernel_launches(self) -> int:
        return lib().ssd_kernel_launches(self._h)
