"""Thin Python binding of libef21 (argument marshalling only).

PyTorch is used for device memory, streams and host<->device copies; every
step of the EF21 hot path runs inside the CUDA library.  There is no CPU or
PyTorch fallback: if ``libef21.so`` has not been built (``python -m
paper_2106_05203_b200.build``) importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libef21.so")

EF21_OK = 0
STATUS_NAMES = {0: "EF21_OK", 1: "EF21_ERR_INVALID_ARG", 2: "EF21_ERR_STATE", 3: "EF21_ERR_WORKSPACE",
                4: "EF21_ERR_CUDA", 5: "EF21_ERR_TIMEOUT", 6: "EF21_ERR_NONFINITE", 7: "EF21_ERR_UNSUPPORTED"}
INIT_COMPRESSED, INIT_ZERO, INIT_GRADIENT = 0, 1, 2
PATH_AUTO, PATH_LAUNCHES, PATH_PERSISTENT = 0, 1, 2
VARIANT_EF21, VARIANT_EF21_PLUS, VARIANT_EF = 0, 1, 2
OBJECTIVE_LOGISTIC, OBJECTIVE_LEAST_SQUARES = 0, 1

# name -> (restype, argtypes); mirrors include/ef21.h
_i32, _i64, _f32, _sz, _vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t, ctypes.c_void_p
_dp = ctypes.POINTER(ctypes.c_double)
SIGNATURES = {
    "ef21_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "ef21_workspace_bytes": (_sz, [_i32, _i64, _i32, _i64]),
    "ef21_create": (ctypes.c_int, [ctypes.POINTER(_vp), _i32, _i64, _i32, _f32, _f32, _i64, _vp, _sz, _vp]),
    "ef21_destroy": (None, [_vp]),
    "ef21_load_shards": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "ef21_load_shards_host": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "ef21_set_x": (ctypes.c_int, [_vp, _vp]),
    "ef21_init": (ctypes.c_int, [_vp, _i32]),
    "ef21_init_grads": (ctypes.c_int, [_vp, _vp, _i32]),
    "ef21_step": (ctypes.c_int, [_vp, _i32]),
    "ef21_step_grads": (ctypes.c_int, [_vp, _vp, _i32]),
    "ef21_step_minibatch": (ctypes.c_int, [_vp, _vp, _i32]),
    "ef21_step_minibatches": (ctypes.c_int, [_vp, _vp, _i32, _i32]),
    "ef21_step_randk": (ctypes.c_int, [_vp, _vp, _vp, _i32]),
    "ef21_local_grads": (ctypes.c_int, [_vp, _vp]),
    "ef21_topk_workspace_bytes": (_sz, [_i32, _i64, _i32]),
    "ef21_topk": (ctypes.c_int, [_vp, _i32, _i64, _i32, _vp, _vp, _vp, _sz, _vp]),
    "ef21_topk_static": (ctypes.c_int, [_vp, _i32, _i64, _i32, _vp, _vp, _vp]),
    "ef21_get_state": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "ef21_get_state_host": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "ef21_set_state": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "ef21_eval": (ctypes.c_int, [_vp, _dp, _dp, _dp]),
    "ef21_poll": (ctypes.c_int, [_vp]),
    "ef21_set_objective": (ctypes.c_int, [_vp, _i32]),
    "ef21_set_variant": (ctypes.c_int, [_vp, _i32]),
    "ef21_get_plus_choice": (ctypes.c_int, [_vp, _vp]),
    "ef21_set_topk_algorithm": (ctypes.c_int, [_vp, _i32]),
    "ef21_fallback_count": (ctypes.c_int, [_vp, ctypes.POINTER(_i64)]),
    "ef21_clear_status": (ctypes.c_int, [_vp]),
    "ef21_selftest_bounded_wait": (ctypes.c_int, [_vp, ctypes.c_uint32]),
    "ef21_selftest_exchange_floor": (ctypes.c_int, [_vp, ctypes.c_int32]),
    "ef21_set_persistent_body": (ctypes.c_int, [_vp, ctypes.c_int32]),
    "ef21_get_persistent_body": (ctypes.c_int32, [_vp]),
    "ef21_set_persistent_shape": (ctypes.c_int, [_vp, _i32, _i32, _i32]),
    "ef21_get_persistent_shape": (ctypes.c_int, [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "ef21_set_persistent_threads": (ctypes.c_int, [_vp, _i32]),
    "ef21_get_persistent_threads": (_i32, [_vp]),
    "ef21_set_path": (ctypes.c_int, [_vp, _i32]),
    "ef21_last_path": (_i32, [_vp]),
    "ef21_launch_count": (_i64, [_vp]),
}


class Ef21Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2106_05203_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)          # AttributeError if the symbol is not exported
        fn.restype = res
        fn.argtypes = args
    return lib


_lib = load_library()


def _check(status: int, where: str) -> None:
    if status != EF21_OK:
        raise Ef21Error(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _stream_handle(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dev_f32(t: torch.Tensor, shape=None) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError("expected a contiguous float32 CUDA tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return t


def workspace_bytes(n: int, d: int, k: int, total_rows: int) -> int:
    return int(_lib.ef21_workspace_bytes(n, d, k, total_rows))


def status_string(status: int) -> str:
    return _lib.ef21_status_string(status).decode()


class EF21:
    """One EF21 problem resident on one GPU (names follow include/ef21.h)."""

    def __init__(self, n: int, d: int, k: int, gamma: float, lam: float = 0.0, total_rows: int = 0,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("libef21 needs a CUDA device; there is no CPU path")
        self.device = torch.device(device if device is not None else "cuda:0")
        self.n, self.d, self.k, self.total_rows = int(n), int(d), int(k), int(total_rows)
        self.stream = stream
        nbytes = workspace_bytes(n, d, k, total_rows)
        if nbytes == 0:
            raise Ef21Error(1, "ef21_workspace_bytes")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            handle = _vp()
            _check(_lib.ef21_create(ctypes.byref(handle), n, d, k, gamma, lam, total_rows,
                                    ctypes.c_void_p(self._ws_ptr), nbytes, _stream_handle(stream)), "ef21_create")
        self._h = handle
        self._keep = []          # tensors that must outlive asynchronous calls

    def close(self) -> None:
        if getattr(self, "_h", None):
            _lib.ef21_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- data ---------------------------------------------------------------
    def load_shards(self, A: torch.Tensor, y: torch.Tensor, row_offsets) -> None:
        off = np.ascontiguousarray(np.asarray(row_offsets), dtype=np.int64)
        if off.shape != (self.n + 1,):
            raise ValueError("row_offsets must have n+1 entries")
        _dev_f32(A, (self.total_rows, self.d)); _dev_f32(y, (self.total_rows,))
        _check(_lib.ef21_load_shards(self._h, _ptr(A), _ptr(y), _np_ptr(off)), "ef21_load_shards")
        self._keep = [A, y]

    def load_shards_host(self, A: np.ndarray, y: np.ndarray, row_offsets) -> None:
        off = np.ascontiguousarray(np.asarray(row_offsets), dtype=np.int64)
        if off.shape != (self.n + 1,):
            raise ValueError("row_offsets must have n+1 entries")
        A = np.ascontiguousarray(A, dtype=np.float32); y = np.ascontiguousarray(y, dtype=np.float32)
        if A.shape != (self.total_rows, self.d) or y.shape != (self.total_rows,):
            raise ValueError("A must be [total_rows, d], y [total_rows]")
        _check(_lib.ef21_load_shards_host(self._h, _np_ptr(A), _np_ptr(y), _np_ptr(off)), "ef21_load_shards_host")
        self._keep = [A, y]

    def set_x(self, x0: torch.Tensor) -> None:
        _check(_lib.ef21_set_x(self._h, _ptr(_dev_f32(x0, (self.d,)))), "ef21_set_x")

    # -- algorithm ----------------------------------------------------------
    def init(self, mode: int = INIT_COMPRESSED) -> None:
        _check(_lib.ef21_init(self._h, mode), "ef21_init")

    def init_grads(self, V: Optional[torch.Tensor], mode: int = INIT_COMPRESSED) -> None:
        if V is not None:
            _dev_f32(V, (self.n, self.d))
        _check(_lib.ef21_init_grads(self._h, _ptr(V), mode), "ef21_init_grads")

    def step(self, steps: int = 1) -> None:
        _check(_lib.ef21_step(self._h, steps), "ef21_step")

    def step_grads(self, V: torch.Tensor, steps: int = 1) -> None:
        _check(_lib.ef21_step_grads(self._h, _ptr(_dev_f32(V, (self.n, self.d))), steps), "ef21_step_grads")

    def step_minibatch(self, batch: torch.Tensor) -> None:
        """One stochastic iteration; batch[n, tau] int32 row numbers inside each worker's shard."""
        if not (batch.is_cuda and batch.dtype == torch.int32 and batch.is_contiguous() and batch.dim() == 2
                and batch.shape[0] == self.n):
            raise TypeError("batch must be a contiguous int32 CUDA tensor of shape [n, tau]")
        _check(_lib.ef21_step_minibatch(self._h, _ptr(batch), int(batch.shape[1])), "ef21_step_minibatch")
        self._keep_batch = batch

    def step_minibatches(self, batches: torch.Tensor) -> None:
        """batches[steps, n, tau] int32 row numbers inside each worker's shard: that many stochastic iterations."""
        if not (batches.is_cuda and batches.dtype == torch.int32 and batches.is_contiguous() and batches.dim() == 3
                and batches.shape[1] == self.n):
            raise TypeError("batches must be a contiguous int32 CUDA tensor of shape [steps, n, tau]")
        _check(_lib.ef21_step_minibatches(self._h, _ptr(batches), int(batches.shape[2]), int(batches.shape[0])),
               "ef21_step_minibatches")
        self._keep_batch = batches

    def step_randk(self, sets: torch.Tensor, V: Optional[torch.Tensor] = None) -> None:
        """sets[steps, n, k] int32 (ascending, distinct coordinates per worker): that many iterations with the scaled
        Rand-k compressor; V[n, d] (optional) replaces the local gradients."""
        if not (sets.is_cuda and sets.dtype == torch.int32 and sets.is_contiguous() and sets.dim() == 3
                and sets.shape[1] == self.n and sets.shape[2] == self.k):
            raise TypeError("sets must be a contiguous int32 CUDA tensor of shape [steps, n, k]")
        if V is not None:
            _dev_f32(V, (self.n, self.d))
        _check(_lib.ef21_step_randk(self._h, _ptr(V), _ptr(sets), int(sets.shape[0])), "ef21_step_randk")
        self._keep_batch = (sets, V)

    def local_grads(self) -> torch.Tensor:
        out = torch.empty((self.n, self.d), dtype=torch.float32, device=self.device)
        _check(_lib.ef21_local_grads(self._h, _ptr(out)), "ef21_local_grads")
        return out

    # -- state --------------------------------------------------------------
    def get_state(self, messages: bool = True):
        """(x, g, gi, last_idx, last_val) as new device tensors."""
        dev = self.device
        x = torch.empty(self.d, dtype=torch.float32, device=dev)
        g = torch.empty(self.d, dtype=torch.float32, device=dev)
        gi = torch.empty((self.n, self.d), dtype=torch.float32, device=dev)
        li = torch.empty((self.n, self.k), dtype=torch.int32, device=dev) if messages else None
        lv = torch.empty((self.n, self.k), dtype=torch.float32, device=dev) if messages else None
        _check(_lib.ef21_get_state(self._h, _ptr(x), _ptr(g), _ptr(gi), _ptr(li), _ptr(lv)), "ef21_get_state")
        return x, g, gi, li, lv

    def get_state_host(self, want_gi: bool = True, messages: bool = True):
        """(x, g, gi, last_idx, last_val) as numpy arrays; synchronises."""
        x = np.empty(self.d, dtype=np.float32)
        g = np.empty(self.d, dtype=np.float32)
        gi = np.empty((self.n, self.d), dtype=np.float32) if want_gi else None
        li = np.empty((self.n, self.k), dtype=np.int32) if messages else None
        lv = np.empty((self.n, self.k), dtype=np.float32) if messages else None
        _check(_lib.ef21_get_state_host(self._h, _np_ptr(x), _np_ptr(g), _np_ptr(gi), _np_ptr(li), _np_ptr(lv)),
               "ef21_get_state_host")
        return x, g, gi, li, lv

    def set_state(self, x: Optional[torch.Tensor] = None, g: Optional[torch.Tensor] = None,
                  gi: Optional[torch.Tensor] = None) -> None:
        if x is not None: _dev_f32(x, (self.d,))
        if g is not None: _dev_f32(g, (self.d,))
        if gi is not None: _dev_f32(gi, (self.n, self.d))
        _check(_lib.ef21_set_state(self._h, _ptr(x), _ptr(g), _ptr(gi)), "ef21_set_state")

    def eval(self) -> Tuple[float, float, float]:
        f, nrm, G = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
        _check(_lib.ef21_eval(self._h, ctypes.byref(f), ctypes.byref(nrm), ctypes.byref(G)), "ef21_eval")
        return f.value, nrm.value, G.value

    def poll(self) -> int:
        return int(_lib.ef21_poll(self._h))

    def set_objective(self, objective: int) -> None:
        _check(_lib.ef21_set_objective(self._h, objective), "ef21_set_objective")

    def set_variant(self, variant: int) -> None:
        _check(_lib.ef21_set_variant(self._h, variant), "ef21_set_variant")

    def get_plus_choice(self) -> np.ndarray:
        out = np.zeros(self.n, dtype=np.int32)
        _check(_lib.ef21_get_plus_choice(self._h, _np_ptr(out)), "ef21_get_plus_choice")
        return out

    def set_topk_algorithm(self, algorithm: int) -> None:
        _check(_lib.ef21_set_topk_algorithm(self._h, algorithm), "ef21_set_topk_algorithm")

    def fallback_count(self) -> int:
        v = _i64()
        _check(_lib.ef21_fallback_count(self._h, ctypes.byref(v)), "ef21_fallback_count")
        return int(v.value)

    def clear_status(self) -> None:
        _check(_lib.ef21_clear_status(self._h), "ef21_clear_status")

    def selftest_bounded_wait(self, spin_limit: int) -> None:
        _check(_lib.ef21_selftest_bounded_wait(self._h, spin_limit), "ef21_selftest_bounded_wait")

    def set_persistent_body(self, body: int) -> None:
        _check(_lib.ef21_set_persistent_body(self._h, body), "ef21_set_persistent_body")

    def get_persistent_body(self) -> int:
        return int(_lib.ef21_get_persistent_body(self._h))

    def selftest_exchange_floor(self, steps: int) -> None:
        _check(_lib.ef21_selftest_exchange_floor(self._h, steps), "ef21_selftest_exchange_floor")

    def set_persistent_shape(self, cluster_blocks: int = 0, rows_per_batch: int = 0, row_source: int = -1) -> None:
        _check(_lib.ef21_set_persistent_shape(self._h, cluster_blocks, rows_per_batch, row_source),
               "ef21_set_persistent_shape")

    def get_persistent_shape(self):
        c, r, s = _i32(), _i32(), _i32()
        _check(_lib.ef21_get_persistent_shape(self._h, ctypes.byref(c), ctypes.byref(r), ctypes.byref(s)),
               "ef21_get_persistent_shape")
        return c.value, r.value, s.value

    def set_persistent_threads(self, threads_per_block: int) -> None:
        _check(_lib.ef21_set_persistent_threads(self._h, threads_per_block), "ef21_set_persistent_threads")

    def get_persistent_threads(self) -> int:
        return int(_lib.ef21_get_persistent_threads(self._h))

    def set_path(self, path: int) -> None:
        _check(_lib.ef21_set_path(self._h, path), "ef21_set_path")

    @property
    def last_path(self) -> int:
        return int(_lib.ef21_last_path(self._h))

    @property
    def launch_count(self) -> int:
        return int(_lib.ef21_launch_count(self._h))


def topk(v: torch.Tensor, k: int, stream: Optional[torch.cuda.Stream] = None):
    """Top-k compressor on a batch of vectors v[batch, d] -> (idx[batch, k] int32, val[batch, k])."""
    if v.dim() == 1:
        v = v.unsqueeze(0)
    _dev_f32(v)
    batch, d = v.shape
    nbytes = int(_lib.ef21_topk_workspace_bytes(batch, d, k))
    if nbytes == 0:
        raise Ef21Error(1, "ef21_topk_workspace_bytes")
    with torch.cuda.device(v.device):
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=v.device)
        ws_ptr = (ws.data_ptr() + 255) // 256 * 256
        idx = torch.empty((batch, k), dtype=torch.int32, device=v.device)
        val = torch.empty((batch, k), dtype=torch.float32, device=v.device)
        _check(_lib.ef21_topk(_ptr(v), batch, d, k, _ptr(idx), _ptr(val), ctypes.c_void_p(ws_ptr), nbytes,
                              _stream_handle(stream)), "ef21_topk")
        ws.record_stream(stream if stream is not None else torch.cuda.current_stream())
    return idx, val


def topk_static(v: torch.Tensor, k: int, idx: torch.Tensor, val: torch.Tensor,
                stream: Optional[torch.cuda.Stream] = None) -> None:
    """ef21_topk_static: Top-k into caller-provided outputs idx[batch, k] (int32) and val[batch, k]
    (float32) with no device scratch handed over and none allocated; for callers that must not
    touch the CUDA allocator.  Raises Ef21Error(EF21_ERR_UNSUPPORTED) beyond the built-in scratch
    (batch <= 64, batch * ceil(d / 4096) <= 16384)."""
    if v.dim() == 1:
        v = v.unsqueeze(0)
    _dev_f32(v)
    batch, d = v.shape
    if not (idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous() and idx.numel() == batch * k):
        raise TypeError("idx must be a contiguous int32 CUDA tensor with batch*k entries")
    if not (val.is_cuda and val.dtype == torch.float32 and val.is_contiguous() and val.numel() == batch * k):
        raise TypeError("val must be a contiguous float32 CUDA tensor with batch*k entries")
    with torch.cuda.device(v.device):
        _check(_lib.ef21_topk_static(_ptr(v), batch, d, k, _ptr(idx), _ptr(val), _stream_handle(stream)),
               "ef21_topk_static")
