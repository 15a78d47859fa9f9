"""ctypes front end of the CPU oracle (test infrastructure, see ef21_oracle.c).

Builds ``ef21_oracle.c`` with gcc into two shared objects next to this file,
one with fp32 state (``precision="f32"``) and one with fp64 state
(``precision="f64"``), and exposes thin numpy wrappers.  Nothing here is used
by the CUDA library or its Python binding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ef21_oracle.c")
_LIBS = {}

_c_int32 = ctypes.c_int32
_c_int64 = ctypes.c_int64
_c_double = ctypes.c_double
_ptr = ctypes.c_void_p


def lib_path(precision: str) -> str:
    return os.path.join(_HERE, f"libef21_oracle_{precision}.so")


def build(force: bool = False) -> None:
    """Compile both precisions of the oracle (gcc -O2 -ffp-contract=off)."""
    for precision, flag in (("f32", []), ("f64", ["-DEF21O_F64"])):
        out = lib_path(precision)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-std=c99", *flag,
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_ptr)


class Oracle:
    """The oracle at one state precision.  All arrays are numpy, C-contiguous."""

    def __init__(self, precision: str = "f32"):
        if precision not in ("f32", "f64"):
            raise ValueError(precision)
        build()
        if precision not in _LIBS:
            _LIBS[precision] = ctypes.CDLL(lib_path(precision))
        self.lib = _LIBS[precision]
        self.real = np.float32 if precision == "f32" else np.float64
        self._creal = ctypes.c_float if precision == "f32" else ctypes.c_double
        self.lib.ef21o_real_bytes.restype = ctypes.c_int
        assert self.lib.ef21o_real_bytes() == np.dtype(self.real).itemsize
        self.lib.ef21o_local_loss.restype = _c_double
        self.lib.ef21o_loss.restype = _c_double

    # -- helpers -----------------------------------------------------------
    def _r(self, a) -> np.ndarray:
        return np.ascontiguousarray(a, dtype=self.real)

    @staticmethod
    def _f32(a) -> np.ndarray:
        return np.ascontiguousarray(a, dtype=np.float32)

    def set_objective(self, objective: int) -> None:
        """0: logistic loss (Eq. 19); 1: least squares (Appendix A.2).  Process-wide for this precision."""
        self.lib.ef21o_set_objective(ctypes.c_int(objective))

    # -- compressor ----------------------------------------------------------
    def topk(self, v, k: int) -> Tuple[np.ndarray, np.ndarray]:
        v = self._r(v)
        d = v.shape[0]
        idx = np.empty(k, dtype=np.int32)
        val = np.empty(k, dtype=self.real)
        self.lib.ef21o_topk(_p(v), _c_int64(d), _c_int64(k), _p(idx), _p(val))
        return idx, val

    def randk(self, v, S, unbiased: bool = False) -> Tuple[np.ndarray, np.ndarray]:
        """Scaled Rand-k of Example 2 on the index set S (ascending, distinct); unbiased=True: Rand-k itself."""
        v = self._r(v)
        S = np.ascontiguousarray(S, dtype=np.int32)
        k = S.shape[0]
        idx = np.empty(k, dtype=np.int32)
        val = np.empty(k, dtype=self.real)
        fn = self.lib.ef21o_randk_unbiased if unbiased else self.lib.ef21o_randk
        fn(_p(v), _c_int64(v.shape[0]), _c_int64(k), _p(S), _p(idx), _p(val))
        return idx, val

    # -- objective -----------------------------------------------------------
    def local_loss(self, A, y, x, lam: float) -> float:
        A = self._f32(A); y = self._f32(y); x = self._r(x)
        m, d = A.shape
        return float(self.lib.ef21o_local_loss(_p(A), _p(y), _c_int64(m), _c_int64(d), _p(x),
                                               _c_double(lam)))

    def local_grad(self, A, y, x, lam: float) -> np.ndarray:
        A = self._f32(A); y = self._f32(y); x = self._r(x)
        m, d = A.shape
        grad = np.empty(d, dtype=self.real)
        self.lib.ef21o_local_grad(_p(A), _p(y), _c_int64(m), _c_int64(d), _p(x), _c_double(lam),
                                  _p(grad))
        return grad

    def all_grads(self, A, y, row_offsets, x, lam: float) -> np.ndarray:
        A = self._f32(A); y = self._f32(y); x = self._r(x)
        off = np.ascontiguousarray(row_offsets, dtype=np.int64)
        n = off.shape[0] - 1
        d = A.shape[1]
        grads = np.empty((n, d), dtype=self.real)
        self.lib.ef21o_all_grads(_c_int32(n), _c_int64(d), _p(A), _p(y), _p(off), _p(x),
                                 _c_double(lam), _p(grads))
        return grads

    def loss(self, A, y, row_offsets, x, lam: float) -> float:
        A = self._f32(A); y = self._f32(y); x = self._r(x)
        off = np.ascontiguousarray(row_offsets, dtype=np.int64)
        n = off.shape[0] - 1
        return float(self.lib.ef21o_loss(_c_int32(n), _c_int64(A.shape[1]), _p(A), _p(y), _p(off),
                                         _p(x), _c_double(lam)))

    def diagnostics(self, A, y, row_offsets, x, lam: float, gi=None) -> Tuple[float, float]:
        """(||grad f(x)||^2, G = (1/n) sum ||g_i - grad f_i(x)||^2)."""
        A = self._f32(A); y = self._f32(y); x = self._r(x)
        off = np.ascontiguousarray(row_offsets, dtype=np.int64)
        n = off.shape[0] - 1
        gi_c = None if gi is None else self._r(gi)
        nrm = _c_double(0.0); G = _c_double(0.0)
        self.lib.ef21o_diagnostics(_c_int32(n), _c_int64(A.shape[1]), _p(A), _p(y), _p(off), _p(x),
                                   _c_double(lam), _p(gi_c), ctypes.byref(nrm), ctypes.byref(G))
        return float(nrm.value), float(G.value)


class State:
    """x, g, g_i and the last round's messages of one EF21 run on the oracle."""

    def __init__(self, oracle: Oracle, n: int, d: int, k: int, gamma: float, lam: float = 0.0,
                 A=None, y=None, row_offsets=None, x0=None):
        self.o = oracle
        self.n, self.d, self.k = int(n), int(d), int(k)
        self.gamma = float(gamma)
        self.lam = float(lam)
        self.A = None if A is None else Oracle._f32(A)
        self.y = None if y is None else Oracle._f32(y)
        self.off = None if row_offsets is None else np.ascontiguousarray(row_offsets, dtype=np.int64)
        real = oracle.real
        self.x = np.zeros(d, dtype=real) if x0 is None else np.array(x0, dtype=real)
        self.g = np.zeros(d, dtype=real)
        self.gi = np.zeros((n, d), dtype=real)
        self.idx = np.zeros((n, k), dtype=np.int32)
        self.val = np.zeros((n, k), dtype=real)

    def _args_state(self):
        return (_p(self.x), _p(self.gi), _p(self.g), _p(self.idx), _p(self.val))

    def init(self, mode: int = 0) -> None:
        lib = self.o.lib
        lib.ef21o_init(_c_int32(mode), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                       _p(self.A), _p(self.y), _p(self.off), _c_double(self.lam), _p(self.x),
                       _p(self.gi), _p(self.g), _p(self.idx), _p(self.val))

    def init_from_grads(self, grads, mode: int = 0) -> None:
        grads = self.o._r(grads)
        self.o.lib.ef21o_init_from_grads(_c_int32(mode), _c_int32(self.n), _c_int64(self.d),
                                         _c_int64(self.k), _p(grads), _p(self.gi), _p(self.g),
                                         _p(self.idx), _p(self.val))

    def step(self, steps: int = 1) -> None:
        self.o.lib.ef21o_step(_c_int32(steps), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                              _p(self.A), _p(self.y), _p(self.off), _c_double(self.lam),
                              self.o._creal(self.gamma), *self._args_state())

    def step_grads(self, V, steps: int = 1) -> None:
        V = self.o._r(V)
        assert V.shape == (self.n, self.d)
        self.o.lib.ef21o_step_grads(_c_int32(steps), _c_int32(self.n), _c_int64(self.d),
                                    _c_int64(self.k), _p(V), self.o._creal(self.gamma),
                                    *self._args_state())

    # -- EF21+ (Algorithm 3) -------------------------------------------------
    def _choice(self):
        if not hasattr(self, "choice"):
            self.choice = np.zeros(self.n, dtype=np.int32)
        return self.choice

    def plus_step(self, steps: int = 1) -> None:
        ch = self._choice()
        self.o.lib.ef21o_plus_step(_c_int32(steps), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                                   _p(self.A), _p(self.y), _p(self.off), _c_double(self.lam),
                                   self.o._creal(self.gamma), *self._args_state(), _p(ch))

    def plus_step_grads(self, V, steps: int = 1) -> None:
        V = self.o._r(V)
        ch = self._choice()
        self.o.lib.ef21o_plus_step_grads(_c_int32(steps), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                                         _p(V), self.o._creal(self.gamma), *self._args_state(), _p(ch))

    def plus_round(self, grads) -> None:
        grads = self.o._r(grads)
        ch = self._choice()
        self.o.lib.ef21o_plus_round(_c_int32(self.n), _c_int64(self.d), _c_int64(self.k), _p(grads),
                                    _p(self.gi), _p(self.g), _p(self.idx), _p(self.val), _p(ch))

    def step_minibatch(self, batch) -> None:
        """One iteration of Algorithm 5 with the given rows (batch[n, tau], row numbers inside each shard)."""
        batch = np.ascontiguousarray(batch, dtype=np.int32)
        assert batch.shape[0] == self.n
        self.o.lib.ef21o_step_minibatch(_c_int32(self.n), _c_int64(self.d), _c_int64(self.k), _p(self.A), _p(self.y),
                                        _p(self.off), _c_double(self.lam), self.o._creal(self.gamma), _p(batch),
                                        _c_int32(batch.shape[1]), *self._args_state())

    def step_randk(self, sets, V=None) -> None:
        """sets[steps, n, k] (ascending, distinct indices per worker): that many iterations of Algorithm 2 with the
        scaled Rand-k; V[n, d] (optional) replaces the local gradients."""
        sets = np.ascontiguousarray(sets, dtype=np.int32)
        assert sets.ndim == 3 and sets.shape[1] == self.n and sets.shape[2] == self.k
        Vc = None if V is None else self.o._r(V)
        self.o.lib.ef21o_step_randk(_c_int32(sets.shape[0]), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                                    _p(self.A), _p(self.y), _p(self.off), _c_double(self.lam), _p(Vc),
                                    self.o._creal(self.gamma), _p(sets), *self._args_state())

    def round(self, grads) -> None:
        """One message round (no x update) given the local gradients."""
        grads = self.o._r(grads)
        self.o.lib.ef21o_round(_c_int32(self.n), _c_int64(self.d), _c_int64(self.k), _p(grads),
                               _p(self.gi), _p(self.g), _p(self.idx), _p(self.val))

    def x_update(self) -> None:
        self.o.lib.ef21o_x_update(_c_int64(self.d), self.o._creal(self.gamma), _p(self.g), _p(self.x))

    def loss(self) -> float:
        return self.o.loss(self.A, self.y, self.off, self.x, self.lam)

    def grads(self) -> np.ndarray:
        return self.o.all_grads(self.A, self.y, self.off, self.x, self.lam)


class EFState:
    """State of the original error feedback method (Algorithm 4) on the oracle: x, the errors e_i, the
    stepsize-scaled gradients a_i = gamma * grad f_i(x) at the current x and the messages w_i last sent."""

    def __init__(self, oracle: Oracle, n: int, d: int, k: int, gamma: float, lam: float = 0.0,
                 A=None, y=None, row_offsets=None, x0=None):
        self.o = oracle
        self.n, self.d, self.k = int(n), int(d), int(k)
        self.gamma = float(gamma)
        self.lam = float(lam)
        self.A = None if A is None else Oracle._f32(A)
        self.y = None if y is None else Oracle._f32(y)
        self.off = None if row_offsets is None else np.ascontiguousarray(row_offsets, dtype=np.int64)
        real = oracle.real
        self.x = np.zeros(d, dtype=real) if x0 is None else np.array(x0, dtype=real)
        self.e = np.zeros((n, d), dtype=real)
        self.a = np.zeros((n, d), dtype=real)
        self.idx = np.zeros((n, k), dtype=np.int32)
        self.val = np.zeros((n, k), dtype=real)

    def _state(self):
        return (_p(self.x), _p(self.e), _p(self.a), _p(self.idx), _p(self.val))

    def init(self) -> None:
        self.o.lib.ef21o_ef_init(_c_int32(self.n), _c_int64(self.d), _c_int64(self.k), _p(self.A), _p(self.y),
                                 _p(self.off), _c_double(self.lam), self.o._creal(self.gamma), *self._state())

    def init_from_grads(self, grads) -> None:
        grads = self.o._r(grads)
        self.o.lib.ef21o_ef_init_from_grads(_c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                                            self.o._creal(self.gamma), _p(grads), *self._state()[1:])

    def step(self, steps: int = 1) -> None:
        self.o.lib.ef21o_ef_step(_c_int32(steps), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                                 _p(self.A), _p(self.y), _p(self.off), _c_double(self.lam),
                                 self.o._creal(self.gamma), *self._state())

    def step_grads(self, V, steps: int = 1) -> None:
        V = self.o._r(V)
        assert V.shape == (self.n, self.d)
        self.o.lib.ef21o_ef_step_grads(_c_int32(steps), _c_int32(self.n), _c_int64(self.d), _c_int64(self.k),
                                       _p(V), self.o._creal(self.gamma), *self._state())

    def loss(self) -> float:
        return self.o.loss(self.A, self.y, self.off, self.x, self.lam)
