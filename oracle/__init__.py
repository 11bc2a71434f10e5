"""CPU oracle for budgeted KV-cache decode attention — TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper over ``scissorhands_oracle.c`` (plain C, fp64, one unit
at a time; see that file's header for the steps, the readings of the paper it
takes and what pins it).  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library and its Python
binding never do, and this package imports neither of them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "scissorhands_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libscissorhands_oracle.so")
_lib = None

AMB_WINDOW = 1e-6


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (strict IEEE arithmetic: no fast-math, no
    contraction).  Returns the path of the shared library."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    tmp = _LIB + f".{os.getpid()}.tmp"
    cmd = ["gcc", "-O2", "-std=gnu11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    dp = c.POINTER(c.c_double)
    bp = c.POINTER(c.c_uint8)
    ip = c.POINTER(c.c_int)
    lib.sho_create.restype = c.c_void_p
    lib.sho_create.argtypes = [c.c_int] * 6 + [c.c_double, c.c_int]
    lib.sho_create_reading.restype = c.c_void_p
    lib.sho_create_reading.argtypes = [c.c_int] * 6 + [c.c_double] + [c.c_int] * 5
    lib.sho_cap.argtypes = [c.c_void_p]
    lib.sho_import_compressed.argtypes = [c.c_void_p, c.c_void_p]
    lib.sho_select_newest_first.argtypes = [ip, c.c_int, c.c_int, c.c_int, ip]
    lib.sho_select_newest_first.restype = None
    lib.sho_destroy.argtypes = [c.c_void_p]
    lib.sho_destroy.restype = None
    lib.sho_threads.restype = c.c_int
    lib.sho_amb_window.restype = c.c_double
    lib.sho_n.argtypes = [c.c_void_p]
    lib.sho_t_now.argtypes = [c.c_void_p]
    lib.sho_t_now.restype = c.c_long
    lib.sho_full.argtypes = [c.c_void_p]
    lib.sho_attend.argtypes = [c.c_void_p, dp, dp, dp, dp, dp, bp, bp]
    lib.sho_record.argtypes = [c.c_void_p, bp]
    lib.sho_record.restype = None
    lib.sho_counters.argtypes = [c.c_void_p, ip]
    lib.sho_counters.restype = None
    lib.sho_positions.argtypes = [c.c_void_p, ip]
    lib.sho_positions.restype = None
    lib.sho_cache.argtypes = [c.c_void_p, c.c_int, dp, dp]
    lib.sho_cache.restype = None
    lib.sho_select.argtypes = [ip, c.c_int, c.c_int, c.c_int, ip]
    lib.sho_select.restype = None
    lib.sho_compress.argtypes = [c.c_void_p, ip]
    lib.sho_recount.argtypes = [c.c_void_p, dp, bp, bp, ip]
    lib.sho_recount.restype = None
    lib.sho_set_record.argtypes = [c.c_void_p, bp, ip]
    lib.sho_set_record.restype = None
    lib.sho_quantize.argtypes = [dp, c.c_int, c.c_int, dp, c.POINTER(c.c_int8), c.POINTER(c.c_float)]
    lib.sho_quantize.restype = None
    _lib = lib
    return lib


def threads() -> int:
    """Number of host threads the oracle's loop over units uses."""
    return int(_load().sho_threads())


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _bp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8))


def _ip(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int))


def _f64(a, shape) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if a.shape != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {a.shape}")
    return a


class Oracle:
    """Budgeted KV cache of ``units`` independent (sequence, head) pairs.

    ``B, r, w, m`` are the budget, recent window, history window and drop
    amount of Algorithms 1 and 2.  ``scale`` multiplies the logits (default
    1/sqrt(head_dim)).  ``quant`` selects the int4 group-64 store.  Inputs must
    already be rounded to the storage dtype of the implementation under test.

    Alternative readings of the paper (all off by default; the CUDA library
    implements the defaults only): ``threshold`` 0 = 1/t of each step, 1 = 1/t of
    the compression step for the whole window (Algorithm 2 literally), 2 = 1/n;
    ``window_plus1`` = the w+1 steps of Algorithm 2's range [t-w, t];
    ``tie_newest`` = among equal counters drop the newest first (a stable
    ascending argsort cut at [:-m]); ``trigger_literal`` = Algorithm 1's
    "if n > B": the cache holds up to B+1 tokens for one step.
    """

    def __init__(self, units: int, B: int, r: int, w: int, m: int, head_dim: int,
                 scale: Optional[float] = None, quant: bool = False, threshold: int = 0,
                 window_plus1: bool = False, tie_newest: bool = False, trigger_literal: bool = False):
        self._lib = _load()
        if scale is None:
            scale = 1.0 / np.sqrt(head_dim)
        self.U, self.r, self.w, self.m, self.d = units, r, w, m, head_dim
        self.budget = B
        self.scale, self.quant = float(scale), bool(quant)
        self._h = self._lib.sho_create_reading(units, B, r, w, m, head_dim, float(scale), int(quant), int(threshold),
                                               int(window_plus1), int(tie_newest), int(trigger_literal))
        # rows of storage per unit (the stride of every [U, .] array below): the budget, or one more
        # under the literal trigger reading
        self.B = int(self._lib.sho_cap(self._h)) if self._h else B
        if not self._h:
            raise ValueError("invalid oracle parameters (need 1 <= m <= B - r, w >= 1, "
                             "head_dim % 64 == 0 for the int4 store)")

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._lib.sho_destroy(h)

    # -- state -------------------------------------------------------------
    @property
    def n(self) -> int:
        return int(self._lib.sho_n(self._h))

    @property
    def t(self) -> int:
        return int(self._lib.sho_t_now(self._h))

    @property
    def full(self) -> bool:
        return bool(self._lib.sho_full(self._h))

    def positions(self) -> np.ndarray:
        """[units, n] 1-based stream positions of the live tokens, ascending."""
        a = np.zeros((self.U, self.B), dtype=np.int32)
        self._lib.sho_positions(self._h, _ip(a))
        return a[:, : self.n].copy()

    def counters(self) -> np.ndarray:
        """[units, n] importance record I of Algorithm 2 at the current step."""
        a = np.zeros((self.U, self.B), dtype=np.int32)
        self._lib.sho_counters(self._h, _ip(a))
        return a[:, : self.n].copy()

    def cache(self, unit: int) -> Tuple[np.ndarray, np.ndarray]:
        """Stored (K, V) rows of one unit, each [n, head_dim]."""
        K = np.zeros((self.B, self.d))
        V = np.zeros((self.B, self.d))
        self._lib.sho_cache(self._h, unit, _dp(K), _dp(V))
        return K[: self.n].copy(), V[: self.n].copy()

    # -- the step, in three phases so a lockstep harness can intervene ------
    def attend(self, q, k, v):
        """Append the token and attend.  Returns ``(out [U,d], alpha [U,n],
        low [U,n] bool, amb [U,n] bool)``; nothing is recorded yet."""
        U, B, d = self.U, self.B, self.d
        q, k, v = _f64(q, (U, d)), _f64(k, (U, d)), _f64(v, (U, d))
        out = np.zeros((U, d))
        alpha = np.zeros((U, B))
        low = np.zeros((U, B), dtype=np.uint8)
        amb = np.zeros((U, B), dtype=np.uint8)
        rc = self._lib.sho_attend(self._h, _dp(q), _dp(k), _dp(v), _dp(out), _dp(alpha), _bp(low), _bp(amb))
        if rc:
            raise RuntimeError("cache is full: compress() before the next step")
        n = self.n
        return out, alpha[:, :n].copy(), low[:, :n].astype(bool), amb[:, :n].astype(bool)

    def record(self, low) -> None:
        """Remember this step's low flags ([U, n] bool) for every live token."""
        low = np.asarray(low)
        if low.shape != (self.U, self.n):
            raise ValueError(f"low must be [{self.U}, {self.n}]")
        buf = np.zeros((self.U, self.B), dtype=np.uint8)
        buf[:, : self.n] = low
        self._lib.sho_record(self._h, _bp(buf))

    def compress(self) -> Optional[np.ndarray]:
        """Algorithm 2 if the cache is full: returns the dropped stream
        positions [U, m] (ascending), else ``None``."""
        ev = np.zeros((self.U, self.m), dtype=np.int32)
        got = self._lib.sho_compress(self._h, _ip(ev))
        return ev if got else None

    def import_compressed(self, src: "Oracle") -> int:
        """The prompting stage read as a bulk operation: ``src`` streamed the whole prompt under a
        budget that never made it compress; its cache is brought under this oracle's budget by
        rounds of Algorithm 2 on the record as it stands, and the survivors become this (fresh)
        oracle's cache.  Returns the number of rounds."""
        rounds = int(self._lib.sho_import_compressed(self._h, src._h))
        if rounds < 0:
            raise ValueError("oracles do not match, the target is not fresh, or too few candidates")
        return rounds

    # -- the record recomputed at compression time (Algorithm 2 as stated) ----
    def recount(self):
        """Scores of the last w queries against the present cache (causal by
        position), as ``(alpha, low, amb)`` each [U, w, n] with row = step mod w,
        and ``steps`` [w] (0 where the window holds no query)."""
        U, w, B = self.U, self.w, self.B
        alpha = np.zeros((U, w, B))
        low = np.zeros((U, w, B), dtype=np.uint8)
        amb = np.zeros((U, w, B), dtype=np.uint8)
        steps = np.zeros(w, dtype=np.int32)
        self._lib.sho_recount(self._h, _dp(alpha), _bp(low), _bp(amb), _ip(steps))
        n = self.n
        return alpha[:, :, :n].copy(), low[:, :, :n].astype(bool), amb[:, :, :n].astype(bool), steps

    def set_record(self, low, steps) -> None:
        """Make ``low`` ([U, w, n] bool, rows as in ``recount``) the importance
        record of the live tokens."""
        low = np.asarray(low)
        if low.shape != (self.U, self.w, self.n):
            raise ValueError(f"low must be [{self.U}, {self.w}, {self.n}]")
        buf = np.zeros((self.U, self.w, self.B), dtype=np.uint8)
        buf[:, :, : self.n] = low
        steps = np.ascontiguousarray(np.asarray(steps, dtype=np.int32))
        self._lib.sho_set_record(self._h, _bp(buf), _ip(steps))

    def step_recompute(self, q, k, v):
        """One step of the recompute-at-compression variant: attend; when the
        cache is full, recount, adopt the recount as the record, compress."""
        out, _alpha, _low, _amb = self.attend(q, k, v)
        dropped = None
        if self.full:
            _a, low, _amb2, steps = self.recount()
            self.set_record(low, steps)
            dropped = self.compress()
        return out, dropped

    def step(self, q, k, v):
        """attend + record + compress.  Returns ``(out, dropped or None)``."""
        out, _alpha, low, _amb = self.attend(q, k, v)
        self.record(low)
        return out, self.compress()


def select(I, r: int, m: int, newest_first: bool = False) -> np.ndarray:
    """Selection of Algorithm 2 on given counters (tokens in position order):
    indices of the ``m`` dropped tokens, ascending.  ``newest_first``: the
    alternative tie-break (among equal counters the newest go)."""
    I = np.ascontiguousarray(np.asarray(I, dtype=np.int32))
    n = I.shape[0]
    if not (0 <= r and 1 <= m <= n - r):
        raise ValueError("need 1 <= m <= n - r")
    ev = np.zeros(m, dtype=np.int32)
    lib = _load()
    (lib.sho_select_newest_first if newest_first else lib.sho_select)(_ip(I), n, r, m, _ip(ev))
    return np.sort(ev)


def quantize_int4_g64(x):
    """Round-trip ``x [rows, d]`` through the int4 group-64 store.  Returns
    ``(stored fp64 [rows,d], codes int8 [rows,d], scales fp32 [rows,d/64])``."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    rows, d = x.shape
    if d % 64:
        raise ValueError("head_dim must be a multiple of 64")
    stored = np.zeros_like(x)
    codes = np.zeros((rows, d), dtype=np.int8)
    scales = np.zeros((rows, d // 64), dtype=np.float32)
    _load().sho_quantize(_dp(x), rows, d, _dp(stored), codes.ctypes.data_as(ctypes.POINTER(ctypes.c_int8)),
                         scales.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    return stored, codes, scales
