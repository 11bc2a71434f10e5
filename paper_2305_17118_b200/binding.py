"""ctypes binding of libscissorhands.so: argument marshalling only.

Every function mirrors one entry point of ``include/scissorhands.h``.  Device
buffers are torch CUDA tensors (PyTorch is used for device memory and streams
only); the kernels do all of the method's work.  There is no CPU fallback: if
the library cannot be loaded this module raises at import.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np
import torch

from . import build as _build

SH_OK, SH_EINVAL, SH_EFULL, SH_ESTATE, SH_ECUDA, SH_ENOMEM, SH_ETOOBIG, SH_EDEVICE = 0, -1, -2, -3, -4, -5, -6, -7
SH_STATIC_SCRATCH_MAX_ENTRIES = 1 << 20
SH_F32, SH_F16, SH_BF16, SH_INT4_G64_F16 = 0, 1, 2, 3
SH_OPT_SOFTMAX_SCALE, SH_OPT_SPLIT, SH_OPT_AUTO_COMPRESS, SH_OPT_DECODE_KERNEL, SH_OPT_PREFILL_CHUNK, SH_OPT_RECORD_MODE = 0, 1, 2, 3, 4, 5
SH_OPT_COMPACTION = 6
SH_OPT_SELFTEST_SKIP_TILE = 7
SH_SELECT_MAX_N = 40000

DTYPE_CODE = {"f32": SH_F32, "f16": SH_F16, "bf16": SH_BF16, "int4": SH_INT4_G64_F16}
INPUT_TORCH_DTYPE = {SH_F32: torch.float32, SH_F16: torch.float16, SH_BF16: torch.bfloat16,
                     SH_INT4_G64_F16: torch.float16}

EXPORTS = ["sh_create", "sh_destroy", "sh_workspace_bytes", "sh_bind", "sh_set_option", "sh_decode_step",
           "sh_decode_step_host", "sh_prefill", "sh_prefill_chunk", "sh_prefill_chunk_max", "sh_export_record", "sh_recompute_record", "sh_prefill_ragged",
           "sh_sequence_state",
           "sh_compress", "sh_compress_static", "sh_scores", "sh_select", "sh_state", "sh_export_unit",
           "sh_restore", "sh_launch_count", "sh_decode_kernel_choice", "sh_import_compressed", "sh_prefill_bulk",
           "sh_prefill_bulk_scratch_bytes", "sh_strerror", "sh_last_cuda_error"]


def _load() -> C.CDLL:
    path = _build.LIB
    if _build.stale():
        try:
            path = _build.build()
        except Exception as e:  # no nvcc here: use what was shipped, if anything
            if not os.path.exists(_build.LIB):
                raise ImportError(f"libscissorhands.so is not built and cannot be built: {e}") from e
    return declare(C.CDLL(path))


def declare(lib: C.CDLL) -> C.CDLL:
    """Argument and result types of every entry point, on a loaded build of the library."""
    vp, ip, llp = C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_longlong)
    lib.sh_create.argtypes = [C.c_int] * 7 + [C.POINTER(vp)]
    lib.sh_destroy.argtypes = [vp]
    lib.sh_destroy.restype = None
    lib.sh_workspace_bytes.argtypes = [vp]
    lib.sh_workspace_bytes.restype = C.c_size_t
    lib.sh_bind.argtypes = [vp, vp, C.c_size_t, vp]
    lib.sh_set_option.argtypes = [vp, C.c_int, C.c_double]
    lib.sh_scores.argtypes = [vp, vp, vp, vp]
    lib.sh_decode_step.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.sh_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.sh_prefill.argtypes = [vp, vp, vp, vp, C.c_int, vp, vp]
    lib.sh_prefill_chunk.argtypes = [vp, vp, vp, vp, C.c_int, vp, vp]
    lib.sh_prefill_chunk_max.argtypes = [vp]
    lib.sh_export_record.argtypes = [vp, C.c_int, vp, vp]
    lib.sh_recompute_record.argtypes = [vp, vp]
    lib.sh_prefill_ragged.argtypes = [vp, vp, vp, vp, C.c_int, ip, C.c_int, vp, vp]
    lib.sh_sequence_state.argtypes = [vp, ip, llp, C.c_int]
    lib.sh_compress.argtypes = [vp, vp, ip]
    lib.sh_compress_static.argtypes = [vp, vp, ip]
    lib.sh_select.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    lib.sh_state.argtypes = [vp, vp, ip, llp, vp, vp, vp]
    lib.sh_export_unit.argtypes = [vp, C.c_int, vp, vp, vp]
    lib.sh_restore.argtypes = [vp, C.c_int, C.c_longlong]
    lib.sh_launch_count.argtypes = [vp]
    lib.sh_launch_count.restype = C.c_longlong
    lib.sh_decode_kernel_choice.argtypes = [vp]
    lib.sh_import_compressed.argtypes = [vp, vp, vp]
    lib.sh_prefill_bulk.argtypes = [vp, vp, vp, vp, C.c_int, vp, vp, C.c_size_t, vp]
    lib.sh_prefill_bulk_scratch_bytes.argtypes = [vp, C.c_int]
    lib.sh_prefill_bulk_scratch_bytes.restype = C.c_size_t
    lib.sh_strerror.argtypes = [C.c_int]
    lib.sh_strerror.restype = C.c_char_p
    lib.sh_last_cuda_error.argtypes = [vp]
    lib.sh_last_cuda_error.restype = C.c_char_p
    return lib


lib = _load()


class ShError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        msg = lib.sh_strerror(status).decode()
        super().__init__(f"libscissorhands: {msg} ({status})" + (f": {detail}" if detail else ""))


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _dev(t: torch.Tensor, dtype: torch.dtype, numel: int, what: str) -> int:
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype and t.numel() == numel):
        raise ValueError(f"{what}: need a contiguous CUDA tensor of {numel} x {dtype}, got "
                         f"{tuple(t.shape)} {t.dtype} on {t.device}")
    return t.data_ptr()


class Handle:
    """One budgeted KV cache: ``heads`` independent units of one layer.

    Mirrors ``sh_create`` + ``sh_bind``; the workspace is a torch uint8 tensor
    owned by this object.
    """

    def __init__(self, B: int, r: int, w: int, m: int, heads: int, head_dim: int, dtype, device="cuda:0",
                 split: Optional[int] = None, scale: Optional[float] = None, auto_compress: bool = True,
                 kernel: Optional[int] = None, prefill_chunk: Optional[bool] = None, recompute_record: bool = False,
                 unordered: Optional[bool] = None):
        self.dtype = DTYPE_CODE[dtype] if isinstance(dtype, str) else int(dtype)
        self.B, self.r, self.w, self.m, self.U, self.D = B, r, w, m, heads, head_dim
        self.Bw = (B + 31) // 32
        self.device = torch.device(device)
        self.in_dtype = INPUT_TORCH_DTYPE.get(self.dtype, torch.float16)
        h = C.c_void_p()
        rc = lib.sh_create(B, r, w, m, heads, head_dim, self.dtype, C.byref(h))
        if rc:
            raise ShError(rc)
        self._h = h
        if scale is not None:
            self.set_option(SH_OPT_SOFTMAX_SCALE, scale)
        if split is not None:
            self.set_option(SH_OPT_SPLIT, split)
        if kernel is not None:
            self.set_option(SH_OPT_DECODE_KERNEL, kernel)
        if recompute_record:
            self.set_option(SH_OPT_RECORD_MODE, 1.0)
        if unordered is not None:
            self.set_option(SH_OPT_COMPACTION, 1.0 if unordered else 0.0)
        if prefill_chunk is not None:
            self.set_option(SH_OPT_PREFILL_CHUNK, float(int(prefill_chunk)))
        self.set_option(SH_OPT_AUTO_COMPRESS, 1.0 if auto_compress else 0.0)
        self.workspace_bytes = int(lib.sh_workspace_bytes(h))
        with torch.cuda.device(self.device):
            self.slab = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
            off = (-self.slab.data_ptr()) % 256
            self._slab_ptr = self.slab.data_ptr() + off
            self._slab_off = off
            self._check(lib.sh_bind(h, self._slab_ptr, self.workspace_bytes, _stream_ptr(None)))

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and lib is not None:      # at interpreter shutdown the module globals may already be gone
            lib.sh_destroy(h)

    def _check(self, rc: int):
        if rc:
            raise ShError(rc, lib.sh_last_cuda_error(self._h).decode() if rc == SH_ECUDA else "")

    # -- sh_set_option -------------------------------------------------------
    def set_option(self, key: int, value: float):
        self._check(lib.sh_set_option(self._h, key, float(value)))

    # -- sh_decode_step ------------------------------------------------------
    def decode_step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                    out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        n = self.U * self.D
        if out is None:
            out = torch.empty(self.U, self.D, dtype=torch.float32, device=self.device)
        self._check(lib.sh_decode_step(self._h, _dev(q, self.in_dtype, n, "q"), _dev(k_new, self.in_dtype, n, "k_new"),
                                       _dev(v_new, self.in_dtype, n, "v_new"), _dev(out, torch.float32, n, "out"),
                                       _stream_ptr(stream)))
        return out

    # -- sh_decode_step_host ---------------------------------------------------
    def decode_step_host(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, out: torch.Tensor,
                         stream=None) -> torch.Tensor:
        n = self.U * self.D
        for t, dt, what in ((q, self.in_dtype, "q"), (k_new, self.in_dtype, "k_new"), (v_new, self.in_dtype, "v_new"),
                            (out, torch.float32, "out")):
            if t.is_cuda or not t.is_contiguous() or t.dtype != dt or t.numel() != n:
                raise ValueError(f"{what}: need a contiguous host tensor of {n} x {dt}")
        self._check(lib.sh_decode_step_host(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
                                            _stream_ptr(stream)))
        return out

    def decode_step_host_raw(self, q_ptr: int, k_ptr: int, v_ptr: int, out_ptr: int, stream_ptr: int = 0):
        """sh_decode_step_host on raw host addresses the caller has validated once (contiguous rows of
        the handle's dtype, [heads, head_dim]; out fp32): no per-call tensor checks."""
        rc = lib.sh_decode_step_host(self._h, q_ptr, k_ptr, v_ptr, out_ptr, stream_ptr)
        if rc:
            self._check(rc)

    # -- sh_prefill ------------------------------------------------------------
    def prefill(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: Optional[torch.Tensor] = None,
                stream=None):
        p = q.shape[0]
        n = p * self.U * self.D
        optr = _dev(out, torch.float32, n, "out") if out is not None else None
        self._check(lib.sh_prefill(self._h, _dev(q, self.in_dtype, n, "q"), _dev(k, self.in_dtype, n, "k"),
                                   _dev(v, self.in_dtype, n, "v"), p, optr, _stream_ptr(stream)))
        return out

    # -- sh_import_compressed / sh_prefill_bulk -------------------------------------
    def import_compressed(self, src: "Handle", stream=None):
        self._check(lib.sh_import_compressed(self._h, src._h, _stream_ptr(stream)))

    def prefill_bulk(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: Optional[torch.Tensor] = None,
                     stream=None):
        p = q.shape[0]
        n = p * self.U * self.D
        need = int(lib.sh_prefill_bulk_scratch_bytes(self._h, p))
        if not need:
            raise ShError(SH_EINVAL, "prompt length outside 1..32767")
        with torch.cuda.device(self.device):
            scratch = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        sptr = scratch.data_ptr() + (-scratch.data_ptr()) % 256
        optr = _dev(out, torch.float32, n, "out") if out is not None else None
        self._check(lib.sh_prefill_bulk(self._h, _dev(q, self.in_dtype, n, "q"), _dev(k, self.in_dtype, n, "k"),
                                        _dev(v, self.in_dtype, n, "v"), p, optr, sptr, need, _stream_ptr(stream)))
        scratch.record_stream(stream or torch.cuda.current_stream())
        return out

    # -- sh_prefill_ragged / sh_sequence_state -----------------------------------
    def prefill_ragged(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, lengths, out: Optional[torch.Tensor] = None,
                       stream=None):
        p = q.shape[0]
        n = p * self.U * self.D
        lens = (C.c_int * len(lengths))(*[int(x) for x in lengths])
        optr = _dev(out, torch.float32, n, "out") if out is not None else None
        self._check(lib.sh_prefill_ragged(self._h, _dev(q, self.in_dtype, n, "q"), _dev(k, self.in_dtype, n, "k"),
                                          _dev(v, self.in_dtype, n, "v"), p, lens, len(lengths), optr,
                                          _stream_ptr(stream)))
        return out

    def sequence_state(self):
        """(n [sequences], t [sequences]) host counters."""
        ns = lib.sh_sequence_state(self._h, None, None, 0)
        n_a, t_a = (C.c_int * ns)(), (C.c_longlong * ns)()
        lib.sh_sequence_state(self._h, n_a, t_a, ns)
        return np.array(n_a[:], dtype=np.int64), np.array(t_a[:], dtype=np.int64)

    def state_full(self, stream=None):
        """sh_state without trimming to a common n: (pos [U,B], counters [U,B], low [U,B] bool)."""
        pos_a = np.zeros((self.U, self.B), dtype=np.int32)
        cnt_a = np.zeros((self.U, self.B), dtype=np.uint16)
        low_a = np.zeros((self.U, self.Bw), dtype=np.uint32)
        self._check(lib.sh_state(self._h, _stream_ptr(stream), None, None, pos_a.ctypes.data, cnt_a.ctypes.data,
                                 low_a.ctypes.data))
        bits = np.unpackbits(low_a.view(np.uint8), axis=1, bitorder="little")[:, : self.B].astype(bool)
        return pos_a, cnt_a, bits

    # -- sh_prefill_chunk --------------------------------------------------------
    @property
    def prefill_chunk_max(self) -> int:
        return int(lib.sh_prefill_chunk_max(self._h))

    def prefill_chunk(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: Optional[torch.Tensor] = None,
                      stream=None):
        c = q.shape[0]
        n = c * self.U * self.D
        optr = _dev(out, torch.float32, n, "out") if out is not None else None
        self._check(lib.sh_prefill_chunk(self._h, _dev(q, self.in_dtype, n, "q"), _dev(k, self.in_dtype, n, "k"),
                                         _dev(v, self.in_dtype, n, "v"), c, optr, _stream_ptr(stream)))
        return out

    # -- sh_recompute_record --------------------------------------------------------
    def recompute_record(self, stream=None):
        self._check(lib.sh_recompute_record(self._h, _stream_ptr(stream)))

    # -- sh_export_record -----------------------------------------------------------
    def export_record(self, unit: int, stream=None) -> np.ndarray:
        """Bit-planes of one unit as a bool array [w, B]: entry (s mod w, j) is step s's comparison for slot j."""
        planes = np.zeros((self.w, self.Bw), dtype=np.uint32)
        self._check(lib.sh_export_record(self._h, unit, planes.ctypes.data, _stream_ptr(stream)))
        return np.unpackbits(planes.view(np.uint8), axis=1, bitorder="little")[:, : self.B].astype(bool)

    # -- sh_scores ---------------------------------------------------------------
    def scores(self, q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """Attention scores of ``q`` [U, d] over each unit's present cache: fp32 [U, B], 0 beyond the live slots."""
        if out is None:
            out = torch.empty(self.U, self.B, dtype=torch.float32, device=self.device)
        self._check(lib.sh_scores(self._h, _dev(q, self.in_dtype, self.U * self.D, "q"),
                                  _dev(out, torch.float32, self.U * self.B, "out"), _stream_ptr(stream)))
        return out

    # -- sh_compress -------------------------------------------------------------
    def compress(self, stream=None) -> int:
        ev = C.c_int(0)
        self._check(lib.sh_compress(self._h, _stream_ptr(stream), C.byref(ev)))
        return ev.value

    # -- sh_compress_static ----------------------------------------------------------
    def compress_static(self, stream=None) -> int:
        """sh_compress without any device allocation or workspace scratch: for
        callers that cannot cudaMalloc (all HBM already pooled, or inside a
        latency-critical loop).  Needs heads * B <= SH_STATIC_SCRATCH_MAX_ENTRIES;
        calls on one device must not overlap."""
        ev = C.c_int(0)
        self._check(lib.sh_compress_static(self._h, _stream_ptr(stream), C.byref(ev)))
        return ev.value

    # -- sh_state ------------------------------------------------------------------
    def state(self, pos: bool = True, counters: bool = True, low: bool = True, stream=None):
        """Returns ``(n, t, pos [U,n] int32 | None, counters [U,n] uint16 | None,
        low [U,n] bool | None)`` on the host."""
        n, t = C.c_int(0), C.c_longlong(0)
        pos_a = np.zeros((self.U, self.B), dtype=np.int32) if pos else None
        cnt_a = np.zeros((self.U, self.B), dtype=np.uint16) if counters else None
        low_a = np.zeros((self.U, self.Bw), dtype=np.uint32) if low else None
        ptr = lambda a: a.ctypes.data if a is not None else None
        self._check(lib.sh_state(self._h, _stream_ptr(stream), C.byref(n), C.byref(t), ptr(pos_a), ptr(cnt_a),
                                 ptr(low_a)))
        nn = n.value
        low_b = None
        if low:
            bits = np.unpackbits(low_a.view(np.uint8), axis=1, bitorder="little")
            low_b = bits[:, :nn].astype(bool)
            assert not bits[:, nn:].any(), "record bits set beyond the live slots"
        return (nn, t.value, pos_a[:, :nn] if pos else None, cnt_a[:, :nn] if counters else None, low_b)

    @property
    def n(self) -> int:
        n = C.c_int(0)
        self._check(lib.sh_state(self._h, _stream_ptr(None), C.byref(n), None, None, None, None))
        return n.value

    # -- sh_export_unit ---------------------------------------------------------------
    def export_unit(self, unit: int, stream=None) -> Tuple[np.ndarray, np.ndarray]:
        K = np.zeros((self.B, self.D), dtype=np.float32)
        V = np.zeros((self.B, self.D), dtype=np.float32)
        self._check(lib.sh_export_unit(self._h, unit, K.ctypes.data, V.ctypes.data, _stream_ptr(stream)))
        return K, V

    # -- checkpoint / sh_restore -------------------------------------------------------
    def snapshot(self):
        """Copy of the whole workspace plus the host counters that go with it."""
        n, t, *_ = self.state(pos=False, counters=False, low=False)
        return self.slab.clone(), n, t

    def restore(self, snap):
        slab, n, t = snap
        self.slab.copy_(slab)
        self._check(lib.sh_restore(self._h, n, t))

    @property
    def launch_count(self) -> int:
        return int(lib.sh_launch_count(self._h))

    @property
    def decode_kernel(self) -> str:
        """Name of the fused decode kernel sh_decode_step launches for this handle."""
        return {1: "sh_decode_kernel", 2: "sh_decode_tma_kernel", 3: "sh_decode_int4_mma_kernel"}[int(lib.sh_decode_kernel_choice(self._h))]


def select(counters: torch.Tensor, r: int, m: int, stream=None) -> torch.Tensor:
    """``sh_select``: counters ``[units, n]`` (CUDA, any integer dtype, values
    <= 16384) -> dropped indices ``[units, m]`` int32, ascending."""
    units, n = counters.shape
    c16 = counters.to(torch.int16).contiguous()   # values <= 16384: same bits as uint16
    out = torch.empty(units, m, dtype=torch.int32, device=counters.device)
    rc = lib.sh_select(c16.data_ptr(), units, n, r, m, out.data_ptr(), _stream_ptr(stream))
    if rc:
        raise ShError(rc)
    return out
