"""Thin ctypes binding of ``libgbmuf.so``: argument marshalling only, same names as the C ABI.

Every step of the synchronisation round runs in the CUDA library.  PyTorch is used here only to
hand over device pointers and the current stream.  If the library is missing this module raises;
there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

GBMUF_OK = 0
ERR_INVALID_ARG, ERR_BAD_STATE, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = 1, 2, 3, 4, 5, 6
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "BAD_STATE", 3: "ALLOC", 4: "CUDA", 5: "TIMEOUT",
                6: "UNSUPPORTED"}
F32, BF16 = 0, 1
MODE_BMUF, MODE_MA = 0, 1

EXPORTS = ["gbmuf_create", "gbmuf_set_partition", "gbmuf_init", "gbmuf_local_perturb",
           "gbmuf_sync_round", "gbmuf_get_neighbors", "gbmuf_final_average", "gbmuf_device_status",
           "gbmuf_set_tuning", "gbmuf_get_launch_info", "gbmuf_last_error", "gbmuf_destroy",
           "gbmuf_sync_round_noalloc", "gbmuf_sync_round_host", "gbmuf_host_create",
           "gbmuf_host_sync_round", "gbmuf_host_destroy", "gbmuf_local_adagrad",
           "gbmuf_selftest_wait_timeout", "gbmuf_selftest_divide", "gbmuf_peer_create", "gbmuf_peer_set_partition",
           "gbmuf_peer_sync_round", "gbmuf_peer_device_status", "gbmuf_peer_destroy"]


class Config(ctypes.Structure):
    """Mirror of ``gbmuf_config``."""
    _fields_ = [("K", ctypes.c_int32), ("N", ctypes.c_int64), ("ld", ctypes.c_int64),
                ("p", ctypes.c_int32), ("q", ctypes.c_int32), ("eta", ctypes.c_float),
                ("zeta", ctypes.c_float), ("mode", ctypes.c_int32), ("theta_dtype", ctypes.c_int32),
                ("seed", ctypes.c_uint64), ("device", ctypes.c_int32), ("comp_base", ctypes.c_int32),
                ("elem_base", ctypes.c_int64)]


class GbmufError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gbmuf status {status} ({STATUS_NAMES.get(status, '?')}): {message}")
        self.status = status


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it is not built: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_1909_09010_b200.build` "
                           "(nvcc, sm_100a).  There is no CPU or other fallback.")
    L = ctypes.CDLL(path)
    i32, i64, u64, f32, vp = (ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_float,
                              ctypes.c_void_p)
    L.gbmuf_create.argtypes = [ctypes.POINTER(Config), vp, vp, vp, ctypes.POINTER(vp)]
    L.gbmuf_set_partition.argtypes = [vp, i32, vp, vp]
    L.gbmuf_init.argtypes = [vp, vp, vp]
    L.gbmuf_local_perturb.argtypes = [vp, u64, f32, f32, i32, vp]
    L.gbmuf_local_adagrad.argtypes = [vp, vp, vp, f32, f32, f32, vp, vp]
    L.gbmuf_sync_round.argtypes = [vp, u64, vp, vp]
    L.gbmuf_get_neighbors.argtypes = [vp, u64, vp]
    L.gbmuf_final_average.argtypes = [vp, vp, vp]
    L.gbmuf_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    L.gbmuf_set_tuning.argtypes = [vp, i32, i32, i32, i32, i32]
    L.gbmuf_get_launch_info.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i32),
                                        ctypes.POINTER(i32), ctypes.POINTER(i32),
                                        ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.gbmuf_sync_round_noalloc.argtypes = [ctypes.POINTER(Config), vp, vp, vp, i32, vp, vp, u64, vp,
                                           ctypes.POINTER(i32)]
    L.gbmuf_sync_round_host.argtypes = [ctypes.POINTER(Config), vp, vp, vp, i32, vp, vp, u64, i64]
    L.gbmuf_host_create.argtypes = [ctypes.POINTER(Config), i32, vp, i64, i32, ctypes.POINTER(vp)]
    L.gbmuf_host_sync_round.argtypes = [vp, vp, vp, vp, vp, u64]
    L.gbmuf_host_destroy.argtypes = [vp]
    L.gbmuf_selftest_wait_timeout.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double)]
    L.gbmuf_selftest_divide.argtypes = [vp, i32, vp, ctypes.POINTER(u64), ctypes.POINTER(ctypes.c_uint32)]
    L.gbmuf_peer_create.argtypes = [ctypes.POINTER(Config), i32, vp, vp, vp, ctypes.POINTER(vp)]
    L.gbmuf_peer_set_partition.argtypes = [vp, i32, vp, vp]
    L.gbmuf_peer_sync_round.argtypes = [vp, u64, vp, i32, vp]
    L.gbmuf_peer_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    L.gbmuf_peer_destroy.argtypes = [vp]
    L.gbmuf_last_error.argtypes = [vp]
    L.gbmuf_last_error.restype = ctypes.c_char_p
    L.gbmuf_destroy.argtypes = [vp]
    for name in EXPORTS:
        if name != "gbmuf_last_error":
            getattr(L, name).restype = i32
    _lib = L
    return L


def _ptr(t) -> int:
    """Device (torch tensor) or host (numpy array) address; None -> NULL."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def sync_round_noalloc(theta, omega, delta, offsets, rnd, *, K, N, ld, p, q, eta, zeta, seed=0,
                       mode=MODE_BMUF, theta_dtype=F32, device=0, comp_base=0, elem_base=0,
                       comp_mask=None, stream=None, want_status=False):
    """``gbmuf_sync_round_noalloc``: one round without a context and without any allocation by the
    library (its tables live in a fixed array of the loaded library).  For callers that cannot
    allocate device memory where they synchronise.  Calls on one GPU share that array: keep them
    on one stream.  Returns the device status word if ``want_status`` (this waits for the stream).
    """
    cfg = Config(K, N, ld, p, q, eta, zeta, mode, theta_dtype, seed, device, comp_base, elem_base)
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    mask = None if comp_mask is None else np.ascontiguousarray(comp_mask, dtype=np.uint8)
    word = ctypes.c_int32(-1)
    st = lib().gbmuf_sync_round_noalloc(ctypes.byref(cfg), _ptr(theta), _ptr(omega), _ptr(delta),
                                        off.shape[0] - 1, _ptr(off), _ptr(mask), rnd,
                                        _stream(stream), ctypes.byref(word) if want_status else None)
    if st != GBMUF_OK:
        raise GbmufError(st, lib().gbmuf_last_error(None).decode())
    return word.value if want_status else None


def sync_round_host(theta, omega, delta, offsets, rnd, *, K, N, ld, p, q, eta, zeta, seed=0,
                    mode=MODE_BMUF, theta_dtype=F32, device=0, comp_base=0, elem_base=0,
                    comp_mask=None, chunk_cols=0):
    """``gbmuf_sync_round_host``: one round over HOST arrays [K][ld] (numpy arrays or CPU torch
    tensors, ideally page-locked), streamed through the GPU in column chunks.  Synchronous."""
    cfg = Config(K, N, ld, p, q, eta, zeta, mode, theta_dtype, seed, device, comp_base, elem_base)
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    mask = None if comp_mask is None else np.ascontiguousarray(comp_mask, dtype=np.uint8)
    st = lib().gbmuf_sync_round_host(ctypes.byref(cfg), _ptr(theta), _ptr(omega), _ptr(delta),
                                     off.shape[0] - 1, _ptr(off), _ptr(mask), rnd, chunk_cols)
    if st != GBMUF_OK:
        raise GbmufError(st, lib().gbmuf_last_error(None).decode())


class GbmufHost:
    """``gbmuf_host_*``: rounds over HOST arrays [K][ld] with the device chunk buffers, streams and
    chunk tables kept across rounds (``sync_round_host`` sets them up and frees them per call)."""

    def __init__(self, offsets, *, K, N, ld, p, q, eta, zeta, seed=0, mode=MODE_BMUF, theta_dtype=F32,
                 device=0, comp_base=0, elem_base=0, chunk_cols=0, row_copies=False):
        self._h = ctypes.c_void_p()
        cfg = Config(K, N, ld, p, q, eta, zeta, mode, theta_dtype, seed, device, comp_base, elem_base)
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        self.m = off.shape[0] - 1
        st = lib().gbmuf_host_create(ctypes.byref(cfg), self.m, _ptr(off), chunk_cols,
                                     1 if row_copies else 0, ctypes.byref(self._h))
        if st != GBMUF_OK:
            raise GbmufError(st, lib().gbmuf_last_error(None).decode())

    def sync_round(self, theta, omega, delta, rnd, comp_mask=None):
        mask = None if comp_mask is None else np.ascontiguousarray(comp_mask, dtype=np.uint8)
        if mask is not None and mask.shape[0] != self.m:
            raise ValueError("comp_mask must have one entry per component")
        st = lib().gbmuf_host_sync_round(self._h, _ptr(theta), _ptr(omega), _ptr(delta), _ptr(mask), rnd)
        if st != GBMUF_OK:
            raise GbmufError(st, lib().gbmuf_last_error(None).decode())

    def destroy(self):
        if self._h:
            lib().gbmuf_host_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class GbmufPeer:
    """One worker of the one-worker-per-GPU form.  ``theta_bufs[b][j]`` is buffer b (0/1) of worker j
    (tensors or raw device addresses; entry ``rank`` is this worker's own memory)."""

    def __init__(self, rank, theta_bufs, omega, delta, *, K, N, ld, p, q, eta, zeta, seed=0,
                 mode=MODE_BMUF, theta_dtype=F32, device=0, comp_base=0):
        self._h = ctypes.c_void_p()
        self.cfg = Config(K, N, ld, p, q, eta, zeta, mode, theta_dtype, seed, device, comp_base, 0)
        self._keep = (theta_bufs, omega, delta)
        addr = [(t if isinstance(t, int) else t.data_ptr()) for b in (0, 1) for t in theta_bufs[b]]
        arr = (ctypes.c_void_p * (2 * K))(*addr)
        st = lib().gbmuf_peer_create(ctypes.byref(self.cfg), rank, arr, _ptr(omega), _ptr(delta),
                                     ctypes.byref(self._h))
        if st != GBMUF_OK:
            raise GbmufError(st, lib().gbmuf_last_error(None).decode())
        self.m = 0

    def _check(self, st):
        if st != GBMUF_OK:
            raise GbmufError(st, lib().gbmuf_last_error(None).decode())

    def set_partition(self, offsets, periods=None):
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        per = None if periods is None else np.ascontiguousarray(periods, dtype=np.int32)
        self._check(lib().gbmuf_peer_set_partition(self._h, off.shape[0] - 1, _ptr(off), _ptr(per)))
        self.m = off.shape[0] - 1

    def sync_round(self, rnd, read_buffer, comp_mask=None, stream=None):
        mask = None if comp_mask is None else np.ascontiguousarray(comp_mask, dtype=np.uint8)
        self._check(lib().gbmuf_peer_sync_round(self._h, rnd, _ptr(mask), read_buffer, _stream(stream)))

    def device_status(self, stream=None) -> int:
        v = ctypes.c_int32(-1)
        self._check(lib().gbmuf_peer_device_status(self._h, _stream(stream), ctypes.byref(v)))
        return v.value

    def destroy(self):
        if self._h:
            lib().gbmuf_peer_destroy(self._h)
            self._h = ctypes.c_void_p()
            self._keep = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Gbmuf:
    """One context: K replicas [K][ld] in caller-owned device tensors theta / omega / delta."""

    def __init__(self, theta, omega, delta, *, K, N, ld, p, q, eta, zeta, seed=0, mode=MODE_BMUF,
                 theta_dtype=F32, device=0, comp_base=0, elem_base=0):
        self._h = ctypes.c_void_p()
        self.cfg = Config(K, N, ld, p, q, eta, zeta, mode, theta_dtype, seed, device, comp_base,
                          elem_base)
        self._keep = (theta, omega, delta)
        self.m = 0
        st = lib().gbmuf_create(ctypes.byref(self.cfg), _ptr(theta), _ptr(omega), _ptr(delta),
                                ctypes.byref(self._h))
        if st != GBMUF_OK:
            raise GbmufError(st, lib().gbmuf_last_error(None).decode())

    def _check(self, st: int):
        if st != GBMUF_OK:
            raise GbmufError(st, lib().gbmuf_last_error(self._h).decode())

    def set_partition(self, offsets, periods=None):
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        per = None if periods is None else np.ascontiguousarray(periods, dtype=np.int32)
        m = off.shape[0] - 1
        if per is not None and per.shape[0] != m:
            raise ValueError("periods must have one entry per component")
        self._check(lib().gbmuf_set_partition(self._h, m, _ptr(off), _ptr(per)))
        self.m = m

    def init(self, theta0, stream=None):
        self._check(lib().gbmuf_init(self._h, _ptr(theta0), _stream(stream)))

    def local_perturb(self, step, lr, sigma, nsteps=1, stream=None):
        self._check(lib().gbmuf_local_perturb(self._h, step, lr, sigma, nsteps, _stream(stream)))

    def local_adagrad(self, grad, accum, lr, eps=0.0, clip_norm=0.0, clip_mask=None, stream=None):
        mask = None
        if clip_mask is not None:
            mask = np.ascontiguousarray(clip_mask, dtype=np.uint8)
            if mask.shape[0] != self.m:
                raise ValueError("clip_mask must have one entry per component")
        self._check(lib().gbmuf_local_adagrad(self._h, _ptr(grad), _ptr(accum), lr, eps, clip_norm,
                                              _ptr(mask), _stream(stream)))

    def sync_round(self, rnd, comp_mask=None, stream=None):
        mask = None
        if comp_mask is not None:
            mask = np.ascontiguousarray(comp_mask, dtype=np.uint8)
            if mask.shape[0] != self.m:
                raise ValueError("comp_mask must have one entry per component")
        self._check(lib().gbmuf_sync_round(self._h, rnd, _ptr(mask), _stream(stream)))

    def get_neighbors(self, rnd) -> np.ndarray:
        out = np.full((self.cfg.K, self.m, self.cfg.q), -1, dtype=np.int32)
        self._check(lib().gbmuf_get_neighbors(self._h, rnd, _ptr(out)))
        return out

    def final_average(self, out, stream=None):
        """The returned model of Algorithm 1.  Also the point where a training run ends, so the
        device status word is read here (this waits for the stream): a bounded device-side wait
        that expired in any earlier round would otherwise go unnoticed."""
        self._check(lib().gbmuf_final_average(self._h, _ptr(out), _stream(stream)))
        self.raise_on_device_error(stream)

    def raise_on_device_error(self, stream=None):
        """Reads (and clears) the device status word; raises if a kernel reported a failure."""
        word = self.device_status(stream)
        if word != GBMUF_OK:
            raise GbmufError(word, "a device-side wait expired in an earlier call on this context; "
                                   "theta, omega and Delta are unspecified")

    def device_status(self, stream=None) -> int:
        v = ctypes.c_int32(-1)
        self._check(lib().gbmuf_device_status(self._h, _stream(stream), ctypes.byref(v)))
        return v.value

    def selftest_wait_timeout(self, stream=None) -> float:
        """Lets a bounded device-side wait expire on purpose; returns the kernel's duration (s)."""
        sec = ctypes.c_double(0.0)
        self._check(lib().gbmuf_selftest_wait_timeout(self._h, _stream(stream), ctypes.byref(sec)))
        return sec.value

    def selftest_divide(self, divisor: int, stream=None) -> tuple[int, int]:
        """Compares the kernels' averaging division with the plain division over all 2^32
        dividends; returns (number of differing patterns, smallest differing pattern)."""
        bad, first = ctypes.c_uint64(0), ctypes.c_uint32(0)
        self._check(lib().gbmuf_selftest_divide(self._h, divisor, _stream(stream), ctypes.byref(bad),
                                                ctypes.byref(first)))
        return bad.value, first.value

    def set_tuning(self, consumer_threads=0, tile_elems=0, theta_stages=0, ring_slots=0, flags=0):
        self._check(lib().gbmuf_set_tuning(self._h, consumer_threads, tile_elems, theta_stages,
                                           ring_slots, flags))

    def launch_info(self) -> dict:
        tiles = ctypes.c_int64()
        g, b, s, t, st = (ctypes.c_int32() for _ in range(5))
        self._check(lib().gbmuf_get_launch_info(self._h, ctypes.byref(tiles), ctypes.byref(g),
                                                ctypes.byref(b), ctypes.byref(s), ctypes.byref(t),
                                                ctypes.byref(st)))
        return {"tiles": tiles.value, "grid": g.value, "block": b.value, "smem_bytes": s.value,
                "tile_elems": t.value, "stages": st.value,
                "variant": "tmem" if st.value == 0 else "tmem-window" if st.value < 0
                else "smem-window" if st.value >= 1000 else "smem"}

    def last_error(self) -> str:
        return lib().gbmuf_last_error(self._h).decode()

    def destroy(self, check_status=True):
        """Frees the context.  Reads the device status word first (unless told not to) and raises
        after freeing if an earlier round reported a failure nobody has looked at."""
        if self._h:
            word = GBMUF_OK
            if check_status:
                try:
                    word = self.device_status()
                except Exception:
                    word = GBMUF_OK
            st = lib().gbmuf_destroy(self._h)
            self._h = ctypes.c_void_p()
            self._keep = None
            if st != GBMUF_OK:
                raise GbmufError(st, "destroy failed")
            if word != GBMUF_OK:
                raise GbmufError(word, "a device-side wait expired in an earlier call on this context "
                                       "and was never read; its results were unspecified")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
