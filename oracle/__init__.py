"""ctypes front of the CPU oracle (``gbmuf_oracle.cpp``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the test suite, the smoke check and the bench's
CPU-baseline leg may import this package.  Every arithmetic step lives in the C++ file; this
module only compiles it (g++), loads it and marshals numpy arrays.  It imports nothing from the
CUDA package.

bf16 arrays are carried as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gbmuf_oracle.cpp")
_LIB = os.path.join(_HERE, "libgbmuf_oracle.so")

F32, BF16 = 0, 1
MODE_BMUF, MODE_MA = 0, 1

CXXFLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compile the oracle with g++; returns the path of the shared object."""
    out = out or _LIB
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
        return out
    tmp = out + f".tmp{os.getpid()}"
    subprocess.run(["g++", *CXXFLAGS, *extra_flags, _SRC, "-o", tmp], check=True)
    os.replace(tmp, out)
    return out


def _bind(path: str) -> ctypes.CDLL:
    L = ctypes.CDLL(path)
    i32, i64, u64, f32, vp = (ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_float,
                              ctypes.c_void_p)
    L.gbo_philox4x32_10.argtypes = [vp, vp, vp]
    L.gbo_philox4x32_10.restype = None
    L.gbo_f32_to_bf16.argtypes = [f32]
    L.gbo_f32_to_bf16.restype = ctypes.c_uint16
    L.gbo_bf16_to_f32.argtypes = [ctypes.c_uint16]
    L.gbo_bf16_to_f32.restype = f32
    L.gbo_f32_to_bf16_array.argtypes = [vp, vp, i64]
    L.gbo_f32_to_bf16_array.restype = None
    L.gbo_candidate_list.argtypes = [i32, i32, i32, vp]
    L.gbo_candidate_list.restype = i32
    L.gbo_sample_neighbors.argtypes = [u64, u64, i32, i32, i32, i32, i32, vp]
    L.gbo_sample_neighbors.restype = i32
    L.gbo_sync_round.argtypes = [i32, i64, i64, i32, vp, vp, vp, vp, vp, i32, vp, vp, vp, i32,
                                 f32, f32, i32, vp]
    L.gbo_sync_round.restype = i32
    L.gbo_init.argtypes = [i32, i64, i64, i32, vp, vp, vp, vp, vp]
    L.gbo_init.restype = i32
    L.gbo_local_perturb.argtypes = [i32, i64, i64, i32, vp, u64, u64, f32, f32, i32, i64]
    L.gbo_local_perturb.restype = i32
    L.gbo_local_adagrad.argtypes = [i32, i64, i64, i32, vp, vp, vp, f32, f32, f32, i32, vp]
    L.gbo_local_adagrad.restype = i32
    L.gbo_final_average.argtypes = [i32, i64, i64, i32, vp, vp]
    L.gbo_final_average.restype = i32
    return L


_lib_cache: ctypes.CDLL | None = None


def lib() -> ctypes.CDLL:
    global _lib_cache
    if _lib_cache is None:
        # GBMUF_ORACLE_LIB: the mutation test points the pins at a deliberately broken copy
        _lib_cache = _bind(os.environ.get("GBMUF_ORACLE_LIB") or build())
    return _lib_cache


def _ptr(a: np.ndarray | None):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _tdtype(dtype: int):
    return np.float32 if dtype == F32 else np.uint16


# ------------------------------------------------------------------------------------------------
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().gbo_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().gbo_f32_to_bf16_array(_ptr(x), _ptr(out), x.size)
    return out


def bf16_to_f32(h: np.ndarray) -> np.ndarray:
    """Exact widening; a pure bit move, done in numpy."""
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << 16).view(np.float32)


def candidate_list(k: int, K: int, p: int) -> list[int]:
    buf = np.zeros(max(2 * p, 1), dtype=np.int32)
    c = lib().gbo_candidate_list(k, K, p, _ptr(buf))
    if c < 0:
        raise ValueError("bad arguments")
    return [int(v) for v in buf[:c]]


def sample_neighbors(seed: int, rnd: int, K: int, m: int, p: int, q: int,
                     comp_base: int = 0) -> np.ndarray:
    """Neighbour table [K][m][q] (int32) of one round."""
    out = np.full((K, m, q), -1, dtype=np.int32)
    rc = lib().gbo_sample_neighbors(seed, rnd, K, m, comp_base, p, q, _ptr(out))
    if rc != 0:
        raise ValueError("bad arguments (q larger than the candidate set?)")
    return out


@dataclass
class State:
    """Host-side state of K simulated workers: theta, omega, Delta and the stored block-start
    value rst (all [K][ld])."""
    K: int
    N: int
    ld: int
    dtype: int
    theta: np.ndarray
    omega: np.ndarray
    delta: np.ndarray
    rst: np.ndarray

    def copy(self) -> "State":
        return State(self.K, self.N, self.ld, self.dtype, self.theta.copy(), self.omega.copy(),
                     self.delta.copy(), self.rst.copy())

    def theta_f32(self) -> np.ndarray:
        return self.theta if self.dtype == F32 else bf16_to_f32(self.theta)


def init(theta0: np.ndarray, K: int, ld: int | None = None, dtype: int = F32) -> State:
    """Algorithm 1's initialisation line for K workers from one theta_0 of length N."""
    theta0 = np.ascontiguousarray(theta0, dtype=_tdtype(dtype))
    N = theta0.shape[0]
    ld = N if ld is None else ld
    st = State(K, N, ld, dtype,
               np.zeros((K, ld), dtype=_tdtype(dtype)), np.zeros((K, ld), dtype=np.float32),
               np.zeros((K, ld), dtype=np.float32), np.zeros((K, ld), dtype=_tdtype(dtype)))
    rc = lib().gbo_init(K, N, ld, dtype, _ptr(theta0), _ptr(st.theta), _ptr(st.omega),
                        _ptr(st.delta), _ptr(st.rst))
    assert rc == 0
    return st


def sync_round(st: State, offsets, nbr: np.ndarray, eta: float, zeta: float, mode: int = MODE_BMUF,
               sync=None, order=None, want_g: bool = False):
    """One synchronisation round, in place on ``st``.  Returns G ([K][ld]) if asked."""
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    m = off.shape[0] - 1
    nbr = np.ascontiguousarray(nbr, dtype=np.int32)
    assert nbr.shape[0] == st.K and nbr.shape[1] == m
    q = nbr.shape[2]
    assert off[0] >= 0 and off[m] <= st.N and np.all(np.diff(off) >= 0)
    if q:
        assert nbr.min() >= 0 and nbr.max() < st.K
    sy = None if sync is None else np.ascontiguousarray(sync, dtype=np.uint8)
    od = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
    g = np.zeros((st.K, st.ld), dtype=np.float32) if want_g else None
    rc = lib().gbo_sync_round(st.K, st.N, st.ld, st.dtype, _ptr(st.theta), _ptr(st.omega),
                              _ptr(st.delta), _ptr(st.rst), _ptr(g), m, _ptr(off), _ptr(sy),
                              _ptr(nbr), q, eta, zeta, mode, _ptr(od))
    assert rc == 0
    return g


def local_perturb(st: State, seed: int, step: int, lr: float, sigma: float, nsteps: int = 1,
                  elem_base: int = 0) -> None:
    rc = lib().gbo_local_perturb(st.K, st.N, st.ld, st.dtype, _ptr(st.theta), seed, step, lr, sigma,
                                 nsteps, elem_base)
    if rc != 0:
        raise ValueError("bad arguments")


def local_adagrad(st: State, grad: np.ndarray, accum: np.ndarray, lr: float, eps: float = 0.0,
                  clip_norm: float = 0.0, ranges=()) -> None:
    """Adagrad local step with group gradient-norm clipping, in place on st.theta and accum."""
    grad = np.ascontiguousarray(grad, dtype=np.float32)
    assert grad.shape == (st.K, st.ld) and accum.shape == (st.K, st.ld) and accum.dtype == np.float32
    rg = np.ascontiguousarray(np.asarray(ranges, dtype=np.int64).reshape(-1, 2))
    rc = lib().gbo_local_adagrad(st.K, st.N, st.ld, st.dtype, _ptr(st.theta), _ptr(grad), _ptr(accum),
                                 lr, eps, clip_norm, rg.shape[0], _ptr(rg) if rg.size else None)
    if rc != 0:
        raise ValueError("bad arguments")


def final_average(st: State) -> np.ndarray:
    out = np.zeros(st.N, dtype=_tdtype(st.dtype))
    rc = lib().gbo_final_average(st.K, st.N, st.ld, st.dtype, _ptr(st.theta), _ptr(out))
    assert rc == 0
    return out
