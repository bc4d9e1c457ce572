"""ctypes front end of the float64 CPU oracle (``bcjr_oracle.c``, ``bcjr_oracle_vec.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by
``bench.py``'s CPU-baseline leg.  The CUDA package never imports this module and this
module never imports the CUDA package.

Inputs are the float32 arrays of the seeded generators, promoted exactly to float64;
outputs are float64 (soft codeword, gradients, log Z) or integers (Viterbi).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRCS = [_HERE / "bcjr_oracle.c", _HERE / "bcjr_oracle_vec.c"]
_LIB = _HERE / "libbcjr_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fused multiply-add contraction, OpenMP over blocks)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < max(f.stat().st_mtime for f in _SRCS):
        cmd = ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", *map(str, _SRCS), "-o", str(_LIB), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_soft_quantize.restype = ctypes.c_int
        lib.oracle_soft_quantize.argtypes = [dp, dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int64, ctypes.c_double, dp, dp,
                                             ctypes.c_int64, dp, dp]
        lib.oracle_backward.restype = ctypes.c_int
        lib.oracle_backward.argtypes = [dp, dp, dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_int64, ctypes.c_double, dp, dp]
        lib.oracle_viterbi.restype = ctypes.c_int
        lib.oracle_viterbi.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                       ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                       ctypes.POINTER(ctypes.c_uint16), ctypes.POINTER(ctypes.c_float),
                                       ctypes.POINTER(ctypes.c_uint8), ctypes.c_int64, dp]
        ci, c64, cd = ctypes.c_int, ctypes.c_int64, ctypes.c_double
        lib.oracle_vec_soft_quantize.restype = ci
        lib.oracle_vec_soft_quantize.argtypes = [dp, dp, ci, ci, ci, ci, c64, cd, dp, dp]
        lib.oracle_vec_backward.restype = ci
        lib.oracle_vec_backward.argtypes = [dp, dp, dp, ci, ci, ci, ci, c64, cd, dp, dp]
        lib.oracle_vec_viterbi.restype = ci
        lib.oracle_vec_viterbi.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                           ci, ci, ci, ci, c64, ctypes.POINTER(ctypes.c_uint16),
                                           ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_uint8), c64, dp]
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _dptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _check(rc):
    if rc != 0:
        raise RuntimeError({-1: "oracle: invalid argument", -2: "oracle: out of memory"}.get(rc, f"oracle: error {rc}"))


def host_cores() -> int:
    return len(os.sched_getaffinity(0))


def set_threads(Lb: int, n: int, num_blocks: int, arrays_per_thread: int = 5,
                mem_budget_bytes: float = 24e9, limit: int | None = None) -> int:
    """Pick the OpenMP thread count: one block per thread, bounded by cores and by memory
    (each thread holds `arrays_per_thread` float64 arrays of n * 2^Lb entries)."""
    per = arrays_per_thread * n * (1 << Lb) * 8
    t = max(1, min(host_cores(), max(1, num_blocks), int(mem_budget_bytes // max(per, 1)) or 1))
    if limit:
        t = max(1, min(t, limit))
    _load().oracle_set_num_threads(t)
    return t


def path_bytes(Lb: int, k: int, n: int) -> int:
    return (Lb + k * (n - 1) + 7) // 8


def soft_quantize(W, c, Lb, k, T, want_gamma_of=None):
    """Soft codeword of Eq. 7.  W: [B, n].  Returns dict(soft [B,n], logZ [B], and, when
    `want_gamma_of` names a block, gamma [n,S] and logZ_t [n] for it)."""
    lib = _load()
    W = _f64(W); c = _f64(c)
    B, n = W.shape
    assert c.shape == (1 << Lb,)
    set_threads(Lb, n, B, arrays_per_thread=2)
    soft = np.empty((B, n)); logZ = np.empty(B)
    gam = lzt = None
    gb = -1
    if want_gamma_of is not None:
        gb = int(want_gamma_of)
        gam = np.empty((n, 1 << Lb)); lzt = np.empty(n)
    _check(lib.oracle_soft_quantize(_dptr(W), _dptr(c), Lb, k, n, B, float(T), _dptr(soft), _dptr(logZ),
                                    gb, _dptr(gam), _dptr(lzt)))
    out = {"soft": soft, "logZ": logZ}
    if gam is not None:
        out["gamma"] = gam; out["logZ_t"] = lzt
    return out


def backward(W, c, g, Lb, k, T):
    """Gradients of sum(g * soft) w.r.t. W ([B,n]) and the table c ([S], summed over blocks)."""
    lib = _load()
    W = _f64(W); c = _f64(c); g = _f64(g)
    B, n = W.shape
    assert g.shape == W.shape and c.shape == (1 << Lb,)
    set_threads(Lb, n, B, arrays_per_thread=5)
    gW = np.empty((B, n)); gc = np.empty(1 << Lb)
    _check(lib.oracle_backward(_dptr(W), _dptr(c), _dptr(g), Lb, k, n, B, float(T), _dptr(gW), _dptr(gc)))
    return {"grad_W": gW, "grad_codebook": gc}


def viterbi(W, c, Lb, k):
    """Hard code.  W, c float32.  Returns dict(states [B,n] u16, hard [B,n] f32, path_bits [B,nbytes] u8, cost [B])."""
    lib = _load()
    W = np.ascontiguousarray(W, dtype=np.float32); c = np.ascontiguousarray(c, dtype=np.float32)
    B, n = W.shape
    assert c.shape == (1 << Lb,)
    set_threads(Lb, n, B, arrays_per_thread=1)
    nb = path_bytes(Lb, k, n)
    states = np.empty((B, n), dtype=np.uint16); hard = np.empty((B, n), dtype=np.float32)
    bits = np.zeros((B, nb), dtype=np.uint8); cost = np.empty(B)
    _check(lib.oracle_viterbi(W.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                              c.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), Lb, k, n, B,
                              states.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)),
                              hard.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                              bits.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), nb, _dptr(cost)))
    return {"states": states, "hard": hard, "path_bits": bits, "cost": cost}


# ---- vector emissions: state s emits the V numbers c[s, :], a step consumes V weights and kb bits
def soft_quantize_vec(W, c, Lb, kb, V, T):
    """W: [B, n] (n a multiple of V), c: [S, V].  Returns dict(soft [B,n], logZ [B])."""
    lib = _load()
    W = _f64(W); c = _f64(c)
    B, n = W.shape
    assert c.shape == (1 << Lb, V)
    set_threads(Lb, n // V, B, arrays_per_thread=2)
    soft = np.empty((B, n)); logZ = np.empty(B)
    _check(lib.oracle_vec_soft_quantize(_dptr(W), _dptr(c), Lb, kb, V, n, B, float(T), _dptr(soft), _dptr(logZ)))
    return {"soft": soft, "logZ": logZ}


def backward_vec(W, c, g, Lb, kb, V, T):
    """Gradients of sum(g * soft): grad_W [B,n], grad_codebook [S,V] (summed over blocks)."""
    lib = _load()
    W = _f64(W); c = _f64(c); g = _f64(g)
    B, n = W.shape
    assert g.shape == W.shape and c.shape == (1 << Lb, V)
    set_threads(Lb, n // V, B, arrays_per_thread=5)
    gW = np.empty((B, n)); gc = np.empty((1 << Lb, V))
    _check(lib.oracle_vec_backward(_dptr(W), _dptr(c), _dptr(g), Lb, kb, V, n, B, float(T), _dptr(gW), _dptr(gc)))
    return {"grad_W": gW, "grad_codebook": gc}


def viterbi_vec(W, c, Lb, kb, V):
    """Hard code.  Returns dict(states [B, n/V] u16, hard [B,n] f32, path_bits [B,nbytes] u8, cost [B])."""
    lib = _load()
    W = np.ascontiguousarray(W, dtype=np.float32); c = np.ascontiguousarray(c, dtype=np.float32)
    B, n = W.shape
    assert c.shape == (1 << Lb, V) and n % V == 0
    nt = n // V
    set_threads(Lb, nt, B, arrays_per_thread=1)
    nb = path_bytes(Lb, kb, nt)
    states = np.empty((B, nt), dtype=np.uint16); hard = np.empty((B, n), dtype=np.float32)
    bits = np.zeros((B, nb), dtype=np.uint8); cost = np.empty(B)
    _check(lib.oracle_vec_viterbi(W.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                  c.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), Lb, kb, V, n, B,
                                  states.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)),
                                  hard.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                  bits.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), nb, _dptr(cost)))
    return {"states": states, "hard": hard, "path_bits": bits, "cost": cost}


def num_threads() -> int:
    return _load().oracle_num_threads()
