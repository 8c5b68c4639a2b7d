"""TEST INFRASTRUCTURE: ctypes front end of the fp64 CPU oracle (``peagle_oracle.c``).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It never touches the CUDA library.  ``build()`` compiles the C file with gcc into
``oracle/libpeagle_oracle.so``; building it is not using it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "peagle_oracle.c")
_SO = os.path.join(_HERE, "libpeagle_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        _lib.peagle_oracle_count_pairs.restype = ctypes.c_int64
    return _lib


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(t):
    """bf16/fp32 torch tensor or array -> contiguous float32 numpy (exact for bf16 values)."""
    if hasattr(t, "detach"):
        t = t.detach().cpu().float().numpy()
    return np.ascontiguousarray(t, dtype=np.float32)


def _kranges(kranges):
    if kranges is None or len(kranges) == 0:
        return np.zeros((0, 2), np.int32), 0
    kr = _i32(kranges).reshape(-1, 2)
    return kr, kr.shape[0]


def num_threads() -> int:
    return int(_load().peagle_oracle_num_threads())


def allowed(a_q: int, d_q: int, a_k: int, d_k: int) -> bool:
    return bool(_load().peagle_oracle_allowed(int(a_q), int(d_q), int(a_k), int(d_k)))


def mask_dense(anchor, depth, seq_id=None) -> np.ndarray:
    """The materialised parallel-prediction mask, uint8 [T][T]."""
    anchor, depth = _i32(anchor), _i32(depth)
    T = anchor.shape[0]
    seq_id = np.zeros(T, np.int32) if seq_id is None else _i32(seq_id)
    M = np.zeros((T, T), np.uint8)
    _load().peagle_oracle_mask_dense(T, _p(seq_id, ctypes.c_int32), _p(anchor, ctypes.c_int32),
                                     _p(depth, ctypes.c_int32), _p(M, ctypes.c_uint8))
    return M


def count_pairs(anchor, depth, rows=None, kranges=None) -> int:
    anchor, depth = _i32(anchor), _i32(depth)
    T = anchor.shape[0]
    rows = _i32(np.arange(T) if rows is None else rows)
    kr, nk = _kranges(kranges)
    return int(_load().peagle_oracle_count_pairs(
        T, _p(anchor, ctypes.c_int32), _p(depth, ctypes.c_int32), _p(kr, ctypes.c_int32), nk,
        _p(rows, ctypes.c_int32), rows.shape[0]))


def classify_tiles(anchor, depth, q_begin, q_end, kranges, BM, BN):
    """Tile classes (0 SKIP, 1 PARTIAL, 2 FULL) [n_qtiles][n_ktiles] plus key-tile starts/lengths."""
    anchor, depth = _i32(anchor), _i32(depth)
    T = anchor.shape[0]
    kr, nk = _kranges(kranges)
    lib = _load()
    args = (T, _p(anchor, ctypes.c_int32), _p(depth, ctypes.c_int32), int(q_begin), int(q_end),
            _p(kr, ctypes.c_int32), nk, int(BM), int(BN))
    n_kt = lib.peagle_oracle_classify_tiles(*args, None, None, None)
    n_qt = (q_end - q_begin + BM - 1) // BM
    out = np.zeros((n_qt, n_kt), np.uint8)
    ks = np.zeros(n_kt, np.int32)
    kl = np.zeros(n_kt, np.int32)
    lib.peagle_oracle_classify_tiles(*args, _p(out, ctypes.c_uint8), _p(ks, ctypes.c_int32),
                                     _p(kl, ctypes.c_int32))
    return out, ks, kl


def attn_fwd(anchor, depth, Q, K, V, scale, rows=None, kranges=None, heads=None):
    """O [nrows][nheads][D] and LSE [nrows][nheads] in fp64 for one sequence."""
    anchor, depth = _i32(anchor), _i32(depth)
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    T, Hq, D = Q.shape
    Hkv = K.shape[1]
    rows = _i32(np.arange(T) if rows is None else rows)
    h0, h1 = (0, Hq) if heads is None else heads
    kr, nk = _kranges(kranges)
    O = np.zeros((rows.shape[0], h1 - h0, D), np.float64)
    LSE = np.zeros((rows.shape[0], h1 - h0), np.float64)
    rc = _load().peagle_oracle_attn_fwd(
        T, _p(anchor, ctypes.c_int32), _p(depth, ctypes.c_int32), Hq, Hkv, D,
        ctypes.c_double(scale), _p(kr, ctypes.c_int32), nk, _p(rows, ctypes.c_int32),
        rows.shape[0], h0, h1, _p(Q, ctypes.c_float), _p(K, ctypes.c_float),
        _p(V, ctypes.c_float), _p(O, ctypes.c_double), _p(LSE, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle attn_fwd: bad head arguments")
    return O, LSE


def attn_bwd(anchor, depth, Q, K, V, dO, scale, rows=None, kranges=None, heads=None,
             dK=None, dV=None):
    """dQ [nrows][nheads][D]; dK, dV [T][Hkv][D] fp64, accumulated into when passed in."""
    anchor, depth = _i32(anchor), _i32(depth)
    Q, K, V, dO = _f32(Q), _f32(K), _f32(V), _f32(dO)
    T, Hq, D = Q.shape
    Hkv = K.shape[1]
    rows = _i32(np.arange(T) if rows is None else rows)
    h0, h1 = (0, Hq) if heads is None else heads
    kr, nk = _kranges(kranges)
    dQ = np.zeros((rows.shape[0], h1 - h0, D), np.float64)
    dK = np.zeros((T, Hkv, D), np.float64) if dK is None else dK
    dV = np.zeros((T, Hkv, D), np.float64) if dV is None else dV
    assert dK.dtype == np.float64 and dK.flags.c_contiguous
    assert dV.dtype == np.float64 and dV.flags.c_contiguous
    rc = _load().peagle_oracle_attn_bwd(
        T, _p(anchor, ctypes.c_int32), _p(depth, ctypes.c_int32), Hq, Hkv, D,
        ctypes.c_double(scale), _p(kr, ctypes.c_int32), nk, _p(rows, ctypes.c_int32),
        rows.shape[0], h0, h1, _p(Q, ctypes.c_float), _p(K, ctypes.c_float),
        _p(V, ctypes.c_float), _p(dO, ctypes.c_float), _p(dQ, ctypes.c_double),
        _p(dK, ctypes.c_double), _p(dV, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle attn_bwd: bad head arguments")
    return dQ, dK, dV
