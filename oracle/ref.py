"""ctypes wrapper around the CPU checker (``relaygr_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Imported by ``tests/``, by ``bench.py``'s CPU
baseline leg and by the smoke check; never by the product package, and it
imports nothing from it.  Arithmetic is fp64; parameters are fp32 arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "relaygr_oracle.c")
_LIB = os.path.join(_HERE, "librelaygr_oracle.so")


class _Cfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("d_head", C.c_int32), ("d_ff", C.c_int32), ("ln_eps", C.c_double), ("attn_kind", C.c_int32)]


_WNAMES = ["emb", "ln1_g", "ln1_b", "ln2_g", "ln2_b", "w_qkv", "b_qkv", "w_o", "b_o",
           "w1", "b1", "w2", "b2", "lnf_g", "lnf_b", "w_score", "b_score"]


class _W(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WNAMES]


def build(force: bool = False) -> str:
    """Compile the checker with gcc (OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=gnu11",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(build())
        i64, p = C.c_int64, C.c_void_p
        l.orc_full.argtypes = [C.POINTER(_Cfg), C.POINTER(_W), i64, p, i64, p, i64, p, p]
        l.orc_preinfer.argtypes = [C.POINTER(_Cfg), C.POINTER(_W), i64, p, p, p]
        l.orc_rank_cached.argtypes = [C.POINTER(_Cfg), C.POINTER(_W), i64, p, p, i64, p, i64, p, p]
        l.orc_kv_bytes.argtypes = [i64, i64, i64, i64]
        l.orc_kv_bytes.restype = i64
        _lib = l
    return _lib


def n_threads() -> int:
    """Threads the checker's OpenMP loops use on this machine."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


class Model:
    """Holds fp32 parameter arrays (kept alive) and the C structs built on them.

    ``params`` maps the names emb, ln1_g, ln1_b, ln2_g, ln2_b, w_qkv, b_qkv,
    w_o, b_o, w1, b1, w2, b2, lnf_g, lnf_b, w_score, b_score to fp32 arrays;
    linear weights are ``[L, out, in]``; a bias may be ``None``.  ``attn_kind``: 0 softmax attention,
    1 pointwise SiLU attention (the checker's header states both).
    """

    def __init__(self, n_layers: int, d_model: int, n_heads: int, d_head: int, d_ff: int,
                 ln_eps: float, params: Dict[str, Optional[np.ndarray]], attn_kind: int = 0):
        assert n_heads * d_head == d_model and attn_kind in (0, 1)
        self.cfg = _Cfg(n_layers, d_model, n_heads, d_head, d_ff, float(ln_eps), int(attn_kind))
        self.L, self.d = n_layers, d_model
        self._keep = {}
        self.w = _W()
        for name in _WNAMES:
            a = params.get(name)
            if a is None:
                setattr(self.w, name, None)
                continue
            a = np.ascontiguousarray(a, dtype=np.float32)
            self._keep[name] = a
            setattr(self.w, name, a.ctypes.data)

    @staticmethod
    def _ids(a) -> np.ndarray:
        return np.ascontiguousarray(a, dtype=np.int32)

    def full(self, prefix_ids, short_ids, cand_ids) -> np.ndarray:
        p, s, c = self._ids(prefix_ids), self._ids(short_ids), self._ids(cand_ids)
        out = np.zeros(len(c), dtype=np.float64)
        rc = lib().orc_full(C.byref(self.cfg), C.byref(self.w), len(p), p.ctypes.data, len(s), s.ctypes.data,
                            len(c), c.ctypes.data, out.ctypes.data)
        assert rc == 0
        return out

    def preinfer(self, prefix_ids) -> Tuple[np.ndarray, np.ndarray]:
        p = self._ids(prefix_ids)
        K = np.zeros((self.L, len(p), self.d), dtype=np.float64)
        V = np.zeros_like(K)
        rc = lib().orc_preinfer(C.byref(self.cfg), C.byref(self.w), len(p), p.ctypes.data,
                                K.ctypes.data, V.ctypes.data)
        assert rc == 0
        return K, V

    def rank_cached(self, K: np.ndarray, V: np.ndarray, short_ids, cand_ids) -> np.ndarray:
        K = np.ascontiguousarray(K, dtype=np.float64)
        V = np.ascontiguousarray(V, dtype=np.float64)
        assert K.shape == V.shape and K.shape[0] == self.L and K.shape[2] == self.d
        s, c = self._ids(short_ids), self._ids(cand_ids)
        out = np.zeros(len(c), dtype=np.float64)
        rc = lib().orc_rank_cached(C.byref(self.cfg), C.byref(self.w), K.shape[1], K.ctypes.data, V.ctypes.data,
                                   len(s), s.ctypes.data, len(c), c.ctypes.data, out.ctypes.data)
        assert rc == 0
        return out


def kv_bytes(prefix_len: int, n_layers: int, d_model: int, elem_bytes: int) -> int:
    return int(lib().orc_kv_bytes(prefix_len, n_layers, d_model, elem_bytes))
