"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, not product code).

Only tests, the smoke check and the benchmark's CPU-baseline / reference arm
import this module.  It imports nothing from the CUDA package and the CUDA
package imports nothing from here.  All arithmetic lives in ``fa_oracle.c``;
this file only allocates numpy arrays and marshals pointers.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fa_oracle.c")
_LIB = os.path.join(_HERE, "build", "libfa_oracle.so")


def build(force: bool = False) -> str:
    """Compile fa_oracle.c with gcc (-O2 -fopenmp) into oracle/build/."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
        ("n_full_k", C.c_int32), ("n_full_v", C.c_int32),
        ("k", C.c_int32), ("norm", C.c_int32),
        ("T", C.c_int64),
        ("L_init", C.c_int32), ("L_local", C.c_int32),
        ("cap_mid", C.c_int32),
        ("scale", C.c_double),
    ]


class _Cache(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "idx_full_k", "idx_comp_k", "idx_full_v", "idx_comp_v",
        "k_init", "v_init", "k_local", "v_local", "k_mid", "v_mid",
        "coef_k", "coef_v", "n_init", "n_local", "n_mid")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.fo_num_threads.restype = C.c_int
        _lib.fo_weight.restype = C.c_double
        _lib.fo_weight.argtypes = [C.c_void_p, C.c_int32]
        _lib.fo_basis_column.argtypes = [C.c_int64, C.c_int32, C.c_int64, C.c_void_p]
        _lib.fo_compress.restype = C.c_int
        _lib.fo_append.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().fo_num_threads())


@dataclass
class OracleConfig:
    B: int
    Hq: int
    Hkv: int
    d: int
    n_full_k: int
    n_full_v: int
    k: int                  # complex states; M = 2k
    T: int
    L_init: int
    L_local: int
    cap_mid: int
    scale: float
    norm: int = 0           # 0 orthogonal weights, 1 literal 1/k

    def c(self) -> _Cfg:
        return _Cfg(self.B, self.Hq, self.Hkv, self.d, self.n_full_k, self.n_full_v, self.k,
                    self.norm, self.T, self.L_init, self.L_local, self.cap_mid, float(self.scale))


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def basis_column(T: int, k: int, j: int) -> np.ndarray:
    """Column j of the matrix in Eq.4, length 2k."""
    f = np.empty(2 * k, dtype=np.float64)
    lib().fo_basis_column(C.c_int64(T), C.c_int32(k), C.c_int64(j), _p(f))
    return f


def weights(cfg: OracleConfig) -> np.ndarray:
    c = cfg.c()
    return np.array([lib().fo_weight(C.byref(c), m) for m in range(2 * cfg.k)], dtype=np.float64)


class OracleCache:
    """The oracle's own cache: natural token-major layouts, all float64."""

    def __init__(self, cfg: OracleConfig, idx_full_k, idx_full_v):
        self.cfg = cfg
        d = cfg.d
        self.idx_full_k = np.ascontiguousarray(idx_full_k, dtype=np.int32).reshape(cfg.Hkv, cfg.n_full_k)
        self.idx_full_v = np.ascontiguousarray(idx_full_v, dtype=np.int32).reshape(cfg.Hkv, cfg.n_full_v)
        self.idx_comp_k = self._complement(self.idx_full_k, d)
        self.idx_comp_v = self._complement(self.idx_full_v, d)
        B, H = cfg.B, cfg.Hkv
        z = lambda *s: np.zeros(s, dtype=np.float64)
        self.k_init, self.v_init = z(B, H, cfg.L_init, d), z(B, H, cfg.L_init, d)
        self.k_local, self.v_local = z(B, H, cfg.L_local, d), z(B, H, cfg.L_local, d)
        self.k_mid, self.v_mid = z(B, H, cfg.cap_mid, cfg.n_full_k), z(B, H, cfg.cap_mid, cfg.n_full_v)
        self.coef_k = z(B, H, 2 * cfg.k, d - cfg.n_full_k)
        self.coef_v = z(B, H, 2 * cfg.k, d - cfg.n_full_v)
        self.n_init = np.zeros(B, dtype=np.int32)
        self.n_local = np.zeros(B, dtype=np.int32)
        self.n_mid = np.zeros(B, dtype=np.int32)

    @staticmethod
    def _complement(idx_full: np.ndarray, d: int) -> np.ndarray:
        rows = []
        for h in range(idx_full.shape[0]):
            keep = np.zeros(d, dtype=bool)
            keep[idx_full[h]] = True
            rows.append(np.nonzero(~keep)[0].astype(np.int32))
        return np.ascontiguousarray(np.stack(rows)) if rows else np.zeros((0, 0), np.int32)

    def c(self) -> _Cache:
        return _Cache(*[_p(getattr(self, n)) for n, _ in _Cache._fields_])

    # ---- the calls -----------------------------------------------------
    def compress(self, K: np.ndarray, V: np.ndarray) -> None:
        """Eq.1-3.  K, V: [B][L][Hkv][d] float64."""
        K = np.ascontiguousarray(K, dtype=np.float64)
        V = np.ascontiguousarray(V, dtype=np.float64)
        L = K.shape[1]
        assert K.shape == (self.cfg.B, L, self.cfg.Hkv, self.cfg.d) and V.shape == K.shape
        c, cc = self.cfg.c(), self.c()
        rc = lib().fo_compress(C.byref(c), C.byref(cc), _p(K), _p(V), C.c_int32(L))
        if rc != 0:
            raise ValueError("oracle: middle segment does not fit")

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """Eq.5.  k_new, v_new: [B][Hkv][d] float64."""
        k_new = np.ascontiguousarray(k_new, dtype=np.float64)
        v_new = np.ascontiguousarray(v_new, dtype=np.float64)
        assert k_new.shape == (self.cfg.B, self.cfg.Hkv, self.cfg.d)
        c, cc = self.cfg.c(), self.c()
        rc = lib().fo_append(C.byref(c), C.byref(cc), _p(k_new), _p(v_new))
        if rc != 0:
            raise ValueError("oracle: middle segment is full")

    def reconstruct(self, b: int, h: int, side: int) -> np.ndarray:
        """Eq.6: dense middle segment [n_mid][d] of K (side 0) or V (side 1)."""
        out = np.zeros((int(self.n_mid[b]), self.cfg.d), dtype=np.float64)
        c, cc = self.cfg.c(), self.c()
        lib().fo_reconstruct(C.byref(c), C.byref(cc), C.c_int(b), C.c_int(h), C.c_int(side), _p(out))
        return out

    def decode(self, q: np.ndarray, heads: tuple[int, int] | None = None) -> np.ndarray:
        """Eq.6: attention output [B][Hq][d].  ``heads=(h0, h1)`` limits the
        work to KV heads h0..h1-1 (other rows of the result stay NaN)."""
        q = np.ascontiguousarray(q, dtype=np.float64)
        assert q.shape == (self.cfg.B, self.cfg.Hq, self.cfg.d)
        out = np.full_like(q, np.nan)
        h0, h1 = heads if heads is not None else (0, self.cfg.Hkv)
        c, cc = self.cfg.c(), self.c()
        lib().fo_decode_heads(C.byref(c), C.byref(cc), _p(q), _p(out), C.c_int(h0), C.c_int(h1))
        return out


def dim_mse(cfg: OracleConfig, X: np.ndarray, b: int, h: int) -> np.ndarray:
    """Sec. 3.4: per-dimension mean squared reconstruction error over the middle."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    mse = np.zeros(cfg.d, dtype=np.float64)
    c = cfg.c()
    lib().fo_dim_mse(C.byref(c), _p(X), C.c_int32(X.shape[1]), C.c_int(b), C.c_int(h), _p(mse))
    return mse


def select_dims(mse: np.ndarray, n_full: int):
    """Sec. 3.4: (idx_full, idx_comp), ascending; the best-reconstructed dims are compressed."""
    mse = np.ascontiguousarray(mse, dtype=np.float64)
    d = mse.shape[0]
    idx_full = np.zeros(n_full, dtype=np.int32)
    idx_comp = np.zeros(d - n_full, dtype=np.int32)
    lib().fo_select_dims(_p(mse), C.c_int(d), C.c_int(n_full), _p(idx_full), _p(idx_comp))
    return idx_full, idx_comp
