"""ctypes front end of the fp64 CPU oracle -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's cpu_baseline / reference leg
may import this module; the product path never does.  It compiles
``attn_jvp_oracle.c`` (plain C, gcc, OpenMP) on first use and exposes

* ``attn_jvp_def``   the definition of Appendix C.1 written out row by row,
* ``attn_jvp_fold``  the definition on key blocks of size ``Bc``, folded block by block with the
  chunk-merge identity (the streaming property: any block size gives the same result),
* ``attn_jvp_def_bf16_rows``  the definition on bf16 [B][L][H][D] inputs for
  a chosen set of query rows (what the GPU parity tests compare against).

All arithmetic is fp64.  The softmax scale ``s`` (absent from the paper's
S = Q K^T) multiplies S and tS; LSE is the natural log; ``mu`` is the row sum
of P.tS (equal to the derivative of LSE along the tangent).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_jvp_oracle.c")
_SO = os.path.join(_HERE, "libattn_jvp_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source; returns the library path."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            dp = ctypes.POINTER(ctypes.c_double)
            u16p = ctypes.POINTER(ctypes.c_uint16)
            i64p = ctypes.POINTER(ctypes.c_int64)
            lg = ctypes.c_long
            lib.attn_jvp_def_f64.argtypes = [dp] * 6 + [lg, lg, lg, ctypes.c_double] + [dp] * 4
            lib.attn_jvp_def_f64.restype = ctypes.c_int
            lib.attn_jvp_fold_f64.argtypes = [dp] * 6 + [lg, lg, lg, lg, ctypes.c_double] + [dp] * 4
            lib.attn_jvp_fold_f64.restype = ctypes.c_int
            lib.attn_jvp_def_bf16_blhd_rows.argtypes = (
                [u16p] * 6 + [lg] * 5 + [ctypes.c_double, i64p, lg] + [dp] * 4
            )
            lib.attn_jvp_def_bf16_blhd_rows.restype = ctypes.c_int
            lib.attn_jvp_oracle_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().attn_jvp_oracle_threads())


def _f64(x, shape=None):
    if x is None:
        return None
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _dptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _run_f64(fn_name, Q, K, V, tQ, tK, tV, scale, Bc=None):
    lib = _load()
    Q = _f64(Q)
    Lq, D = Q.shape
    K = _f64(K)
    Lk = K.shape[0]
    V, tQ = _f64(V, (Lk, D)), _f64(tQ, (Lq, D))
    tK, tV = _f64(tK, (Lk, D)), _f64(tV, (Lk, D))
    if K.shape != (Lk, D):
        raise ValueError("K must be [Lk][D]")
    O = np.empty((Lq, D)); tO = np.empty((Lq, D)); LSE = np.empty(Lq); MU = np.empty(Lq)
    args = [_dptr(Q), _dptr(K), _dptr(V), _dptr(tQ), _dptr(tK), _dptr(tV), Lq, Lk, D]
    if Bc is not None:
        args.append(int(Bc))
    args += [float(scale), _dptr(O), _dptr(tO), _dptr(LSE), _dptr(MU)]
    rc = getattr(lib, fn_name)(*args)
    if rc != 0:
        raise RuntimeError(f"{fn_name} failed with code {rc}")
    return O, tO, LSE, MU


def attn_jvp_def(Q, K, V, tQ, tK, tV, scale):
    """Definition route (Appendix C.1 equations).  2-D fp64 arrays, one head.

    ``tK`` / ``tV`` may be None (zero tangent).  Returns (O, tO, LSE, mu).
    """
    return _run_f64("attn_jvp_def_f64", Q, K, V, tQ, tK, tV, scale)


def attn_jvp_fold(Q, K, V, tQ, tK, tV, scale, Bc):
    """Block-fold route: the definition on consecutive key blocks of ``Bc``, merged one after the other.
    Returns (O, tO, LSE, mu)."""
    return _run_f64("attn_jvp_fold_f64", Q, K, V, tQ, tK, tV, scale, Bc=Bc)


def attn_jvp_def_bf16_rows(q, k, v, tq, tk, tv, B, H, Lq, Lk, D, scale, rows):
    """Definition route on bf16 bit patterns in [B][L][H][D] layout.

    ``q`` .. ``tv`` are uint16 numpy arrays holding bf16 bit patterns
    (``tk`` / ``tv`` may be None).  ``rows`` lists flat query-row indices
    ``(b*H + h)*Lq + i``; they are sorted internally and results are returned
    in the caller's order.  Returns (O, tO, LSE, mu) as fp64 arrays of shape
    [n][D], [n][D], [n], [n].
    """
    lib = _load()
    rows = np.asarray(rows, dtype=np.int64).reshape(-1)
    order = np.argsort(rows, kind="stable")
    srows = np.ascontiguousarray(rows[order])
    n = srows.size

    def u16(a, L):
        if a is None:
            return None, None
        a = np.ascontiguousarray(a)
        if a.dtype != np.uint16 or a.size != B * L * H * D:
            raise ValueError("bf16 tensors are passed as uint16 arrays of B*L*H*D elements")
        return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))

    keep = []
    ptrs = []
    for a, L in ((q, Lq), (k, Lk), (v, Lk), (tq, Lq), (tk, Lk), (tv, Lk)):
        arr, p = u16(a, L)
        keep.append(arr)
        ptrs.append(p)
    O = np.empty((n, D)); tO = np.empty((n, D)); LSE = np.empty(n); MU = np.empty(n)
    rc = lib.attn_jvp_def_bf16_blhd_rows(
        *ptrs, B, H, Lq, Lk, D, float(scale),
        srows.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), n,
        _dptr(O), _dptr(tO), _dptr(LSE), _dptr(MU))
    if rc != 0:
        raise RuntimeError(f"attn_jvp_def_bf16_blhd_rows failed with code {rc}")
    inv = np.empty_like(order)
    inv[order] = np.arange(n)
    return O[inv], tO[inv], LSE[inv], MU[inv]


def splitkv_merge(O_c, tO_c, LSE_c, MU_c):
    """Merges per-chunk results of a split over the keys (fp64 numpy; test infrastructure).

    Chunk c gave (O_c, tO_c, LSE_c, mu_c), each normalised within the chunk.  The full softmax weights are
    P_j = w_c P^c_j with w_c = exp(LSE_c - LSE), LSE = log sum_c exp(LSE_c), so from the aggregated form of
    Appendix C.1 (tO = (P.tS) V + P tV - diag(mu) O):
        O = sum_c w_c O_c,  mu = sum_c w_c mu_c,  tO = sum_c w_c (tO_c + mu_c O_c) - mu O.
    Inputs are lists over chunks of arrays [n][D], [n][D], [n], [n].  Returns (O, tO, LSE, mu).
    """
    L = np.stack(LSE_c)                      # [C][n]
    m = L.max(axis=0)
    LSE = m + np.log(np.exp(L - m).sum(axis=0))
    w = np.exp(L - LSE)                      # [C][n]
    O = sum(w[c][:, None] * O_c[c] for c in range(len(O_c)))
    mu = sum(w[c] * MU_c[c] for c in range(len(O_c)))
    tO = sum(w[c][:, None] * (tO_c[c] + MU_c[c][:, None] * O_c[c]) for c in range(len(O_c))) - mu[:, None] * O
    return O, tO, LSE, mu


def rmsnorm_jvp(x, tx, w, eps):
    """RMS normalisation over the last axis and its tangent (fp64).  x, tx: [rows][D]; w: [D].  Returns (y, ty)."""
    lib = _load()
    if not hasattr(lib, "_rms_ready"):
        dp = ctypes.POINTER(ctypes.c_double)
        lib.rmsnorm_jvp_f64.argtypes = [dp, dp, dp, ctypes.c_long, ctypes.c_long, ctypes.c_double, dp, dp]
        lib.rmsnorm_jvp_f64.restype = ctypes.c_int
        lib._rms_ready = True
    x = _f64(x)
    rows, D = x.shape
    tx = _f64(tx, (rows, D))
    w = _f64(w, (D,))
    y = np.empty((rows, D))
    ty = None if tx is None else np.empty((rows, D))
    rc = lib.rmsnorm_jvp_f64(_dptr(x), _dptr(tx), _dptr(w), rows, D, float(eps), _dptr(y), _dptr(ty))
    if rc != 0:
        raise RuntimeError(f"rmsnorm_jvp_f64 failed with code {rc}")
    return y, ty
