"""ctypes front end of the fp64 CPU oracle (oracle/hass_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg. The CUDA library and its Python binding never import
this package, and this package imports nothing from them.

The C file is compiled with gcc on first use (or by ``build()``) into
``oracle/_build/libhass_oracle.so``; target_clones in the C source pick the SIMD
width at load time, so the same binary runs on hosts with or without AVX-512.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hass_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB = os.path.join(_OUT_DIR, "libhass_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_i64, c_i32, c_dbl, c_vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p
        lib.hass_oracle_threads.restype = ctypes.c_int
        lib.hass_oracle_row_from_logits.restype = ctypes.c_int
        lib.hass_oracle_row_from_logits.argtypes = [c_vp, c_vp, c_i64, c_i32, c_dbl, c_vp,
                                                    c_vp, c_vp, c_vp, c_vp, c_vp, c_vp]
        lib.hass_oracle_features.restype = ctypes.c_int
        lib.hass_oracle_features.argtypes = [c_vp, c_vp, c_vp, ctypes.c_int, c_i64, c_i64, c_i64, c_i32,
                                             c_vp, c_vp, c_i64, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp]
        lib.hass_oracle_row_objective.restype = ctypes.c_int
        lib.hass_oracle_row_objective.argtypes = [c_vp, c_vp, c_i64, c_i32, c_dbl, c_dbl, c_dbl, c_vp,
                                                  c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp]
        lib.hass_oracle_features_objective.restype = ctypes.c_int
        lib.hass_oracle_features_objective.argtypes = [c_vp, c_vp, c_vp, ctypes.c_int, c_i64, c_i64, c_i64, c_i32,
                                                       c_dbl, c_dbl, c_vp, c_vp, c_i64, c_vp, c_vp, c_vp, c_vp,
                                                       c_vp, c_vp, c_vp, c_vp]
        lib.hass_oracle_row_variant.restype = ctypes.c_int
        lib.hass_oracle_row_variant.argtypes = [c_vp, c_vp, c_i64, c_i32, c_dbl, ctypes.c_int, c_dbl, c_vp, c_vp, c_vp,
                                                c_vp, c_vp, c_vp, c_vp]
        lib.hass_oracle_features_variant.restype = ctypes.c_int
        lib.hass_oracle_features_variant.argtypes = [c_vp, c_vp, c_vp, c_i64, c_i64, c_i64, c_i32, ctypes.c_int, c_dbl,
                                                     c_vp, c_vp, c_i64, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp]
        lib.hass_oracle_row_on_set.restype = ctypes.c_int
        lib.hass_oracle_row_on_set.argtypes = [c_vp, c_vp, c_i64, c_vp, c_i32, c_dbl, ctypes.c_int, c_vp, c_vp, c_vp,
                                               c_vp, c_vp]
        lib.hass_oracle_logits_at.restype = ctypes.c_int
        lib.hass_oracle_logits_at.argtypes = [c_vp, c_vp, c_i64, c_i64, c_i64, c_vp, c_vp, c_i64, c_vp]
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().hass_oracle_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def from_logits(z_t, z_d, K: int, g: float = 1.0, forced_idx=None, want_dz: bool = True) -> dict:
    """Steps 2-5 (softmax statistics, Omega_hat, Eq. 1, dL/dz_d) for ONE row of logits."""
    z_t = np.ascontiguousarray(z_t, dtype=np.float64)
    z_d = np.ascontiguousarray(z_d, dtype=np.float64)
    assert z_t.ndim == 1 and z_t.shape == z_d.shape
    V = z_t.shape[0]
    loss = np.zeros(1)
    lse_t = np.zeros(1)
    lse_d = np.zeros(1)
    idx = np.zeros(K, dtype=np.int32)
    q_k = np.zeros(K)
    dz = np.zeros(V) if want_dz else None
    f = None if forced_idx is None else np.ascontiguousarray(forced_idx, dtype=np.int32)
    rc = _load().hass_oracle_row_from_logits(_ptr(z_t), _ptr(z_d), V, K, float(g), _ptr(f), _ptr(loss),
                                             _ptr(idx), _ptr(q_k), _ptr(lse_t), _ptr(lse_d), _ptr(dz))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return dict(loss=float(loss[0]), idx=idx, q_k=q_k, lse_t=float(lse_t[0]), lse_d=float(lse_d[0]), dz_d=dz)


VARIANT_TOPK, VARIANT_TOP_P, VARIANT_NORMED, VARIANT_BIDIR = 0, 1, 2, 3


def variant_from_logits(z_t, z_d, K: int, variant: int, param: float = 0.0, g: float = 1.0) -> dict:
    """One row of logits under a loss variant of Section 4.3 (Top-P, Normed Top-K) or Eq. 1."""
    z_t = np.ascontiguousarray(z_t, dtype=np.float64)
    z_d = np.ascontiguousarray(z_d, dtype=np.float64)
    V = z_t.shape[0]
    loss, lse_t, lse_d = np.zeros(1), np.zeros(1), np.zeros(1)
    kk = 2 * K if variant == VARIANT_BIDIR else K
    idx = np.zeros(kk, dtype=np.int32)
    q_k = np.zeros(kk)
    n = np.zeros(1, dtype=np.int32)
    dz = np.zeros(V)
    rc = _load().hass_oracle_row_variant(_ptr(z_t), _ptr(z_d), V, K, float(g), int(variant), float(param), _ptr(loss),
                                         _ptr(idx), _ptr(q_k), _ptr(n), _ptr(lse_t), _ptr(lse_d), _ptr(dz))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return dict(loss=float(loss[0]), idx=idx, q_k=q_k, n=int(n[0]), lse_t=float(lse_t[0]), lse_d=float(lse_d[0]),
                dz_d=dz)


def on_set_from_logits(z_t, z_d, tokens, g: float = 1.0, normed: bool = False) -> dict:
    """Eq. 1 (or, with ``normed``, the Normed Top-K loss) of ONE row of logits on a given set of token ids."""
    z_t = np.ascontiguousarray(z_t, dtype=np.float64)
    z_d = np.ascontiguousarray(z_d, dtype=np.float64)
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    V, n = z_t.shape[0], tok.shape[0]
    loss, lse_t, lse_d = np.zeros(1), np.zeros(1), np.zeros(1)
    q = np.zeros(n)
    dz = np.zeros(V)
    rc = _load().hass_oracle_row_on_set(_ptr(z_t), _ptr(z_d), V, _ptr(tok), n, float(g), int(bool(normed)),
                                        _ptr(loss), _ptr(q), _ptr(lse_t), _ptr(lse_d), _ptr(dz))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return dict(loss=float(loss[0]), q_k=q, lse_t=float(lse_t[0]), lse_d=float(lse_d[0]), dz_d=dz)


def variant_from_features(H_t, H_d, W, K: int, variant: int, param: float = 0.0, rows=None, grad_loss=None,
                          forced_idx=None) -> dict:
    """Feature-level loss variants on bf16 bit patterns; outputs indexed by position in ``rows``.
    ``forced_idx`` [len(rows), K] (2K for the bi-directional variant): score each row on these token ids
    (entries < 0 are padding) instead of on the oracle's own selection."""
    H_t, H_d, W = np.ascontiguousarray(H_t), np.ascontiguousarray(H_d), np.ascontiguousarray(W)
    assert H_t.dtype == H_d.dtype == W.dtype == np.uint16
    N, d = H_t.shape
    V = W.shape[0]
    rows_a = np.arange(N, dtype=np.int64) if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = rows_a.shape[0]
    gl = None if grad_loss is None else np.ascontiguousarray(grad_loss, dtype=np.float64)
    loss, lse_t, lse_d = np.zeros(n), np.zeros(n), np.zeros(n)
    kk = 2 * K if variant == VARIANT_BIDIR else K
    idx = np.zeros((n, kk), dtype=np.int32)
    q_k = np.zeros((n, kk))
    cnt = np.zeros(n, dtype=np.int32)
    dH = np.zeros((n, d))
    f = None
    if forced_idx is not None:
        f = np.ascontiguousarray(forced_idx, dtype=np.int32)
        assert f.shape == (n, kk)
    rc = _load().hass_oracle_features_variant(_ptr(H_t), _ptr(H_d), _ptr(W), N, d, V, K, int(variant), float(param),
                                              _ptr(gl), _ptr(rows_a), n, _ptr(f), _ptr(loss), _ptr(idx), _ptr(q_k),
                                              _ptr(cnt), _ptr(lse_t), _ptr(lse_d), _ptr(dH))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return dict(loss=loss, idx=idx, q_k=q_k, n=cnt, lse_t=lse_t, lse_d=lse_d, dH_d=dH)


def objective_from_logits(z_t, z_d, K: int, w_ce: float, w_topk: float, g: float = 1.0) -> dict:
    """One row of logits: cross-entropy over the whole vocabulary, Top-K loss, and the derivative of
    w_ce * L_CE + w_topk * L_TopK with respect to the draft logits."""
    z_t = np.ascontiguousarray(z_t, dtype=np.float64)
    z_d = np.ascontiguousarray(z_d, dtype=np.float64)
    V = z_t.shape[0]
    loss, ce, lse_t, lse_d = np.zeros(1), np.zeros(1), np.zeros(1), np.zeros(1)
    idx = np.zeros(K, dtype=np.int32)
    q_k = np.zeros(K)
    dz = np.zeros(V)
    rc = _load().hass_oracle_row_objective(_ptr(z_t), _ptr(z_d), V, K, float(g), float(w_ce), float(w_topk), None,
                                           _ptr(ce), _ptr(loss), _ptr(idx), _ptr(q_k), _ptr(lse_t), _ptr(lse_d),
                                           _ptr(dz))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return dict(loss_ce=float(ce[0]), loss=float(loss[0]), idx=idx, q_k=q_k, lse_t=float(lse_t[0]),
                lse_d=float(lse_d[0]), dz_d=dz)


def objective_from_features(H_t, H_d, W, K: int, w_ce: float, w_topk: float, rows=None, grad_loss=None,
                            forced_idx=None, want_dH: bool = True) -> dict:
    """from_features for the objective w_ce * L_CE + w_topk * L_TopK; also returns loss_ce."""
    return _features(H_t, H_d, W, K, rows, grad_loss, forced_idx, want_dH, float(w_ce), float(w_topk), True)


def from_features(H_t, H_d, W, K: int, rows=None, grad_loss=None, forced_idx=None,
                  want_dH: bool = True) -> dict:
    """Steps 1-5 on feature rows.

    H_t, H_d [N, d] and W [V, d] are either uint16 arrays of bf16 bit patterns (the inputs
    the GPU receives) or float64 arrays (used by the finite-difference pin).
    ``rows`` selects a subset; outputs are indexed by position in ``rows``.
    """
    return _features(H_t, H_d, W, K, rows, grad_loss, forced_idx, want_dH, 0.0, 1.0, False)


def _features(H_t, H_d, W, K, rows, grad_loss, forced_idx, want_dH, w_ce, w_topk, want_ce) -> dict:
    H_t = np.ascontiguousarray(H_t)
    H_d = np.ascontiguousarray(H_d)
    W = np.ascontiguousarray(W)
    assert H_t.dtype == H_d.dtype == W.dtype and H_t.dtype in (np.uint16, np.float64)
    N, d = H_t.shape
    V = W.shape[0]
    assert H_d.shape == (N, d) and W.shape == (V, d)
    if rows is None:
        rows_a, n = None, N
    else:
        rows_a = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows_a.shape[0]
    gl = None if grad_loss is None else np.ascontiguousarray(grad_loss, dtype=np.float64)
    assert gl is None or gl.shape == (N,)
    f = None
    if forced_idx is not None:
        f = np.ascontiguousarray(forced_idx, dtype=np.int32)
        assert f.shape == (n, K)
    loss = np.zeros(n)
    lse_t = np.zeros(n)
    lse_d = np.zeros(n)
    idx = np.zeros((n, K), dtype=np.int32)
    q_k = np.zeros((n, K))
    dH = np.zeros((n, d)) if want_dH else None
    ce = np.zeros(n) if want_ce else None
    rc = _load().hass_oracle_features_objective(_ptr(H_t), _ptr(H_d), _ptr(W), H_t.dtype.itemsize, N, d, V, K,
                                                w_ce, w_topk, _ptr(gl), _ptr(rows_a), n, _ptr(f), _ptr(ce),
                                                _ptr(loss), _ptr(idx), _ptr(q_k), _ptr(lse_t), _ptr(lse_d), _ptr(dH))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    out = dict(loss=loss, idx=idx, q_k=q_k, lse_t=lse_t, lse_d=lse_d, dH_d=dH)
    if want_ce:
        out["loss_ce"] = ce
    return out


def logits_at(H, W, row, tok) -> np.ndarray:
    """z[j] = <H[row_j], W[tok_j]> in fp64 from bf16 bit patterns (step 1 at chosen entries)."""
    H = np.ascontiguousarray(H)
    W = np.ascontiguousarray(W)
    assert H.dtype == np.uint16 and W.dtype == np.uint16
    row = np.ascontiguousarray(row, dtype=np.int64).ravel()
    tok = np.ascontiguousarray(tok, dtype=np.int32).ravel()
    assert row.shape == tok.shape
    z = np.zeros(row.shape[0])
    rc = _load().hass_oracle_logits_at(_ptr(H), _ptr(W), H.shape[0], H.shape[1], W.shape[0], _ptr(row),
                                       _ptr(tok), row.shape[0], _ptr(z))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return z
