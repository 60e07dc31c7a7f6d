"""ctypes binding of the C oracle (test infrastructure only; see l2a_oracle.c for what it computes).

Tensors are numpy arrays: bf16 data as uint16 bit patterns, contiguous [B, L, H, D].
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "l2a_oracle.c")
_LIBS = {False: os.path.join(_HERE, "libl2a_oracle.so"), True: os.path.join(_HERE, "libl2a_oracle_f64in.so")}
_loaded = {}
_F64_INPUTS = False  # module-level switch used by the finite-difference pin (see f64_inputs())


class _CShape(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("Lq", ctypes.c_int32), ("Lk", ctypes.c_int32),
        ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("window", ctypes.c_int32), ("q_pos_offset", ctypes.c_int32),
        ("scale", ctypes.c_double),
    ]


@dataclass
class Shape:
    B: int
    Lq: int
    Lk: int
    Hq: int
    Hkv: int
    D: int
    window: int
    q_pos_offset: int | None = None
    scale: float | None = None

    def c(self) -> _CShape:
        off = self.Lk - self.Lq if self.q_pos_offset is None else self.q_pos_offset
        sc = 1.0 / float(np.sqrt(self.D)) if self.scale is None else self.scale
        return _CShape(self.B, self.Lq, self.Lk, self.Hq, self.Hkv, self.D, self.window, off, sc)


def build(force: bool = False, f64_inputs: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) next to its source; returns the library path.

    ``f64_inputs`` builds the variant whose Q/K/V/dO are fp64 instead of bf16 bit patterns."""
    lib = _LIBS[f64_inputs]
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(_SRC):
        tmp = lib + f".{os.getpid()}.tmp"
        flags = ["-DL2A_ORACLE_F64_INPUT"] if f64_inputs else []
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", *flags, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, lib)
    return lib


class f64_inputs:
    """Context manager: inside it every call takes fp64 Q/K/V/dO (same C code, other input type)."""

    def __enter__(self):
        global _F64_INPUTS
        self._old, _F64_INPUTS = _F64_INPUTS, True

    def __exit__(self, *exc):
        global _F64_INPUTS
        _F64_INPUTS = self._old


def _load():
    key = _F64_INPUTS
    if key not in _loaded:
        lib = ctypes.CDLL(build(f64_inputs=key))
        lib.l2a_oracle_num_threads.restype = ctypes.c_int
        _loaded[key] = lib
    return _loaded[key]


def num_threads() -> int:
    return int(_load().l2a_oracle_num_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    """Input tensor: uint16 bf16 bit patterns, or fp64 inside ``f64_inputs()``."""
    a = np.ascontiguousarray(a)
    want = np.float64 if _F64_INPUTS else np.uint16
    assert a.dtype == want, (a.dtype, want)
    return a


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def route(z: np.ndarray, thr: float = 0.0) -> np.ndarray:
    z = np.ascontiguousarray(z, dtype=np.float32)
    d = np.empty(z.shape, dtype=np.uint8)
    _load().l2a_oracle_route(_p(z), ctypes.c_int64(z.size), ctypes.c_float(thr), _p(d))
    return d


def compact(d: np.ndarray):
    """d uint8 [B, L] -> (q_idx int32 [B, L] tail -1, n_routed int32 [B], prefix int32 [B, L+1])."""
    d = np.ascontiguousarray(d, dtype=np.uint8)
    B, L = d.shape
    q_idx = np.empty((B, L), np.int32)
    n = np.empty((B,), np.int32)
    prefix = np.empty((B, L + 1), np.int32)
    _load().l2a_oracle_compact(_p(d), ctypes.c_int32(B), ctypes.c_int32(L), _p(q_idx), _p(n), _p(prefix))
    return q_idx, n, prefix


def forward_rows(sh: Shape, Q, K, V, d, rb, rh, rt):
    """Rows (b, h, t) -> dict of fp64 arrays s, a, o [n, D] and lse_loc, lse_glb [n]."""
    Q, K, V = _u16(Q), _u16(K), _u16(V)
    d = np.ascontiguousarray(d, dtype=np.uint8)
    rb, rh, rt = _i32(rb), _i32(rh), _i32(rt)
    n = rb.size
    out = {k: np.empty((n, sh.D), np.float64) for k in ("s", "a", "o")}
    out["lse_loc"] = np.empty((n,), np.float64)
    out["lse_glb"] = np.empty((n,), np.float64)
    cs = sh.c()
    _load().l2a_oracle_forward_rows(ctypes.byref(cs), _p(Q), _p(K), _p(V), _p(d), ctypes.c_int64(n),
                                    _p(rb), _p(rh), _p(rt), _p(out["s"]), _p(out["a"]), _p(out["o"]),
                                    _p(out["lse_loc"]), _p(out["lse_glb"]))
    return out


def forward_full(sh: Shape, Q, K, V, d):
    """All rows; outputs shaped [B, Lq, Hq, D] (s, a, o) and [B, Hq, Lq] (lse)."""
    b, t, h = np.meshgrid(np.arange(sh.B), np.arange(sh.Lq), np.arange(sh.Hq), indexing="ij")
    r = forward_rows(sh, Q, K, V, d, b.ravel(), h.ravel(), t.ravel())
    out = {k: r[k].reshape(sh.B, sh.Lq, sh.Hq, sh.D) for k in ("s", "a", "o")}
    for k in ("lse_loc", "lse_glb"):
        out[k] = np.ascontiguousarray(r[k].reshape(sh.B, sh.Lq, sh.Hq).transpose(0, 2, 1))
    return out


def backward_full(sh: Shape, Q, K, V, d, dO):
    Q, K, V, dO = _u16(Q), _u16(K), _u16(V), _u16(dO)
    d = np.ascontiguousarray(d, dtype=np.uint8)
    dQ = np.empty((sh.B, sh.Lq, sh.Hq, sh.D), np.float64)
    dK = np.empty((sh.B, sh.Lk, sh.Hkv, sh.D), np.float64)
    dV = np.empty((sh.B, sh.Lk, sh.Hkv, sh.D), np.float64)
    cs = sh.c()
    _load().l2a_oracle_backward_full(ctypes.byref(cs), _p(Q), _p(K), _p(V), _p(d), _p(dO), _p(dQ), _p(dK), _p(dV))
    return dQ, dK, dV


def dq_rows(sh: Shape, Q, K, V, d, dO, rb, rh, rt):
    Q, K, V, dO = _u16(Q), _u16(K), _u16(V), _u16(dO)
    d = np.ascontiguousarray(d, dtype=np.uint8)
    rb, rh, rt = _i32(rb), _i32(rh), _i32(rt)
    out = np.empty((rb.size, sh.D), np.float64)
    cs = sh.c()
    _load().l2a_oracle_dq_rows(ctypes.byref(cs), _p(Q), _p(K), _p(V), _p(d), _p(dO), ctypes.c_int64(rb.size),
                               _p(rb), _p(rh), _p(rt), _p(out))
    return out


def dkv_cols(sh: Shape, Q, K, V, d, dO, b: int, g: int, js):
    Q, K, V, dO = _u16(Q), _u16(K), _u16(V), _u16(dO)
    d = np.ascontiguousarray(d, dtype=np.uint8)
    js = _i32(js)
    dk = np.empty((js.size, sh.D), np.float64)
    dv = np.empty((js.size, sh.D), np.float64)
    cs = sh.c()
    _load().l2a_oracle_dkv_cols(ctypes.byref(cs), _p(Q), _p(K), _p(V), _p(d), _p(dO), ctypes.c_int32(b),
                                ctypes.c_int32(g), ctypes.c_int32(js.size), _p(js), _p(dk), _p(dv))
    return dk, dv


def dgate_rows(sh: Shape, Q, K, V, dO, rb, rt):
    Q, K, V, dO = _u16(Q), _u16(K), _u16(V), _u16(dO)
    rb, rt = _i32(rb), _i32(rt)
    out = np.empty((rb.size,), np.float64)
    cs = sh.c()
    _load().l2a_oracle_dgate_rows(ctypes.byref(cs), _p(Q), _p(K), _p(V), _p(dO), ctypes.c_int64(rb.size),
                                  _p(rb), _p(rt), _p(out))
    return out


def router_logits(S, w, bias: float = 0.0):
    """Eq. 3 before the sigmoid: z_t = W s_t + bias with s_t the Hq*D local-output values of token t.
    S: bf16 bit patterns (uint16) [B, L, Hq, D]; w: [Hq*D].  Plain fp64 dot products."""
    S = np.ascontiguousarray(S)
    s64 = (S.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    B, L = S.shape[0], S.shape[1]
    return s64.reshape(B, L, -1) @ np.asarray(w, np.float64) + float(bias)


def router_backward(S, w, z, dgate, reg_coeff: float, dO=None):
    """Backward of the router under the straight-through estimator (Section 3.3).

    The decision d_t is replaced by its relaxation d_hat_t = sigmoid(z_t) in the backward pass, so (Eq. 7)
        dL/dd_hat_t = dgate_t + 2 * reg_coeff * d_hat_t,       dgate_t = (dL_NTP/do_t) . a_t,  reg_coeff = lambda / (n L),
        dL/dz_t     = dL/dd_hat_t * d_hat_t * (1 - d_hat_t)    (derivative of the sigmoid),
        dL/dW       = sum over tokens of dL/dz_t * s_t,        dL/dbias = sum over tokens of dL/dz_t,
        dL/ds_t    += dL/dz_t * W                              (on top of dL/do_t, since o_t = s_t + d_t a_t).
    S, dO: bf16 bit patterns (uint16) [B, L, Hq, D]; w: [Hq*D]; z, dgate: [B, L].  Returns fp64
    dz [B, L], dw [Hq*D], dbias (scalar), dS [B, L, Hq, D] (= dO + dz * W; None when dO is None)."""
    S = np.ascontiguousarray(S)
    s64 = (S.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    B, L = S.shape[0], S.shape[1]
    s64 = s64.reshape(B, L, -1)
    w = np.asarray(w, np.float64)
    d_hat = 1.0 / (1.0 + np.exp(-np.asarray(z, np.float64)))
    dd_hat = np.asarray(dgate, np.float64) + 2.0 * float(reg_coeff) * d_hat
    dz = dd_hat * d_hat * (1.0 - d_hat)
    dw = np.einsum("bt,btk->k", dz, s64)
    dbias = dz.sum()
    dS = None
    if dO is not None:
        dO = np.ascontiguousarray(dO)
        do64 = (dO.astype(np.uint32) << 16).view(np.float32).astype(np.float64).reshape(B, L, -1)
        dS = (do64 + dz[:, :, None] * w[None, None, :]).reshape(S.shape)
    return dz, dw, dbias, dS


def gate_regulariser_sum(z):
    """Sum over tokens of sigmoid(z_t)^2 per batch entry (Eq. 6 without its lambda / (n L) factor)."""
    g = 1.0 / (1.0 + np.exp(-np.asarray(z, np.float64)))
    return (g * g).sum(axis=1)
