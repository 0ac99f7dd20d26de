"""ctypes front end of the CPU oracle (oracle/vitint_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.

Codes travel as unpacked int16 numpy arrays; every function returns fresh arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "vitint_oracle.cpp"
_LIB = _HERE / "libvitint_oracle.so"
_lib = None

SOFTMAX_ULP_BAND = 2               # fp32 softmax probabilities may differ by this many ulp (the path's stated bound)


def build(force: bool = False) -> Path:
    """Compile the oracle with contraction off so every fp32 op sequence is literal."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-ffp-contract=off", "-fno-fast-math",
               str(_SRC), "-o", str(_LIB)]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.vo_overflow_bound.restype = ctypes.c_int64
        _lib.vo_get_threads.restype = ctypes.c_int
    return _lib


def set_threads(n: int) -> None:
    lib().vo_set_threads(ctypes.c_int(n))


def get_threads() -> int:
    return int(lib().vo_get_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _i16(a):
    return np.ascontiguousarray(a, dtype=np.int16)


I64 = ctypes.c_int64
I32 = ctypes.c_int
F32 = ctypes.c_float


def code_range(bits: int, signed: bool):
    return (-(1 << (bits - 1)), (1 << (bits - 1)) - 1) if signed else (0, (1 << bits) - 1)


def container_bits(bits: int) -> int:
    return 4 if bits == 3 else bits


def packed_pitch(cols: int, bits: int) -> int:
    """Smallest pitch (bytes) that holds `cols` codes and is a multiple of 16."""
    nbytes = (cols * container_bits(bits) + 7) // 8
    return (nbytes + 15) // 16 * 16


# ---- a1 -------------------------------------------------------------------

def quantize(x, step, bits: int, signed: bool, row_steps=None) -> np.ndarray:
    x = _f32(x)
    rows, cols = x.shape
    rs = _f32(row_steps)
    q = np.empty((rows, cols), dtype=np.int16)
    lib().vo_quantize(_p(x), I64(rows), I64(cols), I64(cols), F32(float(step)), _p(rs), I32(bits), I32(int(signed)),
                      _p(q), I64(cols))
    return q


def pack(q, bits: int, pitch: int | None = None) -> np.ndarray:
    q = _i16(q)
    rows, cols = q.shape
    pitch = packed_pitch(cols, bits) if pitch is None else pitch
    out = np.empty((rows, pitch), dtype=np.uint8)
    lib().vo_pack(_p(q), I64(rows), I64(cols), I64(cols), I32(bits), _p(out), I64(pitch))
    return out


def unpack(packed, cols: int, bits: int, signed: bool) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    rows, pitch = packed.shape
    q = np.empty((rows, cols), dtype=np.int16)
    lib().vo_unpack(_p(packed), I64(rows), I64(cols), I64(pitch), I32(bits), I32(int(signed)), _p(q), I64(cols))
    return q


# ---- a2 / a3 ----------------------------------------------------------------

def matmul_i32(a, b) -> np.ndarray:
    a, b = _i16(a), _i16(b)
    M, K = a.shape
    N, K2 = b.shape
    assert K == K2
    acc = np.empty((M, N), dtype=np.int32)
    lib().vo_matmul_i32(_p(a), I64(K), _p(b), I64(K), I64(M), I64(N), I64(K), _p(acc), I64(N))
    return acc


def matmul_i64(a, b) -> np.ndarray:
    a, b = _i16(a), _i16(b)
    M, K = a.shape
    N, _ = b.shape
    acc = np.empty((M, N), dtype=np.int64)
    lib().vo_matmul_i64(_p(a), I64(K), _p(b), I64(K), I64(M), I64(N), I64(K), _p(acc), I64(N))
    return acc


def overflow_bound(K: int, bits_x: int, signed_x: bool, bits_w: int, signed_w: bool) -> int:
    return int(lib().vo_overflow_bound(I64(K), I32(bits_x), I32(int(signed_x)), I32(bits_w), I32(int(signed_w))))


def epilogue_dequant(acc, s_x, s_w, bias=None, residual=None, act: int = 0) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    M, N = acc.shape
    s_w, bias, residual = _f32(s_w), _f32(bias), _f32(residual)
    y = np.empty((M, N), dtype=np.float32)
    lib().vo_epilogue_dequant(_p(acc), I64(M), I64(N), I64(N), F32(float(s_x)), _p(s_w), _p(bias), _p(residual),
                              I64(N), I32(act), _p(y), I64(N))
    return y


def epilogue_requant(acc, alpha, beta, bits: int, signed: bool) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    M, N = acc.shape
    alpha, beta = _f32(alpha), _f32(beta)
    q = np.empty((M, N), dtype=np.int16)
    lib().vo_epilogue_requant(_p(acc), I64(M), I64(N), I64(N), _p(alpha), _p(beta), I32(bits), I32(int(signed)),
                              _p(q), I64(N))
    return q


def epilogue_gelu_requant(acc, s_x, s_w, bias, inv_s, bits: int, signed: bool = False, tol_rel: float = 0.0):
    """Returns (codes, lowest, highest): the codes of GELU(y) by the erf definition (fp64, rounded once), and the
    codes reached when that value moves by -/+ tol_rel*|y|.  The tolerance belongs to whoever checks an fp32
    implementation against this and is passed in; with the default 0 the three arrays are equal."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    M, N = acc.shape
    s_w, bias, inv_s = _f32(s_w), _f32(bias), _f32(inv_s)
    q = np.empty((M, N), dtype=np.int16)
    lo = np.empty_like(q)
    hi = np.empty_like(q)
    lib().vo_epilogue_gelu_requant(_p(acc), I64(M), I64(N), I64(N), F32(float(s_x)), _p(s_w), _p(bias), _p(inv_s),
                                   I32(bits), I32(int(signed)), F32(tol_rel), _p(q), _p(lo), _p(hi), I64(N))
    return q, lo, hi


# ---- a4 / a5 / a6 -------------------------------------------------------------

def qk(q_slabs, k_slabs) -> np.ndarray:
    """q_slabs, k_slabs: [n_problems, T, d] codes -> S [n_problems, T, T] int32."""
    q_slabs, k_slabs = _i16(q_slabs), _i16(k_slabs)
    n, T, d = q_slabs.shape
    S = np.empty((n, T, T), dtype=np.int32)
    lib().vo_qk(_p(q_slabs), I64(d), I64(T * d), _p(k_slabs), I64(d), I64(T * d), I64(n), I64(T), I64(d), _p(S))
    return S


def pv(p_codes, v_slabs) -> np.ndarray:
    """p_codes [n, T, T], v_slabs [n, T, d] -> O [n, T, d] int32."""
    p_codes, v_slabs = _i16(p_codes), _i16(v_slabs)
    n, T, T2 = p_codes.shape
    d = v_slabs.shape[2]
    O = np.empty((n, T, d), dtype=np.int32)
    lib().vo_pv(_p(p_codes), I64(T2), I64(T * T2), _p(v_slabs), I64(d), I64(T * d), I64(n), I64(T), I64(d), _p(O))
    return O


def softmax_quantize(S, c, p_step, bits: int, ulp_band: int = SOFTMAX_ULP_BAND):
    """S [rows, cols] int32 -> (p fp32, codes, lowest acceptable, highest acceptable)."""
    S = np.ascontiguousarray(S, dtype=np.int32)
    rows, cols = S.shape
    p = np.empty((rows, cols), dtype=np.float32)
    q = np.empty((rows, cols), dtype=np.int16)
    lo = np.empty_like(q)
    hi = np.empty_like(q)
    lib().vo_softmax_quantize(_p(S), I64(rows), I64(cols), I64(cols), F32(float(c)), F32(float(p_step)), I32(bits),
                              I32(ulp_band), _p(p), I64(cols), _p(q), _p(lo), _p(hi), I64(cols))
    return p, q, lo, hi


def softmax_shift_quantize(S, c2, p_step, bits: int, want_p: bool = False):
    """Eq. 4 softmax (2^r ~ 1+r, integer shifts) with the division-free comparator quantizer.
    S [rows, cols] int32 -> codes (and, optionally, the approximate probabilities E_j/Sigma in fp64)."""
    S = np.ascontiguousarray(S, dtype=np.int32)
    rows, cols = S.shape
    q = np.empty((rows, cols), dtype=np.int16)
    p = np.empty((rows, cols), dtype=np.float64) if want_p else None
    lib().vo_softmax_shift_quantize(_p(S), I64(rows), I64(cols), I64(cols), F32(float(c2)), F32(float(p_step)),
                                    I32(bits), _p(q), I64(cols), _p(p), I64(cols))
    return (q, p) if want_p else q


# ---- glue ---------------------------------------------------------------------

def layernorm(x, gamma, beta, eps: float = 1e-6):
    """Returns (y fp32, per-element absolute tolerance for an fp32 implementation)."""
    x, gamma, beta = _f32(x), _f32(gamma), _f32(beta)
    rows, cols = x.shape
    y = np.empty_like(x)
    tol = np.empty_like(x)
    lib().vo_layernorm(_p(x), I64(rows), I64(cols), I64(cols), _p(gamma), _p(beta), F32(eps), _p(y), I64(cols),
                       _p(tol), I64(cols))
    return y, tol


def layernorm_references(gamma, beta, step, bits: int, signed: bool, cols: int):
    """References of the division- and square-root-free LayerNorm comparator (Fig. 5(b)), fp64 then one
    rounding: for column j and threshold k = Qn+1..Qp, c = ((k - 1/2) step - beta_j) / gamma_j, taken with
    the sign flipped where gamma_j < 0.  Returns (ref = c^2 / cols as fp32 [cols, n_thr], neg = c < 0 as
    uint8 [cols, n_thr], flip = gamma < 0 as uint8 [cols])."""
    qn, qp = code_range(bits, signed)
    g = np.asarray(gamma, dtype=np.float64)[:, None]
    b = np.asarray(beta, dtype=np.float64)[:, None]
    k = np.arange(qn + 1, qp + 1, dtype=np.float64)[None, :]
    c = ((k - 0.5) * float(step) - b) / g
    flip = (g[:, 0] < 0)
    c = np.where(flip[:, None], -c, c)
    ref = (c * c / float(cols)).astype(np.float32)
    return np.ascontiguousarray(ref), np.ascontiguousarray((c < 0).astype(np.uint8)), flip.astype(np.uint8)


def layernorm_compare_quantize(x, ref, neg, flip, eps: float, bits: int, signed: bool, want_stats: bool = False):
    """Eq. 5 running statistics in fp32 + the comparator quantizer of Fig. 5(b).  x fp32 [rows, cols] -> codes
    (and, optionally, the row means and V = S_n + n*eps)."""
    x = _f32(x)
    rows, cols = x.shape
    ref = _f32(ref)
    neg = np.ascontiguousarray(neg, dtype=np.uint8)
    flip = np.ascontiguousarray(flip, dtype=np.uint8)
    q = np.empty((rows, cols), dtype=np.int16)
    mu = np.empty(rows, dtype=np.float32)
    v = np.empty(rows, dtype=np.float32)
    n_eps = np.float32(np.float64(cols) * np.float64(np.float32(eps)))
    lib().vo_layernorm_compare_quantize(_p(x), I64(rows), I64(cols), I64(cols), _p(ref), _p(neg), _p(flip),
                                        F32(float(n_eps)), I32(bits), I32(int(signed)), _p(q), I64(cols), _p(mu), _p(v))
    return (q, mu, v) if want_stats else q


def running_stats(x):
    x = _f32(x).ravel()
    mu = ctypes.c_double()
    m2 = ctypes.c_double()
    lib().vo_running_stats(_p(x), I64(x.size), ctypes.byref(mu), ctypes.byref(m2))
    return mu.value, m2.value


def quantize_band(y, tol, step, bits: int, signed: bool):
    y, tol = _f32(y), _f32(tol)
    rows, cols = y.shape
    q = np.empty((rows, cols), dtype=np.int16)
    lo = np.empty_like(q)
    hi = np.empty_like(q)
    lib().vo_quantize_band(_p(y), _p(tol), I64(rows), I64(cols), I64(cols), F32(float(step)), I32(bits),
                           I32(int(signed)), _p(q), _p(lo), _p(hi), I64(cols))
    return q, lo, hi
