"""ctypes binding of libvitint.so: same names as the C entry points, argument marshalling only."""
from __future__ import annotations

import ctypes
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int32, c_int64, c_size_t, c_void_p
from dataclasses import dataclass
from pathlib import Path

import numpy as np
import torch

_LIB_PATH = Path(__file__).resolve().parent / "libvitint.so"

EPI_ACC_I32, EPI_DEQUANT_F32, EPI_REQUANT = 0, 1, 2


class VitintError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {vitint_status_string(code)} ({code})")


class _Codes(Structure):
    _fields_ = [("data", c_void_p), ("rows", c_int64), ("cols", c_int64), ("pitch_bytes", c_int64),
                ("bits", c_int32), ("is_signed", c_int32), ("container_bits", c_int32), ("reserved_", c_int32)]


class _Epilogue(Structure):
    _fields_ = [("mode", c_int32), ("act", c_int32), ("residual", c_void_p), ("ld_res", c_int64),
                ("alpha", c_void_p), ("beta", c_void_p), ("inv_out_step", c_void_p),
                ("out_bits", c_int32), ("out_signed", c_int32), ("out_container_bits", c_int32),
                ("reserved_", c_int32)]


class _Slabs(Structure):
    _fields_ = [("data", c_void_p), ("pitch_bytes", c_int64), ("image_stride_bytes", c_int64),
                ("head_stride_bytes", c_int64), ("bits", c_int32), ("is_signed", c_int32)]


class _AttentionDesc(Structure):
    _fields_ = [("batch", c_int32), ("tokens", c_int32), ("heads", c_int32), ("bits", c_int32),
                ("w_qkv", _Codes), ("alpha_qkv", c_void_p), ("beta_qkv", c_void_p),
                ("q_step", c_float), ("k_step", c_float), ("v_step", c_float), ("p_step", c_float),
                ("o_step", c_float), ("p_bits", c_int32), ("alpha_o", c_void_p), ("beta_o", c_void_p),
                ("w_proj", _Codes), ("w_proj_step", c_void_p), ("b_proj", c_void_p), ("proj_epi", _Epilogue)]


_lib = None


def lib():
    """Loads the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with paper_2504_18547_b200.build.build_library(); "
                               "there is no fallback path")
        L = ctypes.CDLL(str(_LIB_PATH))
        L.vitint_status_string.restype = c_char_p
        L.vitint_status_string.argtypes = [ctypes.c_int]
        L.vitint_version.restype = ctypes.c_int
        L.vitint_device_status.restype = ctypes.c_int
        L.vitint_packed_pitch.restype = c_int64
        L.vitint_packed_pitch.argtypes = [c_int64, c_int32]
        L.vitint_quantize.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_float, c_void_p, POINTER(_Codes), c_void_p]
        L.vitint_widen.argtypes = [POINTER(_Codes), POINTER(_Codes), c_void_p]
        L.vitint_linear.argtypes = [POINTER(_Codes), c_float, POINTER(_Codes), c_void_p, c_void_p, POINTER(_Epilogue),
                                    c_void_p, c_int64, c_void_p]
        L.vitint_qk.argtypes = [POINTER(_Slabs), POINTER(_Slabs), c_int32, c_int32, c_int32, c_void_p, c_int64, c_void_p]
        L.vitint_softmax_quantize.argtypes = [c_void_p, c_int64, c_int32, c_int64, c_float, c_float, POINTER(_Codes),
                                              c_void_p, c_int64, c_void_p]
        L.vitint_softmax_shift_quantize.argtypes = [c_void_p, c_int64, c_int32, c_int64, c_float, c_float,
                                                    POINTER(_Codes), c_void_p]
        L.vitint_pv.argtypes = [POINTER(_Codes), POINTER(_Slabs), c_int32, c_int32, c_int32, c_float, c_float,
                                POINTER(_Epilogue), c_void_p, c_int64, c_void_p]
        L.vitint_attention_core_workspace_bytes.restype = c_size_t
        L.vitint_attention_core_workspace_bytes.argtypes = [c_int32]
        L.vitint_attention_core.argtypes = [POINTER(_Codes), c_int32, c_int32, c_int32, c_float, c_float, c_float,
                                            c_int32, c_void_p, c_void_p, POINTER(_Codes), c_void_p, c_size_t, c_void_p]
        L.vitint_attention_core_shift_workspace_bytes.restype = c_size_t
        L.vitint_attention_core_shift_workspace_bytes.argtypes = [c_int32]
        L.vitint_attention_core_shift.argtypes = [POINTER(_Codes), c_int32, c_int32, c_int32, c_float, c_float, c_float,
                                                  c_int32, c_void_p, c_void_p, POINTER(_Codes), c_void_p, c_size_t,
                                                  c_int32, c_void_p]
        L.vitint_attention_exp_table.argtypes = [c_int32, c_float, c_float, c_void_p, c_size_t, c_void_p]
        L.vitint_attention_core_prepared.argtypes = [POINTER(_Codes), c_int32, c_int32, c_int32, c_float, c_float, c_float,
                                                     c_int32, c_void_p, c_void_p, POINTER(_Codes), c_void_p, c_size_t,
                                                     c_void_p]
        L.vitint_attention_core_noalloc.argtypes = [POINTER(_Codes), c_int32, c_int32, c_int32, c_float, c_float, c_float,
                                                    c_int32, c_void_p, c_void_p, POINTER(_Codes), c_void_p]
        L.vitint_attention_block_workspace_bytes.restype = c_size_t
        L.vitint_attention_block_workspace_bytes.argtypes = [POINTER(_AttentionDesc)]
        L.vitint_attention_block.argtypes = [POINTER(_Codes), POINTER(_AttentionDesc), c_void_p, c_int64,
                                             POINTER(_Codes), POINTER(_Codes), POINTER(_Codes), c_void_p, c_size_t,
                                             c_void_p]
        L.vitint_layernorm_compare_quantize.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_float,
                                                        POINTER(_Codes), c_void_p, c_void_p]
        L.vitint_linear_e2m1.argtypes = [POINTER(_Codes), POINTER(_Codes), c_void_p, c_int64, c_void_p, c_void_p]
        L.vitint_linear_qkv_norm.argtypes = [POINTER(_Codes), c_float, POINTER(_Codes), c_void_p, c_void_p, c_void_p, c_void_p,
                                             c_float, c_void_p, c_void_p, POINTER(_Codes), c_void_p, c_void_p]
        L.vitint_softmax_table_workspace_bytes.restype = c_size_t
        L.vitint_softmax_table_workspace_bytes.argtypes = [c_int32]
        L.vitint_softmax_quantize_bounded.argtypes = [c_void_p, c_int64, c_int32, c_int64, c_float, c_float, c_int32,
                                                      POINTER(_Codes), c_void_p, c_int64, c_void_p, c_size_t, c_int32,
                                                      c_void_p]
        L.vitint_selftest_wait_timeout.argtypes = [c_int64, c_void_p, c_void_p]
        L.vitint_fold_requant.argtypes = [c_float, c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_void_p]
        L.vitint_fold_layernorm_references.argtypes = [c_void_p, c_void_p, c_float, c_int32, c_int32, c_int64, c_void_p,
                                                       c_void_p]
        L.vitint_layernorm_quantize.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_float,
                                                c_float, POINTER(_Codes), c_void_p, c_int64, c_void_p]
        _lib = L
    return _lib


def vitint_status_string(code: int) -> str:
    return lib().vitint_status_string(code).decode()


def vitint_version() -> int:
    return lib().vitint_version()


def vitint_device_status() -> int:
    return lib().vitint_device_status()


def vitint_selftest_wait_timeout(limit_cycles: int, gave_up: torch.Tensor | None = None) -> None:
    """Launches the library's bounded-wait self-test (a wait that nothing completes; gives up after `limit_cycles`)."""
    _check(lib().vitint_selftest_wait_timeout(int(limit_cycles), _ptr(gave_up), _stream()), "vitint_selftest_wait_timeout")


def packed_pitch(cols: int, bits: int) -> int:
    return int(lib().vitint_packed_pitch(cols, bits))


def _check(code: int, where: str):
    if code != 0:
        raise VitintError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def _ld(t) -> int:
    """Leading dimension in elements of a 2-D tensor (a single row reports its width)."""
    return int(t.stride(0)) if t.shape[0] > 1 else max(int(t.stride(0)), int(t.shape[-1]))


@dataclass
class Codes:
    """Packed low-bit codes on the device: a uint8 tensor [rows, pitch] plus the logical shape."""
    data: torch.Tensor
    rows: int
    cols: int
    bits: int
    signed: bool
    container: int = 0        # 0: default container of `bits`; 8: one code per byte

    @staticmethod
    def empty(rows: int, cols: int, bits: int, signed: bool, device="cuda", pitch: int | None = None,
              container: int = 0) -> "Codes":
        pitch = packed_pitch(cols, container or bits) if pitch is None else pitch
        return Codes(torch.empty((rows, pitch), dtype=torch.uint8, device=device), rows, cols, bits, signed, container)

    @property
    def stored_bits(self) -> int:
        """Bits per stored code."""
        return self.container or (4 if self.bits == 3 else self.bits)

    @staticmethod
    def from_packed(packed: np.ndarray, cols: int, bits: int, signed: bool, device="cuda") -> "Codes":
        t = torch.from_numpy(np.ascontiguousarray(packed, dtype=np.uint8)).to(device)
        return Codes(t, t.shape[0], cols, bits, signed)

    @property
    def pitch(self) -> int:
        return int(self.data.stride(0))

    def desc(self) -> _Codes:
        return _Codes(self.data.data_ptr(), self.rows, self.cols, self.pitch, self.bits, int(self.signed),
                      self.container, 0)


@dataclass
class Epilogue:
    mode: int = EPI_ACC_I32
    act: int = 0
    residual: torch.Tensor | None = None
    alpha: torch.Tensor | None = None
    beta: torch.Tensor | None = None
    inv_out_step: torch.Tensor | None = None
    out_bits: int = 4
    out_signed: bool = True
    out_container: int = 0

    def desc(self) -> _Epilogue:
        ld_res = _ld(self.residual) if self.residual is not None else 0
        return _Epilogue(self.mode, self.act, _ptr(self.residual), ld_res, _ptr(self.alpha), _ptr(self.beta),
                         _ptr(self.inv_out_step), self.out_bits, int(self.out_signed), self.out_container, 0)


@dataclass
class Slabs:
    """[tokens, 64] code slabs per (image, head) inside a packed code matrix."""
    base: torch.Tensor        # the uint8 tensor that owns the memory
    byte_offset: int          # of slab (0, 0) from base
    pitch: int
    image_stride: int
    head_stride: int
    bits: int
    signed: bool

    @staticmethod
    def of_qkv(qkv: Codes, tokens: int, dim: int, part: int) -> "Slabs":
        """part 0/1/2 = Q/K/V columns of a [batch*tokens, 3*dim] code matrix."""
        c = 4 if qkv.bits == 3 else qkv.bits
        return Slabs(qkv.data, part * dim * c // 8, qkv.pitch, qkv.pitch * tokens, 64 * c // 8, qkv.bits, qkv.signed)

    def desc(self) -> _Slabs:
        return _Slabs(self.base.data_ptr() + self.byte_offset, self.pitch, self.image_stride, self.head_stride,
                      self.bits, int(self.signed))


def vitint_fold_requant(s_x, s_w, bias, s_out):
    """Host helper of the library (Eq. 2 folding): alpha = s_x*s_w/s_out, beta = b/s_out per output channel.
    s_w, bias (or None), s_out: host arrays (s_out may be a scalar).  Returns (alpha, beta) as fp32 numpy arrays."""
    s_w = np.ascontiguousarray(s_w, dtype=np.float32).ravel()
    n = s_w.size
    s_out = np.ascontiguousarray(np.broadcast_to(np.asarray(s_out, dtype=np.float32), (n,)))
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32).ravel()
    alpha, beta = np.empty(n, np.float32), np.empty(n, np.float32)
    fp = lambda a: None if a is None else a.ctypes.data_as(c_void_p)
    _check(lib().vitint_fold_requant(float(s_x), fp(s_w), fp(bias), fp(s_out), n, fp(alpha), fp(beta)), "vitint_fold_requant")
    return alpha, beta


def vitint_fold_layernorm_references(gamma, beta, step, bits: int, signed: bool, cols: int):
    """Host helper of the library (Fig. 5(b)): signed comparator references and per-column flip flags for
    vitint_layernorm_compare_quantize.  Returns (refs fp32 [cols, 2^bits - 1], flip uint8 [cols])."""
    gamma = np.ascontiguousarray(gamma, dtype=np.float32).ravel()
    beta = np.ascontiguousarray(beta, dtype=np.float32).ravel()
    n_thr = (1 << bits) - 1
    refs, flip = np.empty((cols, n_thr), np.float32), np.empty(cols, np.uint8)
    fp = lambda a: a.ctypes.data_as(c_void_p)
    _check(lib().vitint_fold_layernorm_references(fp(gamma), fp(beta), float(step), bits, int(signed), cols, fp(refs),
                                                  fp(flip)), "vitint_fold_layernorm_references")
    return refs, flip


# names kept for callers of the earlier Python helpers
fold_requant = vitint_fold_requant
fold_layernorm_references = vitint_fold_layernorm_references


# ---------------------------------------------------------------------------
# entry points (same names as include/vitint.h)
# ---------------------------------------------------------------------------

def vitint_quantize(x: torch.Tensor, step: float, bits: int, signed: bool, row_steps: torch.Tensor | None = None,
                    out: Codes | None = None) -> Codes:
    rows, cols = x.shape
    out = Codes.empty(rows, cols, bits, signed, x.device) if out is None else out
    d = out.desc()
    _check(lib().vitint_quantize(x.data_ptr(), rows, cols, _ld(x), float(step), _ptr(row_steps), byref(d),
                                 _stream()), "vitint_quantize")
    return out


def vitint_widen(x: Codes, out: Codes | None = None) -> Codes:
    """The same codes in 8-bit containers (used once for weights)."""
    out = Codes.empty(x.rows, x.cols, x.bits, x.signed, x.data.device, container=8) if out is None else out
    di, do = x.desc(), out.desc()
    _check(lib().vitint_widen(byref(di), byref(do), _stream()), "vitint_widen")
    return out


def _alloc_out(epi: Epilogue, rows: int, cols: int, device):
    if epi.mode == EPI_ACC_I32:
        return torch.empty((rows, cols), dtype=torch.int32, device=device)
    if epi.mode == EPI_DEQUANT_F32:
        return torch.empty((rows, cols), dtype=torch.float32, device=device)
    return Codes.empty(rows, cols, epi.out_bits, epi.out_signed, device, container=epi.out_container)


def _out_ptr_ld(out):
    if isinstance(out, Codes):
        return out.data.data_ptr(), out.pitch
    return out.data_ptr(), _ld(out)


def vitint_linear(x: Codes, x_step: float, w: Codes, w_step: torch.Tensor | None, bias: torch.Tensor | None,
                  epi: Epilogue, out=None):
    out = _alloc_out(epi, x.rows, w.rows, x.data.device) if out is None else out
    ptr, ld = _out_ptr_ld(out)
    dx, dw, de = x.desc(), w.desc(), epi.desc()
    _check(lib().vitint_linear(byref(dx), float(x_step), byref(dw), _ptr(w_step), _ptr(bias), byref(de), ptr, ld,
                               _stream()), "vitint_linear")
    return out


def vitint_linear_qkv_norm(x: Codes, x_step: float, w_qkv: Codes, w_step: torch.Tensor, bias: torch.Tensor | None,
                           refs: torch.Tensor, flip: torch.Tensor | None, n_eps: float, alpha_v: torch.Tensor,
                           beta_v: torch.Tensor | None, bits: int, out: Codes | None = None,
                           stats: torch.Tensor | None = None):
    """QKV projection whose epilogue normalises and quantizes every Q and K head (Eq. 5 statistics, comparator
    quantizer of Fig. 5(b)) and requantizes V.  refs: [2, 64, 2^bits - 1], flip: [2, 64] uint8 or None (Q's then
    K's).  Returns (codes [M, 3D], stats [2, M*heads, 2])."""
    M, N = x.rows, w_qkv.rows
    out = Codes.empty(M, N, bits, True, x.data.device) if out is None else out
    stats = torch.empty((2, M * (N // 192), 2), dtype=torch.float32, device=x.data.device) if stats is None else stats
    dx, dw, do = x.desc(), w_qkv.desc(), out.desc()
    _check(lib().vitint_linear_qkv_norm(byref(dx), float(x_step), byref(dw), w_step.data_ptr(), _ptr(bias), refs.data_ptr(),
                                        _ptr(flip), float(n_eps), alpha_v.data_ptr(), _ptr(beta_v), byref(do),
                                        stats.data_ptr(), _stream()), "vitint_linear_qkv_norm")
    return out, stats


def vitint_linear_e2m1(x: Codes, w: Codes, out: torch.Tensor | None = None, inexact: torch.Tensor | None = None):
    """Raw accumulators of the integer linear layer computed through the FP4 (e2m1) tensor-core kind.  x, w: codes
    stored one per byte, signed of at most 3 bits or unsigned of at most 2.  Returns (int32 [M, N], flag): the flag
    (device int32) becomes 1 if any fp32 accumulator was not an integer."""
    out = torch.empty((x.rows, w.rows), dtype=torch.int32, device=x.data.device) if out is None else out
    inexact = torch.zeros(1, dtype=torch.int32, device=x.data.device) if inexact is None else inexact
    dx, dw = x.desc(), w.desc()
    _check(lib().vitint_linear_e2m1(byref(dx), byref(dw), out.data_ptr(), _ld(out), inexact.data_ptr(), _stream()),
           "vitint_linear_e2m1")
    return out, inexact


def vitint_qk(q: Slabs, k: Slabs, batch: int, heads: int, tokens: int, out: torch.Tensor | None = None,
              ld_s: int | None = None) -> torch.Tensor:
    ld_s = (tokens + 3) // 4 * 4 if ld_s is None else ld_s
    if out is None:
        out = torch.empty((batch * heads, tokens, ld_s), dtype=torch.int32, device=q.base.device)
    dq, dk = q.desc(), k.desc()
    _check(lib().vitint_qk(byref(dq), byref(dk), batch, heads, tokens, out.data_ptr(), ld_s, _stream()), "vitint_qk")
    return out


def vitint_softmax_quantize(s: torch.Tensor, cols: int, c: float, p_step: float, bits: int,
                            want_p: bool = False, out: Codes | None = None):
    """s: int32 [rows, ld_s] (only the first `cols` columns of each row are read)."""
    rows, ld_s = s.shape[0], _ld(s)
    out = Codes.empty(rows, cols, bits, False, s.device) if out is None else out
    p = torch.empty((rows, cols), dtype=torch.float32, device=s.device) if want_p else None
    d = out.desc()
    _check(lib().vitint_softmax_quantize(s.data_ptr(), rows, cols, ld_s, float(c), float(p_step), byref(d), _ptr(p),
                                         cols if want_p else 0, _stream()), "vitint_softmax_quantize")
    return (out, p) if want_p else out


def vitint_softmax_table_workspace_bytes(score_bound: int) -> int:
    return int(lib().vitint_softmax_table_workspace_bytes(int(score_bound)))


def vitint_softmax_quantize_bounded(s: torch.Tensor, cols: int, c: float, p_step: float, bits: int, score_bound: int,
                                    want_p: bool = False, out: Codes | None = None,
                                    workspace: torch.Tensor | None = None, table_ready: bool = False):
    """vitint_softmax_quantize for scores known to lie in -score_bound .. score_bound (exp from a table).
    workspace: uint8 device tensor of vitint_softmax_table_workspace_bytes(score_bound) bytes (allocated if None)."""
    rows, ld_s = s.shape[0], _ld(s)
    out = Codes.empty(rows, cols, bits, False, s.device) if out is None else out
    p = torch.empty((rows, cols), dtype=torch.float32, device=s.device) if want_p else None
    if workspace is None:
        workspace = torch.empty(vitint_softmax_table_workspace_bytes(score_bound), dtype=torch.uint8, device=s.device)
    d = out.desc()
    _check(lib().vitint_softmax_quantize_bounded(s.data_ptr(), rows, cols, ld_s, float(c), float(p_step), int(score_bound),
                                                 byref(d), _ptr(p), cols if want_p else 0, workspace.data_ptr(),
                                                 workspace.numel(), int(table_ready), _stream()),
           "vitint_softmax_quantize_bounded")
    return (out, p) if want_p else out


def vitint_softmax_shift_quantize(s: torch.Tensor, cols: int, c2: float, p_step: float, bits: int,
                                  out: Codes | None = None) -> Codes:
    """Eq. 4 softmax (2^r ~ 1 + r, integer shifts) with the division-free comparator quantizer."""
    rows, ld_s = s.shape[0], _ld(s)
    out = Codes.empty(rows, cols, bits, False, s.device) if out is None else out
    d = out.desc()
    _check(lib().vitint_softmax_shift_quantize(s.data_ptr(), rows, cols, ld_s, float(c2), float(p_step), byref(d),
                                               _stream()), "vitint_softmax_shift_quantize")
    return out


def vitint_pv(p: Codes, v: Slabs, batch: int, heads: int, tokens: int, p_step: float, v_step: float, epi: Epilogue,
              out=None):
    out = _alloc_out(epi, batch * tokens, heads * 64, p.data.device) if out is None else out
    ptr, ld = _out_ptr_ld(out)
    dp, dv, de = p.desc(), v.desc(), epi.desc()
    _check(lib().vitint_pv(byref(dp), byref(dv), batch, heads, tokens, float(p_step), float(v_step), byref(de), ptr,
                           ld, _stream()), "vitint_pv")
    return out


def vitint_attention_core_workspace_bytes(bits: int) -> int:
    return int(lib().vitint_attention_core_workspace_bytes(bits))


def vitint_attention_core(qkv: Codes, batch: int, heads: int, tokens: int, q_step: float, k_step: float,
                          p_step: float, p_bits: int, alpha_o: torch.Tensor, beta_o: torch.Tensor | None,
                          out: Codes | None = None, out_bits: int | None = None,
                          workspace: torch.Tensor | None = None) -> Codes:
    """Fused Q K^T -> softmax -> quantize -> P V -> requantize; `out` holds signed codes [batch*tokens, heads*64]."""
    if out is None:
        out = Codes.empty(batch * tokens, heads * 64, qkv.bits if out_bits is None else out_bits, True, qkv.data.device)
    if workspace is None:
        workspace = torch.empty(vitint_attention_core_workspace_bytes(qkv.bits), dtype=torch.uint8,
                                device=qkv.data.device)
    dq, do = qkv.desc(), out.desc()
    _check(lib().vitint_attention_core(byref(dq), batch, heads, tokens, float(q_step), float(k_step), float(p_step),
                                       p_bits, _ptr(alpha_o), _ptr(beta_o), byref(do), workspace.data_ptr(),
                                       workspace.numel(), _stream()), "vitint_attention_core")
    return out


def vitint_attention_core_shift_workspace_bytes(bits: int) -> int:
    return int(lib().vitint_attention_core_shift_workspace_bytes(int(bits)))


def vitint_attention_core_shift(qkv: Codes, batch: int, heads: int, tokens: int, q_step: float, k_step: float,
                                p_step: float, p_bits: int, alpha_o: torch.Tensor, beta_o: torch.Tensor | None,
                                out: Codes | None = None, out_bits: int | None = None,
                                workspace: torch.Tensor | None = None, table_ready: bool = False) -> Codes:
    """The fused attention core with the Eq. 4 softmax and its division-free comparator quantizer (byte-stored codes).
    table_ready: `workspace` still holds the table an earlier call with the same bits and steps built."""
    if out is None:
        out = Codes.empty(batch * tokens, heads * 64, qkv.bits if out_bits is None else out_bits, True, qkv.data.device)
    if workspace is None:
        workspace = torch.empty(vitint_attention_core_shift_workspace_bytes(qkv.bits), dtype=torch.uint8,
                                device=qkv.data.device)
    dq, do = qkv.desc(), out.desc()
    _check(lib().vitint_attention_core_shift(byref(dq), batch, heads, tokens, float(q_step), float(k_step), float(p_step),
                                             p_bits, _ptr(alpha_o), _ptr(beta_o), byref(do), workspace.data_ptr(),
                                             workspace.numel(), int(table_ready), _stream()), "vitint_attention_core_shift")
    return out


def vitint_attention_exp_table(bits: int, q_step: float, k_step: float, table: torch.Tensor | None = None,
                               device="cuda") -> torch.Tensor:
    """Fills (and returns) the exp table of the fused attention core for these steps; see
    vitint_attention_core_prepared."""
    if table is None:
        table = torch.empty(vitint_attention_core_workspace_bytes(bits), dtype=torch.uint8, device=device)
    _check(lib().vitint_attention_exp_table(bits, float(q_step), float(k_step), table.data_ptr(), table.numel(),
                                            _stream()), "vitint_attention_exp_table")
    return table


def vitint_attention_core_prepared(qkv: Codes, batch: int, heads: int, tokens: int, q_step: float, k_step: float,
                                   p_step: float, p_bits: int, alpha_o: torch.Tensor, beta_o: torch.Tensor | None,
                                   out: Codes, table: torch.Tensor) -> Codes:
    """vitint_attention_core with a table filled once by vitint_attention_exp_table (same bits and steps)."""
    dq, do = qkv.desc(), out.desc()
    _check(lib().vitint_attention_core_prepared(byref(dq), batch, heads, tokens, float(q_step), float(k_step),
                                                float(p_step), p_bits, _ptr(alpha_o), _ptr(beta_o), byref(do),
                                                table.data_ptr(), table.numel(), _stream()),
           "vitint_attention_core_prepared")
    return out


def vitint_attention_core_noalloc(qkv: Codes, batch: int, heads: int, tokens: int, q_step: float, k_step: float,
                                  p_step: float, p_bits: int, alpha_o: torch.Tensor, beta_o: torch.Tensor | None,
                                  out: Codes) -> Codes:
    """vitint_attention_core for callers that may not allocate device memory: the kernel's scratch is a
    fixed array inside the library and `out` must be supplied.  This wrapper allocates nothing either."""
    dq, do = qkv.desc(), out.desc()
    _check(lib().vitint_attention_core_noalloc(byref(dq), batch, heads, tokens, float(q_step), float(k_step),
                                               float(p_step), p_bits, _ptr(alpha_o), _ptr(beta_o), byref(do),
                                               _stream()), "vitint_attention_core_noalloc")
    return out


@dataclass
class AttentionWeights:
    """Device-resident parameters of one integerized attention block."""
    batch: int
    tokens: int
    heads: int
    bits: int
    w_qkv: Codes
    alpha_qkv: torch.Tensor
    beta_qkv: torch.Tensor
    q_step: float
    k_step: float
    v_step: float
    p_step: float
    o_step: float
    p_bits: int
    alpha_o: torch.Tensor
    beta_o: torch.Tensor | None
    w_proj: Codes
    w_proj_step: torch.Tensor
    b_proj: torch.Tensor | None
    proj_epi: Epilogue

    def desc(self) -> _AttentionDesc:
        return _AttentionDesc(self.batch, self.tokens, self.heads, self.bits, self.w_qkv.desc(),
                              _ptr(self.alpha_qkv), _ptr(self.beta_qkv), self.q_step, self.k_step, self.v_step,
                              self.p_step, self.o_step, self.p_bits, _ptr(self.alpha_o), _ptr(self.beta_o),
                              self.w_proj.desc(), _ptr(self.w_proj_step), _ptr(self.b_proj), self.proj_epi.desc())


def vitint_attention_block_workspace_bytes(a: AttentionWeights) -> int:
    d = a.desc()
    return int(lib().vitint_attention_block_workspace_bytes(byref(d)))


def vitint_attention_block(x: Codes, a: AttentionWeights, out=None, workspace: torch.Tensor | None = None,
                           dbg_qkv: Codes | None = None, dbg_p: Codes | None = None, dbg_o: Codes | None = None):
    dim = a.heads * 64
    out = _alloc_out(a.proj_epi, x.rows, dim, x.data.device) if out is None else out
    if workspace is None:
        workspace = torch.empty(vitint_attention_block_workspace_bytes(a), dtype=torch.uint8, device=x.data.device)
    ptr, ld = _out_ptr_ld(out)
    d, dx = a.desc(), x.desc()
    dbg = [None if c is None else c.desc() for c in (dbg_qkv, dbg_p, dbg_o)]
    refs = [None if c is None else byref(c) for c in dbg]
    _check(lib().vitint_attention_block(byref(dx), byref(d), ptr, ld, refs[0], refs[1], refs[2],
                                        workspace.data_ptr(), workspace.numel(), _stream()), "vitint_attention_block")
    return out


def vitint_layernorm_quantize(x: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor, eps: float, step: float,
                              bits: int, signed: bool = True, want_y: bool = False, out: Codes | None = None):
    rows, cols = x.shape
    out = Codes.empty(rows, cols, bits, signed, x.device) if out is None else out
    y = torch.empty((rows, cols), dtype=torch.float32, device=x.device) if want_y else None
    d = out.desc()
    _check(lib().vitint_layernorm_quantize(x.data_ptr(), rows, cols, _ld(x), gamma.data_ptr(), beta.data_ptr(),
                                           float(eps), float(step), byref(d), _ptr(y), cols if want_y else 0,
                                           _stream()), "vitint_layernorm_quantize")
    return (out, y) if want_y else out


def vitint_layernorm_compare_quantize(x: torch.Tensor, refs: torch.Tensor, flip: torch.Tensor | None, n_eps: float,
                                      bits: int, signed: bool = True, out: Codes | None = None,
                                      stats: torch.Tensor | None = None):
    """Eq. 5 running statistics + the comparator quantizer of Fig. 5(b).  Returns (codes, stats [rows, 2])."""
    rows, cols = x.shape
    out = Codes.empty(rows, cols, bits, signed, x.device) if out is None else out
    stats = torch.empty((rows, 2), dtype=torch.float32, device=x.device) if stats is None else stats
    d = out.desc()
    _check(lib().vitint_layernorm_compare_quantize(x.data_ptr(), rows, cols, _ld(x), refs.data_ptr(), _ptr(flip),
                                                   float(n_eps), byref(d), stats.data_ptr(), _stream()),
           "vitint_layernorm_compare_quantize")
    return out, stats
