"""Helpers for the GPU parity tests: move oracle data to the device and back."""
from __future__ import annotations

import numpy as np
import torch

import oracle as vo
import paper_2504_18547_b200 as vt


# Tolerance granted to the library's fp32 GELU (glue between the integerized linears, not part of the integer
# path): |GELU_gpu(y) - GELU(y)| <= GELU_TOL_REL * |y| = 2^-22 |y|, about one unit in the last place of y itself.
# Measured over 3 * 2^20 arguments in [-9, 9] against the fp64 definition the kernel's largest error is
# 1.13e-7 * |y| (2^-23 = 1.19e-7; the bound leaves room for the rounding of the fp32 reference value itself); for
# y >= 0 that is at most 2.9 ulp of GELU(y), for y in [-0.5, 0) 3.4 ulp, and further down the negative side the
# bound is wide in ulp of the (tiny) result - where the quantizer that follows is unsigned and every such value
# becomes code 0.  The tolerance is the checker's, not the oracle's: the oracle defines GELU by erf in fp64 and
# takes the tolerance as an argument when it reports a band of codes.
GELU_TOL_REL = float(2.0 ** -22)


def to_codes(q: np.ndarray, bits: int, signed: bool, pitch: int | None = None) -> vt.Codes:
    """Oracle codes (int16 [rows, cols]) -> packed device codes, packed by the oracle's packer."""
    return vt.Codes.from_packed(vo.pack(q, bits, pitch), q.shape[1], bits, signed)


def from_codes(c: vt.Codes) -> np.ndarray:
    """Packed device codes -> int16 [rows, cols], unpacked by the oracle's unpacker."""
    return vo.unpack(c.data.cpu().numpy(), c.cols, c.stored_bits, c.signed)


def padding_is_zero(c: vt.Codes) -> bool:
    """Bytes between the last code of each row and the pitch must be zero."""
    raw = c.data.cpu().numpy()
    cb = c.stored_bits
    nbits = c.cols * cb
    full = nbits // 8
    ok = not raw[:, (nbits + 7) // 8:].any()
    if nbits % 8:
        ok = ok and not (raw[:, full] >> (nbits % 8)).any()
    return bool(ok)


def dev(a: np.ndarray | None):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def ulp_diff(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Distance in units in the last place between two fp32 arrays (same sign assumed or zero)."""
    ai = a.astype(np.float32).view(np.int32).astype(np.int64)
    bi = b.astype(np.float32).view(np.int32).astype(np.int64)
    ai = np.where(ai < 0, -(ai & 0x7FFFFFFF), ai)
    bi = np.where(bi < 0, -(bi & 0x7FFFFFFF), bi)
    return np.abs(ai - bi)


def rand_codes(seed: int, shape, bits: int, signed: bool) -> np.ndarray:
    import synth_inputs as si
    qn, qp = si.code_range(bits, signed)
    n = int(np.prod(shape))
    return ((si.splitmix64(seed, n) % np.uint64(qp - qn + 1)).astype(np.int64) + qn).astype(np.int16).reshape(shape)


# ---- guard bands: the stand-in for a memory checker -------------------------------------------------
# Every buffer handed out below sits between two 4 KB margins filled with a pattern; check_guards() verifies that
# no kernel wrote outside what it was given (a store past a row, a tile or the last element lands in a margin).
GUARD_BYTES = 4096
GUARD_PATTERN = 0xA5
_guarded = []


def guarded_bytes(nbytes: int, device="cuda") -> torch.Tensor:
    """uint8 tensor of `nbytes` (256-byte aligned) with patterned margins on both sides."""
    size = (nbytes + 255) // 256 * 256
    buf = torch.empty(size + 2 * GUARD_BYTES, dtype=torch.uint8, device=device)
    buf.fill_(GUARD_PATTERN)
    _guarded.append((buf, size))
    return buf[GUARD_BYTES:GUARD_BYTES + nbytes]


def guarded_codes(rows: int, cols: int, bits: int, signed: bool, container: int = 0, pitch: int | None = None) -> vt.Codes:
    pitch = vt.packed_pitch(cols, container or bits) if pitch is None else pitch
    data = guarded_bytes(rows * pitch).view(rows, pitch)
    return vt.Codes(data, rows, cols, bits, signed, container)


def guarded_tensor(shape, dtype) -> torch.Tensor:
    n = int(np.prod(shape))
    item = torch.empty((), dtype=dtype).element_size()
    return guarded_bytes(n * item).view(dtype).view(*shape)


def check_guards() -> int:
    """Asserts that every margin handed out since the last call still holds the pattern; returns how many buffers."""
    n = len(_guarded)
    for buf, size in _guarded:
        lo, hi = buf[:GUARD_BYTES], buf[GUARD_BYTES + size:]
        assert bool((lo == GUARD_PATTERN).all()), "a kernel wrote in front of its output buffer"
        assert bool((hi == GUARD_PATTERN).all()), "a kernel wrote behind its output buffer"
    _guarded.clear()
    return n
