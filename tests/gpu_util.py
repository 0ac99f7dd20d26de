"""Helpers for the GPU parity tests: move oracle data to the device and back."""
from __future__ import annotations

import numpy as np
import torch

import oracle as vo
import paper_2504_18547_b200 as vt


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
