"""Readers of the byte layouts that the C ABI (include/ais.h) states for its microscaling outputs.

Test helpers only.  The oracle returns plain arrays (one scale code per row and 32-element block, one 4-bit code
per element); the library returns the packed buffers the header documents.  These functions index a packed buffer
with the header's formulas, so that the comparison with the oracle is made on plain arrays and the oracle holds no
layout of the CUDA path.
"""

from __future__ import annotations

import numpy as np


def mx_scale_offsets(rows: int, cols: int) -> np.ndarray:
    """Byte offset of the scale of (row r, block kb) inside the packed array of ais_quantize_mxfp8 / _mxfp4, for
    all r < rows and kb < cols / 32, from the header's statement: chunk (r / 128, kb / 4) starts at
    ((r / 256) * (cols / 128) + kb / 4) * 1024 + ((r % 256) / 128) * 512 and the byte inside it is
    (r % 32) * 16 + ((r % 128) / 32) * 4 + kb % 4."""
    r = np.arange(rows, dtype=np.int64)[:, None]
    kb = np.arange(cols // 32, dtype=np.int64)[None, :]
    chunk = ((r // 256) * (cols // 128) + kb // 4) * 1024 + ((r % 256) // 128) * 512
    return chunk + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4


def mx_scale_bytes(rows: int, cols: int) -> int:
    """Size of the packed array: rows padded to a multiple of 256, one byte per row and block."""
    return (rows + 255) // 256 * 256 * (cols // 32)


def unpack_mx_scales(packed, rows: int, cols: int) -> np.ndarray:
    """Packed scale bytes -> plain uint8 [rows, cols / 32]."""
    flat = np.asarray(packed, dtype=np.uint8).reshape(-1)
    assert flat.size == mx_scale_bytes(rows, cols), (flat.size, rows, cols)
    return flat[mx_scale_offsets(rows, cols)]


def mx_scale_padding(packed, rows: int, cols: int) -> np.ndarray:
    """The bytes of the packed array that belong to no row < rows (the header says they hold 127)."""
    flat = np.asarray(packed, dtype=np.uint8).reshape(-1)
    used = np.zeros(flat.size, dtype=bool)
    used[mx_scale_offsets(rows, cols).reshape(-1)] = True
    return flat[~used]


def unpack_fp4_pairs(packed_codes) -> np.ndarray:
    """Bytes holding two 4-bit codes, the element with the lower index in the low nibble -> one code per entry."""
    b = np.asarray(packed_codes, dtype=np.uint8)
    out = np.empty(b.shape[:-1] + (b.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = b & 0x0F
    out[..., 1::2] = b >> 4
    return out
