"""Oracle of the overlaid bit-plane page format.  TEST INFRASTRUCTURE ONLY (see oracle.py).

The paper stores a linear-block as overlaid bit-planes plus a lookup table per supported bitwidth: a subset
of the planes is a lower-precision version of the same block, a bit-plane together with its lookup-table
state is one weight page, and lowering the precision moves no arithmetic at all -- the planes above the
committed precision simply stop being read (Sec. 2.2 "Any-Precision"; Sec. 3.1, page-table row; Eq. 3, size
table with the lookup-table metadata).  The paper does not say how its codes and centroids are fit, so this
build defines a nested code on top of its own group quantizer:

    master code   c4 = the 4-bit code of the group quantizer (quantize_block(w, 4): scale s4, zero-point z4)
    nested code   c_q = c4 >> (4 - q)                 for q = 4, 3, 2  (the first q bits, most significant first)
    lookup table  LUT_q[c] = fp16(z_q + c * s_q)      (affine), with
                  s_q = fp16(s4 * 2^(4-q))            (exact: a power of two)
                  z_q = fp16(fp32(z4) + fp32(s4) * (2^(4-q) - 1) / 2)   (the middle of the merged levels)

so the q-bit view of a block is an ordinary page (codes c_q, scales s_q, zero-points z_q) whose weights are
D(c_q, s_q, z_q), and every other part of the oracle applies to it unchanged.  Storage, in the order the
planes are attached: plane group "top" = the two most significant bits of c4, plane "bit1", plane "bit0";
the lookup-table state of each of the three bitwidths is kept with the block (it is a few bytes per group).
Canonical layout of a plane: little-endian bit stream in row-major element order, two bits per element for
"top", one bit per element for "bit1" / "bit0".
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Tuple

import numpy as np

from . import oracle

NESTED_BITS = (4, 3, 2)


@dataclass
class PlaneBlock:
    rows: int
    cols: int
    top: np.ndarray                    # uint8 stream, 2 bits per element
    bit1: np.ndarray                   # uint8 stream, 1 bit per element
    bit0: np.ndarray
    lut: Dict[int, Tuple[np.ndarray, np.ndarray]]   # q -> (scales, zero-points) uint16 [rows, cols/128]
    attached: int = 4                  # planes attached on the device: 2 (top), 3 (top, bit1), 4 (all)


def _f16(x: np.ndarray) -> np.ndarray:
    return x.astype(np.float32).astype(np.float16)


def quantize_planes(w_fp16: np.ndarray) -> PlaneBlock:
    """Nested quantization of an fp16 block: planes of the 4-bit master code + the three lookup-table states."""
    p4 = oracle.quantize_block(w_fp16, 4)
    c4 = oracle.unpack_codes(p4)                                   # uint8 [rows, cols]
    rows, cols = p4.rows, p4.cols
    top = np.packbits(np.unpackbits((c4 >> 2).reshape(-1, 1), axis=1, bitorder="little")[:, :2].reshape(-1),
                      bitorder="little")
    bit1 = np.packbits(((c4 >> 1) & 1).reshape(-1), bitorder="little")
    bit0 = np.packbits((c4 & 1).reshape(-1), bitorder="little")
    s4 = p4.scales.view(np.float16).astype(np.float32)
    z4 = p4.zps.view(np.float16).astype(np.float32)
    lut = {4: (p4.scales.copy(), p4.zps.copy())}
    for q in (3, 2):
        f = np.float32(2 ** (4 - q))
        sq = _f16(s4 * f)                                           # exact scaling
        zq = _f16(z4 + s4 * np.float32((f - 1) / 2))                # fp32 product (exact), fp32 add, one rounding to fp16
        lut[q] = (sq.view(np.uint16), zq.view(np.uint16))
    return PlaneBlock(rows, cols, top, bit1, bit0, lut)


def codes(block: PlaneBlock, q: int) -> np.ndarray:
    """The nested code c_q of every element, uint8 [rows, cols]: read from the first q bits only."""
    assert q in NESTED_BITS and q <= block.attached, "a plane that is not attached cannot be read"
    n = block.rows * block.cols
    t = np.unpackbits(block.top, bitorder="little")[: 2 * n].reshape(n, 2)
    c = (t[:, 0] | (t[:, 1] << 1)).astype(np.uint8)
    if q >= 3:
        c = (c << 1) | np.unpackbits(block.bit1, bitorder="little")[:n]
    if q == 4:
        c = (c << 1) | np.unpackbits(block.bit0, bitorder="little")[:n]
    return c.reshape(block.rows, block.cols)


def view(block: PlaneBlock, q: int) -> oracle.Page:
    """The block at q bits as an ordinary canonical page (codes c_q, lookup-table state of q)."""
    c = codes(block, q)
    bits = np.unpackbits(c.reshape(-1, 1), axis=1, bitorder="little")[:, :q].reshape(-1)
    stream = np.packbits(bits, bitorder="little")
    s, z = block.lut[q]
    return oracle.Page(stream, s.copy(), z.copy(), block.rows, block.cols, q)


def detach(block: PlaneBlock, q: int) -> PlaneBlock:
    """Lower the precision to q bits: the planes above it are no longer attached.  No value is touched."""
    assert q in NESTED_BITS and q <= block.attached
    return PlaneBlock(block.rows, block.cols, block.top, block.bit1, block.bit0, block.lut, attached=q)


def attach(block: PlaneBlock, q: int) -> PlaneBlock:
    """Raise the precision to q bits by re-attaching planes (they were kept, e.g. in host memory)."""
    assert q in NESTED_BITS and q >= block.attached
    return PlaneBlock(block.rows, block.cols, block.top, block.bit1, block.bit0, block.lut, attached=q)


def plane_bytes(rows: int, cols: int, q: int) -> int:
    """Size-table entry of Eq. 3 for a block read at q bits: q bit-planes + one lookup-table state
    (fp16 scale and zero-point per 128-weight group)."""
    assert q in NESTED_BITS
    return rows * cols * q // 8 + 4 * rows * (cols // oracle.GROUP)
