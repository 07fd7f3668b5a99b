"""ctypes front end of the CPU oracle (``pw_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
module; nothing in the product package does.  Arrays are numpy, pages are held in
the canonical layout (little-endian bit stream of codes in row-major element
order, fp16 scale / zero-point per 128-weight group).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pw_oracle.cpp")
_LIB = os.path.join(_HERE, "libpw_oracle.so")
_lib = None

BITS = (16, 8, 4, 3, 2)
GROUP = 128


def build(force: bool = False) -> str:
    """Compile the oracle with the flags its arithmetic rules require."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
               _SRC, "-o", _LIB]
        subprocess.check_call(cmd)
    return _LIB


class _CPage(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("zps", C.c_void_p),
                ("rows", C.c_uint32), ("cols", C.c_uint32), ("group", C.c_int32), ("bits", C.c_int32)]


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.orc_f32_to_f16.restype = C.c_uint16
        L.orc_f32_to_f16.argtypes = [C.c_float]
        L.orc_f16_to_f32.restype = C.c_float
        L.orc_f16_to_f32.argtypes = [C.c_uint16]
        L.orc_page_bytes.restype = C.c_uint64
        L.orc_page_bytes.argtypes = [C.c_uint32, C.c_uint32, C.c_int, C.c_int] + [C.POINTER(C.c_uint64)] * 3
        vp = C.c_void_p
        L.orc_quantize_block.restype = C.c_int
        L.orc_quantize_block.argtypes = [vp, C.c_uint32, C.c_uint32, C.c_int, C.c_int, vp, vp, vp]
        L.orc_dequantize_block.restype = C.c_int
        L.orc_dequantize_block.argtypes = [vp, vp, vp, C.c_uint32, C.c_uint32, C.c_int, C.c_int, vp]
        L.orc_demote_block.restype = C.c_int
        L.orc_demote_block.argtypes = [vp, vp, vp, C.c_uint32, C.c_uint32, C.c_int, C.c_int, C.c_int, vp, vp, vp]
        L.orc_router.restype = C.c_int
        L.orc_router.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp]
        L.orc_permute.restype = C.c_int
        L.orc_permute.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp]
        L.orc_moe_forward.restype = C.c_int
        L.orc_moe_forward.argtypes = [vp, vp] + [C.c_int] * 6 + [C.POINTER(_CPage), vp, vp]
        L.orc_moe_forward_bruteforce.restype = C.c_int
        L.orc_moe_forward_bruteforce.argtypes = [vp, vp] + [C.c_int] * 6 + [C.POINTER(_CPage), vp]
        L.orc_num_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class Page:
    """One linear-block at one bitwidth, canonical layout, host memory."""
    codes: np.ndarray                 # uint8 stream (bits < 16) or the raw fp16 weights viewed as uint8
    scales: Optional[np.ndarray]      # uint16 [rows, cols/group] (fp16 bit patterns); None at 16 bits
    zps: Optional[np.ndarray]
    rows: int
    cols: int
    bits: int
    group: int = GROUP

    @property
    def nbytes(self) -> int:
        return page_bytes(self.rows, self.cols, self.bits, self.group)[0]


def page_bytes(rows: int, cols: int, bits: int, group: int = GROUP):
    """(total, codes, scales, zps) bytes of a block at ``bits`` -- the size table M_i^b of Eq. 3."""
    cb, sb, zb = C.c_uint64(), C.c_uint64(), C.c_uint64()
    tot = lib().orc_page_bytes(rows, cols, bits, group, C.byref(cb), C.byref(sb), C.byref(zb))
    if tot == 0:
        raise ValueError("invalid page shape or bitwidth")
    return int(tot), int(cb.value), int(sb.value), int(zb.value)


def _as_u16(w: np.ndarray) -> np.ndarray:
    if w.dtype == np.float16:
        w = w.view(np.uint16)
    assert w.dtype == np.uint16
    return np.ascontiguousarray(w)


def quantize_block(w_fp16: np.ndarray, bits: int, group: int = GROUP) -> Page:
    w = _as_u16(w_fp16)
    rows, cols = w.shape
    _, cb, sb, _ = page_bytes(rows, cols, bits, group)
    codes = np.zeros(cb, np.uint8)
    if bits == 16:
        scales = zps = None
    else:
        scales = np.zeros((rows, cols // group), np.uint16)
        zps = np.zeros((rows, cols // group), np.uint16)
    rc = lib().orc_quantize_block(_p(w), rows, cols, bits, group, _p(codes), _p(scales), _p(zps))
    if rc:
        raise ValueError("orc_quantize_block failed (%d)" % rc)
    return Page(codes, scales, zps, rows, cols, bits, group)


def dequantize_block(pg: Page) -> np.ndarray:
    out = np.zeros((pg.rows, pg.cols), np.uint16)
    rc = lib().orc_dequantize_block(_p(pg.codes), _p(pg.scales), _p(pg.zps), pg.rows, pg.cols, pg.bits, pg.group,
                                    _p(out))
    if rc:
        raise ValueError("orc_dequantize_block failed (%d)" % rc)
    return out.view(np.float16)


def demote_block(src: Page, dst_bits: int) -> Page:
    _, cb, _, _ = page_bytes(src.rows, src.cols, dst_bits, src.group)
    codes = np.zeros(cb, np.uint8)
    ng = src.cols // src.group
    scales = np.zeros((src.rows, ng), np.uint16)
    zps = np.zeros((src.rows, ng), np.uint16)
    rc = lib().orc_demote_block(_p(src.codes), _p(src.scales), _p(src.zps), src.rows, src.cols, src.bits, dst_bits,
                                src.group, _p(codes), _p(scales), _p(zps))
    if rc:
        raise ValueError("orc_demote_block failed (%d)" % rc)
    return Page(codes, scales, zps, src.rows, src.cols, dst_bits, src.group)


def unpack_codes(pg: Page) -> np.ndarray:
    """Codes of a sub-16-bit page as a uint8 [rows, cols] array (reads the canonical bit stream)."""
    assert pg.bits < 16
    bits = np.unpackbits(pg.codes, bitorder="little").reshape(pg.rows * pg.cols, pg.bits)
    weights = (1 << np.arange(pg.bits)).astype(np.uint8)
    return (bits * weights).sum(axis=1).astype(np.uint8).reshape(pg.rows, pg.cols)


def router(logits: np.ndarray, k: int):
    logits = np.ascontiguousarray(logits, np.float32)
    T, E = logits.shape
    ids = np.zeros((T, k), np.int32)
    gates = np.zeros((T, k), np.float32)
    rc = lib().orc_router(_p(logits), T, E, k, _p(ids), _p(gates))
    if rc:
        raise ValueError("orc_router failed (%d)" % rc)
    return ids, gates


def permute(topk_ids: np.ndarray, E: int):
    ids = np.ascontiguousarray(topk_ids, np.int32)
    T, k = ids.shape
    counts = np.zeros(E, np.int32)
    offsets = np.zeros(E + 1, np.int32)
    perm = np.zeros(T * k, np.int32)
    inv = np.zeros(T * k, np.int32)
    rc = lib().orc_permute(_p(ids), T, k, E, _p(counts), _p(offsets), _p(perm), _p(inv))
    if rc:
        raise ValueError("orc_permute failed (%d)" % rc)
    return counts, offsets, perm, inv


def _cpages(pages: Sequence[Page]):
    arr = (_CPage * len(pages))()
    for i, pg in enumerate(pages):
        arr[i].codes = pg.codes.ctypes.data
        arr[i].scales = 0 if pg.scales is None else pg.scales.ctypes.data
        arr[i].zps = 0 if pg.zps is None else pg.zps.ctypes.data
        arr[i].rows, arr[i].cols, arr[i].group, arr[i].bits = pg.rows, pg.cols, pg.group, pg.bits
    return arr


def moe_forward(hidden_fp16: np.ndarray, logits: np.ndarray, k: int, pages: Sequence[Page], n_shared: int = 0,
                tokens: Optional[Sequence[int]] = None, brute_force: bool = False) -> np.ndarray:
    """Layer output fp32 [T, H].  ``pages`` is ordered [expert][gate, up, down], shared experts last.

    ``tokens`` restricts the computation to those output rows (the others come back as NaN).
    """
    hid = _as_u16(hidden_fp16)
    logits = np.ascontiguousarray(logits, np.float32)
    T, H = hid.shape
    E = logits.shape[1]
    assert len(pages) == (E + n_shared) * 3
    F = pages[0].rows
    out = np.full((T, H), np.nan, np.float32)
    arr = _cpages(pages)
    if brute_force:
        assert tokens is None
        rc = lib().orc_moe_forward_bruteforce(_p(hid), _p(logits), T, E, n_shared, k, H, F, arr, _p(out))
    else:
        mask = None
        if tokens is not None:
            mask = np.zeros(T, np.uint8)
            mask[np.asarray(tokens, np.int64)] = 1
        rc = lib().orc_moe_forward(_p(hid), _p(logits), T, E, n_shared, k, H, F, arr, _p(mask), _p(out))
    if rc:
        raise ValueError("orc_moe_forward failed (%d)" % rc)
    return out


def num_threads() -> int:
    return int(lib().orc_num_threads())
