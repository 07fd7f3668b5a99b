"""Pins of the bit-plane oracle (oracle/planes.py) against what the format's definition fixes: the full-plane
view is the plain 4-bit page, fewer planes give the leading bits of the same code, the lookup table of a
lower precision is the midpoint of the levels it merges (closed form on a ramp), the error bound of each
view, the size table of Eq. 3, and detaching / re-attaching planes touches no value."""
import numpy as np
import pytest

from paper_2607_16184_b200 import synth


@pytest.fixture(scope="module")
def pl():
    from oracle import planes
    return planes


def block(rows=128, cols=512, seed=3):
    g = np.random.default_rng(seed)
    w = g.normal(0, 0.02, (rows, cols)).astype(np.float32)
    w = np.where(g.random((rows, cols)) < 0.001, w * 10, w)
    return w.astype(np.float16)


def f16(u):
    return u.view(np.float16).astype(np.float64)


def test_all_planes_are_the_plain_four_bit_page(orc, pl):
    w = block()
    b = pl.quantize_planes(w)
    v4, ref = pl.view(b, 4), orc.quantize_block(w, 4)
    assert np.array_equal(v4.codes, ref.codes) and np.array_equal(v4.scales, ref.scales) and np.array_equal(v4.zps, ref.zps)


@pytest.mark.parametrize("q", [3, 2])
def test_fewer_planes_are_the_leading_bits(orc, pl, q):
    b = pl.quantize_planes(block(seed=q))
    c4 = orc.unpack_codes(pl.view(b, 4))
    cq = orc.unpack_codes(pl.view(b, q))
    assert np.array_equal(cq, c4 >> (4 - q))
    assert cq.max() <= (1 << q) - 1


def test_ramp_group_closed_form(orc, pl):
    # w_i = (i mod 16) / 64 - 1/8: 4-bit scale 2^-6, zero-point -1/8, code i mod 16 (exact)
    w = np.tile(((np.arange(128) % 16) * 2.0 ** -6 - 0.125).astype(np.float16), (128, 1))
    b = pl.quantize_planes(w)
    s3, z3 = b.lut[3]
    s2, z2 = b.lut[2]
    assert np.all(f16(s3) == 2.0 ** -5) and np.all(f16(z3) == -0.125 + 2.0 ** -7)
    assert np.all(f16(s2) == 2.0 ** -4) and np.all(f16(z2) == -0.125 + 1.5 * 2.0 ** -6)
    d3 = orc.dequantize_block(pl.view(b, 3)).astype(np.float64)
    d2 = orc.dequantize_block(pl.view(b, 2)).astype(np.float64)
    i = np.arange(128) % 16
    # the value of a merged level is the mean of the levels it merges
    assert np.array_equal(d3[0], ((i >> 1) * 2 + 0.5) * 2.0 ** -6 - 0.125)
    assert np.array_equal(d2[0], ((i >> 2) * 4 + 1.5) * 2.0 ** -6 - 0.125)


@pytest.mark.parametrize("q", [4, 3, 2])
def test_error_bound_of_each_view(orc, pl, q):
    w = block(256, 256, seed=11)
    b = pl.quantize_planes(w)
    d = orc.dequantize_block(pl.view(b, q)).astype(np.float64)
    sq = np.repeat(f16(b.lut[q][0]), 128, axis=1)
    zq = np.repeat(np.abs(f16(b.lut[q][1])), 128, axis=1)
    # |w - D_q| <= s_q / 2: half a 4-bit step from the master code plus the width of the merged levels;
    # slack for the two fp16 roundings on the way (the zero-point of the table, the table entry)
    err = np.abs(w.astype(np.float64) - d)
    assert np.all(err <= sq / 2 * (1 + 1e-6) + (zq + np.abs(d)) * 2.0 ** -11 + 1e-12)


@pytest.mark.parametrize("q", [3, 2])
def test_table_is_the_midpoint_of_merged_levels(orc, pl, q):
    b = pl.quantize_planes(block(128, 256, seed=5))
    s4, z4 = f16(b.lut[4][0]), f16(b.lut[4][1])
    sq, zq = f16(b.lut[q][0]), f16(b.lut[q][1])
    n = 1 << (4 - q)
    for c in range(1 << q):
        children = np.mean([z4 + (c * n + j) * s4 for j in range(n)], axis=0)
        entry = zq + c * sq
        assert np.all(np.abs(entry - children) <= np.abs(zq) * 2.0 ** -11 + 1e-9)       # one fp16 rounding of z_q


def test_size_table_matches_eq3(orc, pl):
    for q in (4, 3, 2):
        assert pl.plane_bytes(14336, 4096, q) == orc.page_bytes(14336, 4096, q)[0]
    # released bytes of dropping planes are positive and additive
    d43 = pl.plane_bytes(1408, 2048, 4) - pl.plane_bytes(1408, 2048, 3)
    d32 = pl.plane_bytes(1408, 2048, 3) - pl.plane_bytes(1408, 2048, 2)
    assert d43 == d32 == 1408 * 2048 // 8


def test_detach_and_attach_touch_no_value(orc, pl):
    b = pl.quantize_planes(block(seed=9))
    before = [x.copy() for x in (b.top, b.bit1, b.bit0)]
    low = pl.detach(b, 2)
    with pytest.raises(AssertionError):
        pl.view(low, 3)                                    # a detached plane cannot be read
    v2 = pl.view(low, 2)
    back = pl.attach(low, 4)
    assert all(np.array_equal(a, c) for a, c in zip(before, (back.top, back.bit1, back.bit0)))
    assert np.array_equal(pl.view(back, 4).codes, pl.view(b, 4).codes)
    assert np.array_equal(v2.codes, pl.view(b, 2).codes)


def test_forward_on_views_matches_dense_numpy(orc, pl):
    cfg = synth.LayerConfig("planes_tiny", 2, 1, 128, 256, 5)
    rng = np.random.default_rng(0)
    pages, dense = [], []
    for e in range(2):
        for u, q in zip(range(3), (4, 3, 2)):
            rows, cols = cfg.block_shape(u)
            w = (rng.normal(0, 0.05, (rows, cols))).astype(np.float16)
            b = pl.quantize_planes(w)
            pg = pl.view(b, q)
            pages.append(pg)
            c = orc.unpack_codes(pg).astype(np.float64)
            s = np.repeat(f16(pg.scales), 128, axis=1)
            z = np.repeat(f16(pg.zps), 128, axis=1)
            dense.append((c * s + z).astype(np.float16).astype(np.float64))   # LUT_q[c], restated
    x = rng.normal(0, 1, (5, 128)).astype(np.float16)
    logits = rng.normal(0, 1, (5, 2)).astype(np.float32)
    out = orc.moe_forward(x, logits, 1, pages)
    ids = np.argmax(logits, axis=1)
    for t in range(5):
        wg, wu, wd = dense[ids[t] * 3: ids[t] * 3 + 3]
        g = wg @ x[t].astype(np.float64)
        u = wu @ x[t].astype(np.float64)
        h = (g / (1 + np.exp(-g))) * u
        assert np.allclose(out[t], wd @ h, rtol=2e-5, atol=1e-6)
