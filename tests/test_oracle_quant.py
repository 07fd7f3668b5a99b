"""Pins of the oracle's quantizer, dequantizer, demote and packed layout (CPU only).

Each check compares the oracle with something that is not the oracle: numpy's own
fp16 conversion, closed forms worked by hand, error bounds, integer identities.
"""
import os

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def synth_w(rows, cols, seed=0):
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((rows, cols)) * 0.02
    w = np.where(rng.random((rows, cols)) < 0.001, w * 10, w)
    return w.astype(np.float16)


def test_half_to_float_exhaustive(orc):
    L = orc.lib()
    allh = np.arange(65536, dtype=np.uint16)
    ref = allh.view(np.float16).astype(np.float32)
    got = np.array([L.orc_f16_to_f32(int(h)) for h in allh], np.float32)
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin].view(np.uint32), ref[fin].view(np.uint32))
    assert np.all(np.isnan(got[np.isnan(ref)]))
    assert np.array_equal(got[np.isinf(ref)], ref[np.isinf(ref)])


def test_float_to_half_matches_numpy_rne(orc):
    L = orc.lib()
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(40000) * 10.0 ** rng.integers(-9, 6, 40000)).astype(np.float32)
    # exact ties, subnormal boundaries, overflow boundary
    extra = np.array([0.0, -0.0, 2.0 ** -25, 2.0 ** -25 * 1.0000001, 2.0 ** -24, 3 * 2.0 ** -25, 65504.0, 65519.99,
                      65520.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2.0 ** -14, 2.0 ** -14 - 2.0 ** -25,
                      1e-10, -1e-10, 7e4, -7e4], np.float32)
    x = np.concatenate([x, extra, -extra])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = np.array([L.orc_f32_to_f16(float(v)) for v in x], np.uint16)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("bits", [16, 8, 4, 3, 2])
def test_page_bytes_golden_and_closed_form(orc, bits):
    rows_seen = 0
    for line in open(os.path.join(GOLD, "page_bytes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        r, c, b, nbytes = map(int, line.split())
        if b != bits:
            continue
        rows_seen += 1
        tot, cb, sb, zb = orc.page_bytes(r, c, b)
        assert tot == nbytes
        assert tot == cb + sb + zb
    assert rows_seen == 1
    # released bytes of a demotion are positive (Eq. 3)
    sizes = [orc.page_bytes(512, 1024, b)[0] for b in (16, 8, 4, 3, 2)]
    assert all(sizes[i] - sizes[i + 1] > 0 for i in range(4))
    with pytest.raises(ValueError):
        orc.page_bytes(4, 100, 4)      # cols not a multiple of the group
    with pytest.raises(ValueError):
        orc.page_bytes(4, 128, 5)      # unsupported bitwidth


def test_sixteen_bit_page_round_trips(orc):
    w = synth_w(8, 256)
    pg = orc.quantize_block(w, 16)
    assert pg.scales is None and pg.zps is None
    assert np.array_equal(pg.codes.view(np.uint16).reshape(8, 256), w.view(np.uint16))
    assert np.array_equal(orc.dequantize_block(pg).view(np.uint16), w.view(np.uint16))


def test_ramp_group_closed_form(orc):
    # w_i = (i mod 16) * 2^-6 - 0.125 at 4 bits: range 15/64, scale 2^-6, zp -0.125, code_i = i mod 16
    i = np.arange(128)
    w = ((i % 16) * 2.0 ** -6 - 0.125).astype(np.float16)[None, :]
    pg = orc.quantize_block(w, 4)
    assert pg.scales.view(np.float16)[0, 0] == np.float16(2.0 ** -6)
    assert pg.zps.view(np.float16)[0, 0] == np.float16(-0.125)
    assert np.array_equal(orc.unpack_codes(pg)[0], (i % 16).astype(np.uint8))
    assert np.array_equal(orc.dequantize_block(pg), w)


@pytest.mark.parametrize("bits", [8, 4, 3, 2])
def test_constant_two_level_and_negative_zero_groups(orc, bits):
    L = 2 ** bits - 1
    const = np.full((1, 128), 0.3125, np.float16)
    pg = orc.quantize_block(const, bits)
    assert pg.scales.view(np.float16)[0, 0] == np.float16(1.0)
    assert pg.zps.view(np.float16)[0, 0] == np.float16(0.3125)
    assert not orc.unpack_codes(pg).any()
    assert np.array_equal(orc.dequantize_block(pg), const)
    two = np.where(np.arange(128) % 3 == 0, -0.5, 0.25).astype(np.float16)[None, :]
    pg = orc.quantize_block(two, bits)
    codes = orc.unpack_codes(pg)[0]
    assert set(codes.tolist()) == {0, L}
    assert np.array_equal(codes == L, two[0] == np.float16(0.25))
    nz = np.zeros((1, 128), np.float16)
    nz[0, ::2] = -0.0
    nz[0, 5] = 0.5
    pg = orc.quantize_block(nz, bits)
    assert pg.zps[0, 0] == 0x0000            # minimum of -0 / +0 is stored as +0
    # a group of only negative zeros: zero range, scale 1, zero-point +0
    pg = orc.quantize_block(np.full((1, 128), -0.0, np.float16), bits)
    assert pg.zps[0, 0] == 0x0000 and pg.scales.view(np.float16)[0, 0] == np.float16(1.0)


def test_tiny_range_scale_is_clamped_to_smallest_subnormal(orc):
    w = np.zeros((1, 128), np.float16)
    w[0, 7] = np.float16(2.0 ** -24)         # range 2^-24; /255 underflows to zero in fp16
    pg = orc.quantize_block(w, 8)
    assert pg.scales[0, 0] == 0x0001
    codes = orc.unpack_codes(pg)[0]
    assert codes[7] == 1 and codes.sum() == 1
    assert np.array_equal(orc.dequantize_block(pg), w)


@pytest.mark.parametrize("bits", [8, 4, 3, 2])
def test_quantize_invariants(orc, bits):
    L = 2 ** bits - 1
    w = synth_w(64, 1024, seed=bits)
    pg = orc.quantize_block(w, bits)
    codes = orc.unpack_codes(pg).reshape(64, 8, 128)
    assert codes.max() <= L
    assert (codes.min(axis=2) == 0).all()              # the minimum always maps to code 0
    assert (codes.max(axis=2) == L).all()              # the maximum maps to L whenever the range is non-zero
    s = pg.scales.view(np.float16).astype(np.float64)
    z = pg.zps.view(np.float16).astype(np.float64)
    wg = w.astype(np.float64).reshape(64, 8, 128)
    assert np.array_equal(z, wg.min(axis=2))           # zero-point is the group minimum, stored exactly
    # fp16(range / L), written with numpy's own fp32 divide and fp16 rounding
    rng32 = (wg.max(axis=2) - wg.min(axis=2)).astype(np.float32)
    assert np.array_equal(pg.scales.view(np.float16), (rng32 / np.float32(L)).astype(np.float16))
    recon = z[:, :, None] + codes.astype(np.float64) * s[:, :, None]
    ratio = np.abs(wg - recon) / s[:, :, None]
    assert ratio.max() <= 0.5 * (1 + 1e-6)             # error <= scale / 2 on the unrounded decode
    # nearest-code property, stated independently: no other code is strictly closer
    for dc in (-1, 1):
        other = np.clip(codes.astype(np.int64) + dc, 0, L)
        alt = np.abs(wg - (z[:, :, None] + other * s[:, :, None]))
        assert (np.abs(wg - recon) <= alt * (1 + 1e-3) + 1e-12).all()


@pytest.mark.parametrize("bits", [8, 4, 3, 2])
def test_canonical_bit_stream_layout(orc, bits):
    w = synth_w(4, 256, seed=11)
    pg = orc.quantize_block(w, bits)
    codes = orc.unpack_codes(pg).reshape(-1).astype(object)
    # the whole page as one little-endian integer: code n occupies bits [n*b, (n+1)*b)
    big = int.from_bytes(pg.codes.tobytes(), "little")
    for n in (0, 1, 2, 7, 127, 128, 129, 255, 256, 1023):
        assert (big >> (n * bits)) & (2 ** bits - 1) == codes[n]
    assert pg.codes.size == 4 * 256 * bits // 8
    if bits == 8:
        assert np.array_equal(pg.codes, np.asarray(codes, np.uint8))
    if bits == 4:
        c = np.asarray(codes, np.uint8)
        assert np.array_equal(pg.codes, c[0::2] | (c[1::2] << 4))


def test_three_bit_stream_worked_example(orc):
    # eight 3-bit codes 1,2,3,4,5,6,7,0 form the 24-bit integer sum(c_i << 3i) = 0x1F58D1 -> bytes D1 58 1F
    assert sum(c << (3 * i) for i, c in enumerate([1, 2, 3, 4, 5, 6, 7, 0])) == 0x1F58D1
    w = np.zeros((1, 128), np.float16)
    w[0, :8] = np.array([1, 2, 3, 4, 5, 6, 7, 0], np.float16)      # range 7, scale 1, zp 0 -> code = value
    pg = orc.quantize_block(w, 3)
    assert pg.scales.view(np.float16)[0, 0] == 1.0 and pg.zps[0, 0] == 0
    assert pg.codes[:3].tolist() == [0xD1, 0x58, 0x1F]
    assert not pg.codes[3:].any()


@pytest.mark.parametrize("bits", [8, 4, 3, 2])
def test_dequantize_formula_numpy(orc, bits):
    w = synth_w(16, 512, seed=5)
    pg = orc.quantize_block(w, bits)
    c = orc.unpack_codes(pg).astype(np.float32)
    s = pg.scales.view(np.float16).astype(np.float32).repeat(128, axis=1)
    z = pg.zps.view(np.float16).astype(np.float32).repeat(128, axis=1)
    ref = (c * s + z).astype(np.float16)               # fp32 product (exact) + fp32 add, then one fp16 rounding
    assert np.array_equal(orc.dequantize_block(pg).view(np.uint16), ref.view(np.uint16))


@pytest.mark.parametrize("src,dst", [(16, 8), (16, 4), (16, 3), (16, 2)])
def test_demote_from_16_is_quantize(orc, src, dst):
    w = synth_w(8, 512, seed=2)
    a = orc.demote_block(orc.quantize_block(w, 16), dst)
    b = orc.quantize_block(w, dst)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales) and np.array_equal(a.zps, b.zps)


@pytest.mark.parametrize("src,dst", [(8, 4), (8, 3), (8, 2), (4, 3), (4, 2), (3, 2)])
def test_demote_chain_properties(orc, src, dst):
    w = synth_w(32, 1024, seed=src * 10 + dst)
    p_src = orc.quantize_block(w, src)
    before = (p_src.codes.copy(), p_src.scales.copy(), p_src.zps.copy())
    p_dst = orc.demote_block(p_src, dst)
    assert np.array_equal(before[0], p_src.codes) and np.array_equal(before[1], p_src.scales)   # source untouched
    assert np.array_equal(p_dst.zps, p_src.zps)        # code 0 decodes to zp exactly, so the minimum survives
    Ls, Ld = 2 ** src - 1, 2 ** dst - 1
    s_src = p_src.scales.view(np.float16).astype(np.float32)
    z = p_src.zps.view(np.float16).astype(np.float32)
    top = (np.float32(Ls) * s_src + z).astype(np.float16).astype(np.float32)       # D(L_src)
    assert np.array_equal(p_dst.scales.view(np.float16), ((top - z) / np.float32(Ld)).astype(np.float16))
    deq = orc.dequantize_block(p_src).astype(np.float64)
    s = p_dst.scales.view(np.float16).astype(np.float64).repeat(128, axis=1)
    recon = p_dst.zps.view(np.float16).astype(np.float64).repeat(128, axis=1) + orc.unpack_codes(p_dst) * s
    assert (np.abs(deq - recon) / s).max() <= 0.5 * (1 + 1e-6)
    if Ls % Ld == 0:                                   # integer map code' = rne(code * Ld / Ls)
        c = orc.unpack_codes(p_src).astype(np.int64)
        q = Ls // Ld
        mapped = (c + q // 2) // q                     # q is odd (5, 17, 85), so there are no ties
        assert q % 2 == 1
        assert np.array_equal(orc.unpack_codes(p_dst), mapped.astype(np.uint8))


def test_chain_differs_from_direct(orc):
    w = synth_w(64, 1024, seed=9)
    chain = orc.demote_block(orc.demote_block(orc.quantize_block(w, 16), 4), 2)
    direct = orc.quantize_block(w, 2)
    assert not np.array_equal(chain.scales, direct.scales)         # 16->4->2 is not 16->2


def test_demote_rejects_non_lowering(orc):
    pg = orc.quantize_block(synth_w(2, 128), 4)
    with pytest.raises(ValueError):
        orc.demote_block(pg, 4)
    with pytest.raises(ValueError):
        orc.demote_block(pg, 8)
