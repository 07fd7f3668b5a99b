"""GPU parity of pw_quantize_block / pw_demote_block / pw_export_page / pw_import_page (bit-exact)."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import export_to_oracle, import_from_oracle, make_ctx, pages_equal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = make_ctx(synth.CONFIGS["tiny"])
    yield c
    c.close()


def special_block(rows=128, cols=512):
    """fp16 block with the degenerate groups of the quantizer next to ordinary ones."""
    g = torch.Generator().manual_seed(5)
    w = (torch.randn(rows, cols, generator=g) * 0.02).to(torch.float16)
    w[0, :128] = 0.3125                                   # constant group
    w[1, :128] = torch.where(torch.arange(128) % 3 == 0, -0.5, 0.25).to(torch.float16)   # two levels
    w[2, :128] = 0.0
    w[2, 0:128:2] = -0.0                                  # negative zeros, zero range
    w[3, :128] = 0.0
    w[3, 7] = 2.0 ** -24                                  # scale underflows to the smallest subnormal
    w[4, :128] = ((torch.arange(128) % 16) * 2.0 ** -6 - 0.125).to(torch.float16)         # exact ramp
    w[5, :128] = torch.linspace(-3.0, 5.0, 128).to(torch.float16)                          # many rounding ties
    w[6, 128:256] = -0.0
    w[6, 130] = 0.5                                       # minimum is -0
    w[7, :128] = 65504.0
    w[7, 1] = -65504.0                                    # range overflows fp16 but not fp32
    return w


@pytest.mark.parametrize("bits", [16, 8, 4, 3, 2])
@pytest.mark.parametrize("shape", [(128, 128), (256, 512), (512, 256), (1408, 2048)])
def test_quantize_matches_oracle(ctx, orc, bits, shape):
    g = torch.Generator().manual_seed(bits * 7 + shape[0])
    w = torch.randn(*shape, generator=g) * 0.02
    w = torch.where(torch.rand(*shape, generator=g) < 0.001, w * 10, w).to(torch.float16)
    pg = ctx.pw_quantize_block(w.cuda(), bits)
    assert pg.layout == B.PW_LAYOUT_TILED and pg.bits == bits
    got = export_to_oracle(ctx, pg, orc)
    ref = orc.quantize_block(w.numpy(), bits)
    assert pages_equal(got, ref)


@pytest.mark.parametrize("bits", [8, 4, 3, 2])
def test_quantize_degenerate_groups(ctx, orc, bits):
    w = special_block()
    got = export_to_oracle(ctx, ctx.pw_quantize_block(w.cuda(), bits), orc)
    ref = orc.quantize_block(w.numpy(), bits)
    assert pages_equal(got, ref)


@pytest.mark.parametrize("src,dst", [(16, 8), (16, 4), (16, 3), (16, 2), (8, 4), (8, 3), (8, 2), (4, 3), (4, 2), (3, 2)])
def test_demote_matches_oracle_and_leaves_source_alone(ctx, orc, src, dst):
    cfg = synth.CONFIGS["tiny"]
    w = synth.block_weights(cfg, 0, 3, 2)                 # 256 x 512
    w[:8] = special_block(128, 512)[:8]
    p_src = ctx.pw_quantize_block(w.cuda(), src)
    before = export_to_oracle(ctx, p_src, orc)
    p_dst = ctx.pw_demote_block(p_src, dst)
    assert p_dst.bits == dst
    got = export_to_oracle(ctx, p_dst, orc)
    ref = orc.demote_block(orc.quantize_block(w.numpy(), src), dst)
    assert pages_equal(got, ref)
    assert pages_equal(export_to_oracle(ctx, p_src, orc), before)


def test_demote_chain_16_4_2(ctx, orc):
    cfg = synth.CONFIGS["tiny"]
    w = synth.block_weights(cfg, 0, 1, 0)
    p = ctx.pw_quantize_block(w.cuda(), 16)
    p4 = ctx.pw_demote_block(p, 4)
    p2 = ctx.pw_demote_block(p4, 2)
    ref = orc.demote_block(orc.demote_block(orc.quantize_block(w.numpy(), 16), 4), 2)
    assert pages_equal(export_to_oracle(ctx, p2, orc), ref)


@pytest.mark.parametrize("dst", [3, 2])
def test_demote_from_4_bits_of_pages_that_do_not_use_their_code_range(ctx, orc, dst):
    """A 4-bit page from elsewhere (imported) need not contain code 0 and code 15 in every group: the demote then
    takes minimum and maximum from the codes that are present.  Groups of every kind side by side."""
    rows, cols = 128, 1024
    rng = np.random.default_rng(11)
    codes = rng.integers(0, 16, (rows, cols), dtype=np.uint8)
    codes[0:32, :] = rng.integers(3, 12, (32, cols))                 # neither extreme
    codes[32:64, :] = rng.integers(0, 9, (32, cols))                 # no 15 (almost surely a 0)
    codes[64:96, :] = rng.integers(5, 16, (32, cols))                # no 0
    codes[96, :128] = 7                                              # a single level
    codes[97, :128] = np.where(np.arange(128) % 2 == 0, 2, 13)       # two levels
    scales = rng.uniform(1e-3, 2e-2, (rows, cols // 128)).astype(np.float16)
    zps = rng.uniform(-0.2, 0.05, (rows, cols // 128)).astype(np.float16)
    zps[98, 0] = np.float16(-0.0)
    codes[98, :128] = rng.integers(0, 16, 128)
    codes[98, 5] = 0
    stream = np.packbits(np.unpackbits(codes.reshape(-1, 1), axis=1, bitorder="little")[:, :4].reshape(-1),
                         bitorder="little")
    ref4 = orc.Page(stream, scales.view(np.uint16).copy(), zps.view(np.uint16).copy(), rows, cols, 4)
    assert np.array_equal(orc.unpack_codes(ref4), codes)
    dev4 = import_from_oracle(ctx, ref4)
    low = ctx.pw_demote_block(dev4, dst)
    torch.cuda.synchronize()
    assert pages_equal(export_to_oracle(ctx, low, orc), orc.demote_block(ref4, dst))


@pytest.mark.parametrize("bits", [16, 8, 4, 3, 2])
def test_import_export_round_trip(ctx, orc, bits):
    cfg = synth.CONFIGS["tiny"]
    w = synth.block_weights(cfg, 0, 2, 1)
    ref = orc.quantize_block(w.numpy(), bits)
    dev = import_from_oracle(ctx, ref)
    assert dev.layout == B.PW_LAYOUT_TILED
    assert pages_equal(export_to_oracle(ctx, dev, orc), ref)
    # the imported page is byte-identical to the one the GPU quantizer builds
    own = ctx.pw_quantize_block(w.cuda(), bits)
    torch.cuda.synchronize()
    # (a TILED page is one buffer: the codes, scales and zero-points of every tile)
    assert own.scales is None and own.zps is None
    assert own.codes.numel() == B.pw_page_bytes(w.shape[0], w.shape[1], bits)[0]
    assert torch.equal(own.codes, dev.codes)


def test_argument_errors_enqueue_nothing(ctx):
    w = torch.zeros(128, 128, dtype=torch.float16, device="cuda")
    n0 = ctx.pw_launch_count()
    with pytest.raises(B.PwError) as e:
        ctx.pw_quantize_block(w, 5)
    assert e.value.status == 3
    with pytest.raises(B.PwError) as e:
        ctx.pw_quantize_block(torch.zeros(100, 128, dtype=torch.float16, device="cuda"), 4)
    assert e.value.status == 2
    pg = ctx.pw_quantize_block(w, 4)
    for bad in (4, 8, 16, 5):
        with pytest.raises(B.PwError) as e:
            ctx.pw_demote_block(pg, bad)
        assert e.value.status == 3
    mis = B.Page(128, 128, 4)
    mis.c.codes = mis.codes.data_ptr() + 8
    with pytest.raises(B.PwError) as e:
        ctx.pw_quantize_block(w, 4, dst=mis)
    assert e.value.status == 4
    can = ctx.pw_export_page(pg)
    with pytest.raises(B.PwError) as e:
        ctx.pw_demote_block(can, 2)                       # demote wants the TILED layout
    assert e.value.status == 5
    assert ctx.pw_launch_count() == n0 + 2                # only the two valid calls launched
    assert ctx.pw_last_device_status() == 0
