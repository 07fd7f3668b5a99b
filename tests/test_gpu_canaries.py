"""Guard regions around every buffer the library writes: page buffers of quantize / demote / export / the plane
quantizer, the output of a forward call, and the workspace.  Each guard is filled with a known pattern before
the call and must still hold it afterwards; the buffer itself must have been written in full where that can be
told.  (The stand-in for a memory checker on the kernels' stores.)"""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, make_ctx

pytestmark = pytest.mark.gpu

GUARD = 8192            # bytes on each side
PATTERN = 0xA5


def guarded(nbytes):
    """(buffer with guards, view of the nbytes in the middle); the view starts on a 256-byte boundary."""
    big = torch.full((GUARD + nbytes + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
    assert big.data_ptr() % 256 == 0
    return big, big[GUARD:GUARD + nbytes]


def guards_intact(big, nbytes):
    return bool((big[:GUARD] == PATTERN).all().item()) and bool((big[GUARD + nbytes:] == PATTERN).all().item())


def guarded_page(rows, cols, bits, layout=B.PW_LAYOUT_TILED):
    pg = B.Page(rows, cols, bits, "cuda", layout)
    keep = []
    for name in ("codes", "scales", "zps"):
        t = getattr(pg, name)
        if t is None:
            continue
        nbytes = t.numel() * t.element_size()
        big, mid = guarded(nbytes)
        view = mid.view(t.dtype)
        setattr(pg, name, view)
        setattr(pg.c, name, view.data_ptr())
        keep.append((big, nbytes))
    return pg, keep


def test_the_guard_check_sees_a_stray_byte():
    big, mid = guarded(1024)
    assert guards_intact(big, 1024)
    big[GUARD + 1024] = 0                       # one byte past the end
    assert not guards_intact(big, 1024)
    big[GUARD + 1024] = PATTERN
    big[GUARD - 1] = 0                          # one byte before the start
    assert not guards_intact(big, 1024)
    c = B.Context(1, 8, 0, 256, 512, 16, 2, guard_bytes=GUARD)
    try:
        assert c.workspace_guards_intact()
        off, nbytes = c._ws_span
        c.workspace[off + nbytes] = 0
        assert not c.workspace_guards_intact()
    finally:
        c.close()


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(1, 8, 0, 256, 512, 160, 2, guard_bytes=GUARD)
    yield c
    assert c.workspace_guards_intact()
    c.close()


@pytest.mark.parametrize("shape", [(128, 128), (384, 640)])
def test_quantize_demote_and_export_stay_inside_their_pages(ctx, shape):
    g = torch.Generator().manual_seed(11)
    w = (torch.randn(*shape, generator=g) * 0.02).to(torch.float16).cuda()
    pages = {}
    for bits in (16, 8, 4, 3, 2):
        pg, keep = guarded_page(shape[0], shape[1], bits)
        ctx.pw_quantize_block(w, bits, dst=pg)
        torch.cuda.synchronize()
        assert all(guards_intact(b, n) for b, n in keep), ("quantize", bits)
        pages[bits] = (pg, keep)
    for src in (16, 8, 4, 3):
        for dst in (8, 4, 3, 2):
            if dst >= src:
                continue
            pg, keep = guarded_page(shape[0], shape[1], dst)
            ctx.pw_demote_block(pages[src][0], dst, dst=pg)
            torch.cuda.synchronize()
            assert all(guards_intact(b, n) for b, n in keep), ("demote", src, dst)
            assert all(guards_intact(b, n) for b, n in pages[src][1]), ("demote source", src, dst)
    for bits in (8, 4, 3, 2):
        dst, keep = guarded_page(shape[0], shape[1], bits, B.PW_LAYOUT_CANONICAL)
        B._check(ctx.L.pw_export_page(ctx.handle, B.C.byref(pages[bits][0].c), B.C.byref(dst.c), None), "pw_export_page")
        torch.cuda.synchronize()
        assert all(guards_intact(b, n) for b, n in keep), ("export", bits)
    assert ctx.workspace_guards_intact()


def test_plane_quantizer_stays_inside_its_three_buffers(ctx):
    rows, cols = 256, 384
    g = torch.Generator().manual_seed(12)
    w = (torch.randn(rows, cols, generator=g) * 0.02).to(torch.float16).cuda()
    _, tb, bb = B.pw_plane_bytes(rows, cols)
    bufs = [guarded(n) for n in (tb, bb, bb)]
    dst = B.PlanePage(rows, cols, "cuda", _buffers=tuple(mid for _, mid in bufs))
    B._check(ctx.L.pw_quantize_planes(ctx.handle, w.data_ptr(), rows, cols, B.C.byref(dst.c), None), "pw_quantize_planes")
    torch.cuda.synchronize()
    for (big, _), n in zip(bufs, (tb, bb, bb)):
        assert guards_intact(big, n)
    assert ctx.workspace_guards_intact()


@pytest.mark.parametrize("mode", [B.PW_MODE_SIMT, B.PW_MODE_TENSOR])
@pytest.mark.parametrize("T", [1, 17, 64, 130, 160])
def test_forward_writes_every_output_row_and_nothing_else(ctx, T, mode):
    cfg = synth.CONFIGS["tiny_cover"]
    build_layer(ctx, cfg, 0, None)
    x = synth.activations(cfg, device="cuda", tokens=T)
    logits = synth.router_logits(cfg, device="cuda", tokens=T)
    nbytes = T * cfg.hidden * 4
    big, mid = guarded(nbytes)
    mid.fill_(PATTERN)                                    # a float of 0xA5A5A5A5 is about -2.9e-16: never a result here
    out = mid.view(torch.float32).view(T, cfg.hidden)
    ctx.pw_moe_forward(0, x, logits, cfg.top_k, out=out, mode=mode)
    torch.cuda.synchronize()
    assert ctx.pw_last_device_status() == 0
    assert guards_intact(big, nbytes)
    assert not bool((out.view(torch.int32) == torch.tensor(-0x5A5A5A5B, dtype=torch.int32, device="cuda")).any().item())
    assert ctx.workspace_guards_intact()


def test_forward_of_a_larger_layer_stays_inside_the_workspace():
    """Many experts, shared experts, several token tiles and a K split: every region of the workspace in use."""
    cfg = synth.LayerConfig("canary_fg", 32, 4, 256, 384, 200, n_shared=2, routing="zipf", zipf_a=1.2,
                            bit_rule="int4_10fp16_20int2")
    c = B.Context(1, cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.ffn, cfg.tokens, cfg.top_k, guard_bytes=GUARD)
    try:
        build_layer(c, cfg, 0, None)
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        for mode in (B.PW_MODE_TENSOR, B.PW_MODE_SIMT):
            for _ in range(3):
                c.pw_moe_forward(0, x, logits, cfg.top_k, mode=mode)
            assert c.pw_last_device_status() == 0
            assert c.workspace_guards_intact()
        c.pw_observe(True)
        c.pw_moe_forward(0, x, logits, cfg.top_k)
        assert c.workspace_guards_intact()
        c.pw_observe(False)
    finally:
        c.close()
