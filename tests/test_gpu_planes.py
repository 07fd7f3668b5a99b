"""GPU parity of the overlaid bit-plane page format: the nested quantizer against the oracle bit for bit (every
view: codes, lookup-table scales and zero-points), forward calls that read only the first q planes against the
oracle on the same views, and lowering / raising the precision without any kernel (the plane buffers stay
byte-identical, the forward follows the published bitwidth)."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import error_metrics, make_ctx, pages_equal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pl():
    from oracle import planes
    return planes


def export_view(ctx, page, orc):
    ex = ctx.pw_export_planes(page)
    torch.cuda.synchronize()
    ng = page.cols // B.GROUP
    return orc.Page(ex.codes.cpu().numpy(),
                    ex.scales.view(torch.int16).cpu().numpy().view(np.uint16).reshape(page.rows, ng),
                    ex.zps.view(torch.int16).cpu().numpy().view(np.uint16).reshape(page.rows, ng),
                    page.rows, page.cols, page.bits)


@pytest.mark.parametrize("shape", [(128, 128), (256, 512), (1408, 2048)])
def test_nested_quantizer_matches_oracle_at_every_bitwidth(orc, pl, shape):
    ctx = make_ctx(synth.CONFIGS["tiny"])
    try:
        g = torch.Generator().manual_seed(shape[0] + 1)
        w = torch.randn(*shape, generator=g) * 0.02
        w = torch.where(torch.rand(*shape, generator=g) < 0.001, w * 10, w).to(torch.float16)
        w[0, :128] = 0.25                                  # constant group
        w[1, :128] = 0.0
        w[1, 5] = 2.0 ** -24                               # scale underflows
        blk = ctx.pw_quantize_planes(w.cuda())
        ref = pl.quantize_planes(w.numpy())
        for q in (4, 3, 2):
            assert pages_equal(export_view(ctx, blk.at(q), orc), pl.view(ref, q)), q
        # the full view is the page the plain 4-bit quantizer builds
        plain = ctx.pw_export_page(ctx.pw_quantize_block(w.cuda(), 4))
        torch.cuda.synchronize()
        assert np.array_equal(plain.codes.cpu().numpy(), pl.view(ref, 4).codes)
    finally:
        ctx.close()


def build_plane_layer(ctx, cfg, pl, qs):
    """Every routed block as a bit-plane block read at qs[e, u]; returns (blocks, oracle views)."""
    blocks, views, entries = [], [], []
    for e in range(cfg.n_experts):
        for u in range(3):
            w = synth.block_weights(cfg, 0, e, u, device="cuda")
            blk = ctx.pw_quantize_planes(w)
            page = blk.at(int(qs[e, u]), detach=True)
            blocks.append(blk)
            views.append(pl.view(pl.quantize_planes(w.cpu().numpy()), int(qs[e, u])))
            entries.append((0, e, u, page))
    ctx.pw_set_page_table(entries)
    return blocks, views


@pytest.mark.parametrize("tokens", [16, 3, 70])
def test_forward_reads_the_first_q_planes(orc, pl, tokens):
    cfg = synth.LayerConfig("planes_fw", 8, 2, 256, 512, tokens, routing="normal")
    ctx = make_ctx(cfg)
    try:
        qs = np.array([[4, 3, 2], [3, 2, 4], [2, 4, 3], [4, 4, 4], [3, 3, 3], [2, 2, 2], [4, 2, 3], [2, 3, 4]])
        _, views = build_plane_layer(ctx, cfg, pl, qs)
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        out = ctx.pw_moe_forward(0, x, logits, cfg.top_k).cpu().numpy()
        assert ctx.pw_last_device_status() == 0
        ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, views)
        max_abs, rel_f = error_metrics(out, ref)
        assert max_abs <= 2e-2 and rel_f <= 5e-3, (max_abs, rel_f)
    finally:
        ctx.close()


def test_planes_next_to_ordinary_pages(orc, pl):
    # gate as bit-planes, up as an ordinary TILED page (16 / 8 / 4 bits), down as bit-planes
    cfg = synth.LayerConfig("planes_mix", 4, 2, 512, 1024, 40, routing="zipf", zipf_a=1.1)
    ctx = make_ctx(cfg)
    try:
        entries, views, keep = [], [], []
        for e in range(cfg.n_experts):
            for u in range(3):
                w = synth.block_weights(cfg, 0, e, u, device="cuda")
                if u == 1:
                    b = (16, 8, 4, 2)[e]
                    pg = ctx.pw_quantize_block(w, b)
                    views.append(orc.quantize_block(w.cpu().numpy(), b))
                else:
                    q = (4, 3, 2, 3)[e] if u == 0 else (2, 4, 3, 4)[e]
                    blk = ctx.pw_quantize_planes(w)
                    pg = blk.at(q)
                    views.append(pl.view(pl.quantize_planes(w.cpu().numpy()), q))
                keep.append(pg)
                entries.append((0, e, u, pg))
        ctx.pw_set_page_table(entries)
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        out = ctx.pw_moe_forward(0, x, logits, cfg.top_k).cpu().numpy()
        assert ctx.pw_last_device_status() == 0
        ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, views)
        max_abs, rel_f = error_metrics(out, ref)
        assert max_abs <= 2e-2 and rel_f <= 5e-3, (max_abs, rel_f)
    finally:
        ctx.close()


def test_lowering_and_raising_the_precision_runs_no_kernel(orc, pl):
    cfg = synth.LayerConfig("planes_move", 4, 2, 256, 512, 24, routing="normal")
    ctx = make_ctx(cfg)
    try:
        blocks, _ = build_plane_layer(ctx, cfg, pl, np.full((4, 3), 4))
        refs = [pl.quantize_planes(synth.block_weights(cfg, 0, e, u, device="cuda").cpu().numpy())
                for e in range(4) for u in range(3)]
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        snap = [(b.top.clone(), b.bit1.clone(), b.bit0.clone()) for b in blocks]
        outs = {}
        for q in (4, 2, 3, 4):                              # lower to 2 bits, raise again plane by plane
            n0 = ctx.pw_launch_count()
            ctx.pw_set_page_table([(0, e, u, blocks[e * 3 + u].at(q, detach=True)) for e in range(4) for u in range(3)])
            assert ctx.pw_launch_count() - n0 == 1          # the commit itself; no page is rewritten
            assert ctx.pw_query_row(0, 1, 2).page.bits == q
            out = ctx.pw_moe_forward(0, x, logits, cfg.top_k)
            ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, [pl.view(r, q) for r in refs])
            max_abs, rel_f = error_metrics(out.cpu().numpy(), ref)
            assert max_abs <= 2e-2 and rel_f <= 5e-3, (q, max_abs, rel_f)
            if q in outs:
                assert torch.equal(out, outs[q])            # back at 4 bits: the bits of the first call
            outs[q] = out.clone()
        for b, (t, b1, b0) in zip(blocks, snap):
            assert torch.equal(b.top, t) and torch.equal(b.bit1, b1) and torch.equal(b.bit0, b0)
        assert not torch.equal(outs[2], outs[4])
    finally:
        ctx.close()


def test_plane_page_argument_errors():
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg)
    try:
        w = synth.block_weights(cfg, 0, 0, 0, device="cuda")
        blk = ctx.pw_quantize_planes(w)
        low = blk.at(2, detach=True)
        low.c.bits = 3                                      # asks for a plane the header no longer names
        with pytest.raises(B.PwError) as e:
            ctx.pw_set_page_table([(0, 0, 0, low)])
        assert e.value.status == 5
        bad = blk.at(4)
        bad.c.bits = 8
        with pytest.raises(B.PwError) as e:
            ctx.pw_set_page_table([(0, 0, 0, bad)])
        assert e.value.status == 3
    finally:
        ctx.close()
