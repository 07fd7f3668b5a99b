"""Offload and reload of weight pages on the GPU, replayed against the life-cycle oracle: states after every
step, the two ordering rules (Sec. 3.1 / 3.3), bytes that survive the round trip bit for bit, and a forward
call that returns the same bits once the reloaded page is committed again."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, make_ctx

pytestmark = pytest.mark.gpu

STATE_ERR, ARG_ERR = 5, 1


def expect(status, fn, *a, **k):
    with pytest.raises(B.PwError) as ei:
        fn(*a, **k)
    assert ei.value.status == status


def test_offload_reload_round_trip_follows_the_oracle():
    from oracle import residency as R
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, np.full((8, 3), 16, np.int32))
        e, u = 2, B.PW_GATE
        row = (0, e, u)
        M = {b: B.pw_page_bytes(cfg.ffn, cfg.hidden, b)[0] for b in synth.BITS}
        orow = R.Row(M)
        page16 = pages[e * 3 + u]
        orow.add_gpu_page(16)
        orow.commit(16)

        def same_state(bits):
            assert ctx.pw_page_state(*row, bits) == orow.state.get(bits, R.NONE)

        x = synth.activations(cfg, device="cuda")
        lg = synth.router_logits(cfg, device="cuda")
        out_a = ctx.pw_moe_forward(0, x, lg, cfg.top_k).clone()
        same_state(16)
        same_state(4)                                               # nothing known at 4 bits yet
        expect(STATE_ERR, ctx.pw_offload_page, *row, page16)        # the committed page cannot leave
        with pytest.raises(R.IllegalTransition):
            orow.offload(16)

        # offload direction: demote, commit the lower bitwidth, then move the 16-bit page out on a side stream
        side = torch.cuda.Stream()
        page4 = ctx.pw_demote_block(page16, 4)
        ctx.pw_set_page_table([(0, e, u, page4)])
        orow.add_gpu_page(4)
        orow.commit(4)
        out_b = ctx.pw_moe_forward(0, x, lg, cfg.top_k).clone()
        image16 = page16.codes.clone()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            torch.cuda._sleep(200_000_000)                          # ~0.1 s: the copy behind it cannot have finished
            host = ctx.pw_offload_page(*row, page16, stream=side)
        orow.offload(16)
        same_state(16)                                              # IN_TRANSFER
        expect(STATE_ERR, ctx.pw_offload_page, *row, page16)
        expect(STATE_ERR, ctx.pw_reload_page, *row, 16, host)
        expect(STATE_ERR, ctx.pw_drop_page, *row, 16)
        side.synchronize()
        orow.transfer_done(16)
        same_state(16)                                              # CPU_RESIDENT
        assert torch.equal(host[: image16.numel()], image16.cpu())  # the bytes that left are the page
        assert sum(M[b] for b in synth.BITS if ctx.pw_page_state(*row, b) in (0, 2)) == orow.gpu_bytes() == M[4]
        pages[e * 3 + u] = None
        del page16                                                  # the device buffer is released
        out_b2 = ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        torch.cuda.synchronize()
        assert torch.equal(out_b, out_b2)

        # reload direction: the page comes back first, the commit follows once it is resident
        stale = B.Page(cfg.ffn, cfg.hidden, 16, ctx.device)
        expect(STATE_ERR, ctx.pw_set_page_table, [(0, e, u, stale)])      # 16 bits is CPU-resident
        expect(ARG_ERR, ctx.pw_reload_page, *row, 16, torch.empty(M[16], dtype=torch.uint8).pin_memory())
        with torch.cuda.stream(side):
            torch.cuda._sleep(200_000_000)
            back = ctx.pw_reload_page(*row, 16, host, stream=side)
        orow.reload(16)
        same_state(16)                                              # IN_TRANSFER
        expect(STATE_ERR, ctx.pw_set_page_table, [(0, e, u, back)])       # q_i is not raised yet
        with pytest.raises(R.IllegalTransition):
            orow.commit(16)
        assert ctx.pw_query_row(*row).page.bits == 4
        side.synchronize()
        orow.transfer_done(16)
        same_state(16)                                              # GPU_RESIDENT
        assert torch.equal(back.codes, image16)
        ctx.pw_set_page_table([(0, e, u, back)])
        orow.commit(16)
        out_c = ctx.pw_moe_forward(0, x, lg, cfg.top_k)
        torch.cuda.synchronize()
        assert torch.equal(out_c, out_a) and not torch.equal(out_b, out_a)
        assert ctx.pw_last_device_status() == 0

        # a page can be forgotten once the row is off it; then a new page of that bitwidth may be committed
        expect(STATE_ERR, ctx.pw_drop_page, *row, 16)
        ctx.pw_drop_page(*row, 4)
        assert ctx.pw_page_state(*row, 4) == B.PW_STATE_NONE
        ctx.pw_set_page_table([(0, e, u, ctx.pw_demote_block(back, 4))])
        assert ctx.pw_page_state(*row, 4) == B.PW_STATE_GPU_RESIDENT
    finally:
        ctx.close()


def test_argument_errors_enqueue_nothing():
    cfg = synth.CONFIGS["tiny"]
    ctx = make_ctx(cfg, n_layers=1)
    try:
        pages, _ = build_layer(ctx, cfg, 0, np.full((8, 3), 8, np.int32))
        n0 = ctx.pw_launch_count()
        wrong_shape = B.Page(cfg.hidden, cfg.ffn, 16, ctx.device)            # a down-shaped page for a gate row
        expect(2, ctx.pw_offload_page, 0, 1, B.PW_GATE, wrong_shape)
        expect(ARG_ERR, ctx.pw_offload_page, 0, 99, B.PW_GATE, pages[0])
        expect(3, ctx.pw_page_state, 0, 1, B.PW_GATE, 5)
        expect(STATE_ERR, ctx.pw_reload_page, 0, 1, B.PW_GATE, 16, torch.empty(16, dtype=torch.uint8))
        assert ctx.pw_page_state(0, 1, B.PW_GATE, 8) == B.PW_STATE_GPU_RESIDENT
        assert ctx.pw_page_state(0, 1, B.PW_GATE, 16) == B.PW_STATE_NONE
        assert ctx.pw_launch_count() == n0
    finally:
        ctx.close()


def test_planes_leave_and_return_following_the_oracle():
    """A row that holds overlaid bit-planes: the precision is lowered by publishing the same buffers at fewer
    bits, the planes above it move to host memory, and come back before the precision is raised again."""
    from oracle import oracle as orc
    from oracle import planes as PL
    from oracle import residency as R
    cfg = synth.LayerConfig("planes_res", 4, 2, 256, 512, 24, routing="normal")
    ctx = make_ctx(cfg, n_layers=1)
    try:
        blocks, refs, entries = [], [], []
        for e in range(cfg.n_experts):
            for u in range(3):
                w = synth.block_weights(cfg, 0, e, u, device="cuda")
                blk = ctx.pw_quantize_planes(w)
                blocks.append(blk)
                refs.append(PL.quantize_planes(w.cpu().numpy()))
                entries.append((0, e, u, blk.at(4)))
        ctx.pw_set_page_table(entries)
        e, u = 1, B.PW_UP
        row, blk = (0, e, u), blocks[e * 3 + u]
        _, top_bytes, bit_bytes = B.pw_plane_bytes(blk.rows, blk.cols)
        orow = R.PlaneRow(top_bytes, bit_bytes)
        orow.commit(4)
        x = synth.activations(cfg, device="cuda")
        lg = synth.router_logits(cfg, device="cuda")

        def forward_matches(q):
            views = [PL.view(r, q if i == e * 3 + u else 4) for i, r in enumerate(refs)]
            out = ctx.pw_moe_forward(0, x, lg, cfg.top_k)
            ref = orc.moe_forward(x.cpu().numpy(), lg.cpu().numpy(), cfg.top_k, views)
            d = out.cpu().numpy().astype(np.float64) - ref
            assert np.abs(d).max() <= 2e-2 and np.linalg.norm(d) / np.linalg.norm(ref) <= 5e-3
            return out.clone()

        def same_states():
            for p in (3, 4):
                assert ctx.pw_plane_state(*row, p) == orow.state[p]

        out4 = forward_matches(4)
        same_states()
        for p in (3, 4):                                            # q_i = 4 reads both planes
            expect(STATE_ERR, ctx.pw_offload_plane, *row, blk, p)
            with pytest.raises(R.IllegalTransition):
                orow.offload(p)
        # lower to 2 bits (a new header, no kernel), then both planes move out on a side stream
        ctx.pw_set_page_table([(0, e, u, blk.at(2))])
        orow.commit(2)
        forward_matches(2)
        image1, image0 = blk.bit1.clone(), blk.bit0.clone()
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            torch.cuda._sleep(200_000_000)                          # ~0.1 s: the copies behind it cannot have finished
            host1 = ctx.pw_offload_plane(*row, blk, 3, stream=side)
            host0 = ctx.pw_offload_plane(*row, blk, 4, stream=side)
        orow.offload(3)
        orow.offload(4)
        same_states()                                               # in transfer
        expect(STATE_ERR, ctx.pw_set_page_table, [(0, e, u, blk.at(3))])
        with pytest.raises(R.IllegalTransition):
            orow.commit(3)
        side.synchronize()
        orow.transfer_done(3)
        orow.transfer_done(4)
        same_states()                                               # CPU-resident
        assert orow.gpu_bytes() == top_bytes
        assert torch.equal(host1, image1.cpu()) and torch.equal(host0, image0.cpu())
        blk.bit1.fill_(0xEE)                                        # the device buffers are released (here: trashed)
        blk.bit0.fill_(0xEE)
        forward_matches(2)                                          # the 2-bit view does not touch them
        expect(STATE_ERR, ctx.pw_set_page_table, [(0, e, u, blk.at(3))])
        expect(STATE_ERR, ctx.pw_offload_plane, *row, blk, 3)       # already away
        expect(ARG_ERR, ctx.pw_reload_plane, *row, 3, host0)        # not the buffer plane 3 went to
        # raise to 3 bits: plane 3 comes back first
        new1 = ctx.pw_reload_plane(*row, 3, host1, stream=side)
        orow.reload(3)
        side.synchronize()
        orow.transfer_done(3)
        same_states()
        back = B.PlanePage(blk.rows, blk.cols, _buffers=(blk.top, new1, blk.bit0), bits=3)
        ctx.pw_set_page_table([(0, e, u, back)])
        orow.commit(3)
        forward_matches(3)
        expect(STATE_ERR, ctx.pw_set_page_table, [(0, e, u, back.at(4))])   # plane 4 is still on the host
        new0 = ctx.pw_reload_plane(*row, 4, host0, stream=side)
        orow.reload(4)
        side.synchronize()
        orow.transfer_done(4)
        full = B.PlanePage(blk.rows, blk.cols, _buffers=(blk.top, new1, new0), bits=4)
        ctx.pw_set_page_table([(0, e, u, full)])
        orow.commit(4)
        same_states()
        assert torch.equal(new1, image1) and torch.equal(new0, image0)
        assert torch.equal(forward_matches(4), out4)                # the bits of the first call
        assert orow.gpu_bytes() == top_bytes + 2 * bit_bytes
        assert ctx.pw_last_device_status() == 0
    finally:
        ctx.close()
