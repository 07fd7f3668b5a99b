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
