"""The failure path of the expert-FFN kernels: a device-side wait that runs out must make the kernel return
with PW_ERR_TIMEOUT in the status word (no trap, no fault, no unbounded spin), leave the context usable, and
the next ordinary call must be correct again.  The wait is made to run out safely: the wait limit is lowered
to a few milliseconds and a test hook keeps the token-tile producer of the gate/up kernel from arming its
second tile, so that the roles that depend on it give up one after the other."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import build_layer, error_metrics, export_to_oracle, make_ctx

pytestmark = pytest.mark.gpu


def test_wait_runs_out_then_context_recovers(orc):
    cfg = synth.CONFIGS["tiny_cover"]
    ctx = make_ctx(cfg)
    try:
        pages, _ = build_layer(ctx, cfg, 0)
        x = synth.activations(cfg, device="cuda")
        logits = synth.router_logits(cfg, device="cuda")
        opages = [export_to_oracle(ctx, p, orc) for p in pages]
        ref = orc.moe_forward(x.cpu().numpy(), logits.cpu().numpy(), cfg.top_k, opages)
        good = ctx.pw_moe_forward(0, x, logits, cfg.top_k).clone()
        assert ctx.pw_last_device_status() == 0
        ctx.pw_debug_set_wait(polls=200, hook=1)             # the 4 ms build; the second token tile never comes
        ctx.pw_moe_forward(0, x, logits, cfg.top_k)
        torch.cuda.synchronize()                              # the call returns: every wait is bounded
        assert ctx.pw_last_device_status() == 8               # PW_ERR_TIMEOUT, and reading it clears it
        assert ctx.pw_last_device_status() == 0
        ctx.pw_debug_set_wait(polls=0, hook=0)                # defaults again
        for _ in range(2):
            out = ctx.pw_moe_forward(0, x, logits, cfg.top_k)
            torch.cuda.synchronize()
            assert ctx.pw_last_device_status() == 0
            assert torch.equal(out, good)                      # tensor memory, barriers and counters start clean
        max_abs, rel_f = error_metrics(out.cpu().numpy(), ref)
        assert max_abs <= 2e-2 and rel_f <= 5e-3
    finally:
        ctx.close()
