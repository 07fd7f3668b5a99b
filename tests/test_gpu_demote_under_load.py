"""Runtime demotion under load (small replica of the 32-layer configuration): blocks are demoted
16->4 and then 4->2 with pw_demote_block on a side stream while forward calls keep running on the main
stream; every finished demote is published with pw_set_page_table at the next call boundary.  Every
demoted page is compared bit for bit with the oracle's chain, and a forward call of every table epoch
is compared with the oracle run on that epoch's pages."""
import numpy as np
import pytest
import torch

from paper_2607_16184_b200 import binding as B
from paper_2607_16184_b200 import synth

from util_gpu import error_metrics, export_to_oracle, pages_equal

pytestmark = pytest.mark.gpu


def test_demote_schedule_overlapping_forward(orc):
    cfg = synth.LayerConfig("demote_small", 8, 2, 512, 1024, 48, n_layers=3, routing="zipf", zipf_a=1.1,
                            bit_rule="all16")
    ctx = B.Context(cfg.n_layers, cfg.n_experts, 0, cfg.hidden, cfg.ffn, cfg.tokens, cfg.top_k)
    pages, opages = {}, {}
    for l in range(cfg.n_layers):
        entries = []
        for e in range(cfg.n_experts):
            for u in range(3):
                w = synth.block_weights(cfg, l, e, u, device="cuda")
                pages[(l, e, u)] = ctx.pw_quantize_block(w, 16)
                opages[(l, e, u)] = orc.quantize_block(w.cpu().numpy(), 16)
                entries.append((l, e, u, pages[(l, e, u)]))
        ctx.pw_set_page_table(entries)
    xs = [synth.activations(cfg, l, device="cuda") for l in range(cfg.n_layers)]
    lgs = [synth.router_logits(cfg, l, device="cuda") for l in range(cfg.n_layers)]
    sched = synth.demote_schedule(cfg)                  # a third of the blocks
    assert len(sched) == cfg.n_layers * cfg.n_experts
    main, side = torch.cuda.current_stream(), torch.cuda.Stream()
    side.wait_stream(main)
    keep_alive, checks = [], []
    step = 0
    for phase_bits in (4, 2):                           # 16 -> 4 for all scheduled blocks, then 4 -> 2
        inflight = []
        for (l, e, u) in sched:
            new = ctx.pw_demote_block(pages[(l, e, u)], phase_bits, stream=side)
            ev = torch.cuda.Event()
            ev.record(side)
            inflight.append(((l, e, u), new, ev))
            # forward calls keep running while the side stream works; publish what has finished
            layer = step % cfg.n_layers
            done = [x for x in inflight if x[2].query()]
            if done:
                for key, pg, ev2 in done:
                    main.wait_event(ev2)
                    keep_alive.append(pages[key])       # the old page stays alive: earlier calls may still read it
                    pages[key] = pg
                    opages[key] = orc.demote_block(opages[key], phase_bits)
                ctx.pw_set_page_table([(k[0], k[1], k[2], pg) for k, pg, _ in done])
                inflight = [x for x in inflight if not any(x is d for d in done)]
            out = ctx.pw_moe_forward(layer, xs[layer], lgs[layer], cfg.top_k)
            if step % 5 == 0:
                snap = [opages[(layer, ee, uu)] for ee in range(cfg.n_experts) for uu in range(3)]
                checks.append((layer, out.clone(), snap))
            step += 1
        for key, pg, ev2 in inflight:                   # drain the phase
            ev2.synchronize()
            keep_alive.append(pages[key])
            pages[key] = pg
            opages[key] = orc.demote_block(opages[key], phase_bits)
        if inflight:
            ctx.pw_set_page_table([(k[0], k[1], k[2], pg) for k, pg, _ in inflight])
    torch.cuda.synchronize()
    assert ctx.pw_last_device_status() == 0
    for key in sched:                                   # every demoted page, bit for bit, after the chain
        assert pages[key].bits == 2
        assert pages_equal(export_to_oracle(ctx, pages[key], orc), opages[key]), key
        assert ctx.pw_query_row(*key).page.bits == 2
    for layer, out, snap in checks:                     # forwards saw exactly the table of their epoch
        ref = orc.moe_forward(xs[layer].cpu().numpy(), lgs[layer].cpu().numpy(), cfg.top_k, snap)
        max_abs, rel_f = error_metrics(out.cpu().numpy(), ref)
        assert max_abs <= 2e-2 and rel_f <= 5e-3, (layer, max_abs, rel_f)
    ctx.close()
